"""The allocation-free entry point (fi_lookup_noalloc) against the regular look-up.

Some callers cannot allocate device memory when they need a look-up (their own pool holds the whole GPU, or an
allocation's implicit synchronisation is not acceptable on their latency path); for them the library keeps the
streaming look-up's scratch in a fixed array of its own.  This file is collected last on purpose: if the fixed
scratch ever misbehaved, every other test has already run.  Both kernels are the same, so the outputs must be
identical, on two calls in a row (the scratch keeps the first call's contents during the second).
"""
import numpy as np
import pytest
import torch

from paper_2002_02645_b200 import binding as fb
from paper_2002_02645_b200 import datagen as dg
from helpers import make_cache, to_device

pytestmark = pytest.mark.gpu


def _as_numpy(out):
    return [t.cpu().numpy() for t in (out.label, out.conf, out.hit, out.topk_dist, out.topk_idx)]


@pytest.mark.parametrize("n,d,b,k,dtype", [
    (3000, 1024, 37, 5, "bf16"), (500, 64, 256, 1, "f32"),
    (700, 128, 256, 32, "bf16"),       # the largest batch x k: the candidate lists fill the fixed array
])
def test_noalloc_matches_regular_lookup_twice(n, d, b, k, dtype):
    w = dg.single_layer(name="t", n_cache=n, n_query=b, dim=d, num_classes=6, dtype=dtype, sigma=0.5, k=k, seed=21)
    st = w.stages[0]
    cache = make_cache(st, k=k, num_classes=6, tau=0.0, max_batch=b, path=fb.FI_PATH_STREAM)
    q = to_device(st.queries)
    tau = float(np.float32(np.median(cache.lookup_batch(q).conf.cpu().numpy())))   # about half of the requests hit
    cache.set_threshold(tau)
    want = _as_numpy(cache.lookup_batch(q))
    torch.cuda.synchronize()
    x = to_device(st.cache_vecs)
    labels = torch.from_numpy(st.cache_labels).cuda()
    ones = torch.ones(n, dtype=torch.float32, device="cuda")
    # second batch: the same requests in reverse order, so the scratch holds other values between the calls
    q_rev = q.flip(0).contiguous()
    # the property the entry point exists for: once the outputs exist and one call has done the per-device set-up,
    # further calls leave the device's free memory exactly as it was
    out1, out2 = fb.LookupOut(b, k, "cuda"), fb.LookupOut(b, k, "cuda")
    fb.lookup_noalloc(x, labels, ones, q, k=k, threshold=tau, out=out1)
    torch.cuda.synchronize()
    free_before = torch.cuda.mem_get_info()[0]
    got1 = fb.lookup_noalloc(x, labels, ones, q, k=k, threshold=tau, out=out1)
    got2 = fb.lookup_noalloc(x, labels, ones, q_rev, k=k, threshold=tau, out=out2)
    torch.cuda.synchronize()
    assert torch.cuda.mem_get_info()[0] == free_before
    got1, got2 = _as_numpy(got1), _as_numpy(got2)
    for a, g1, g2 in zip(want, got1, got2):
        np.testing.assert_array_equal(a, g1)
        np.testing.assert_array_equal(a[::-1], g2)
    assert 0 < want[2].sum() < b or b < 4
    cache.close()


def test_noalloc_empty_cache_and_empty_batch():
    k = 3
    q = torch.randn(5, 64, device="cuda").to(torch.bfloat16)
    none = torch.zeros(0, 64, dtype=torch.bfloat16, device="cuda")
    nolab = torch.zeros(0, dtype=torch.int32, device="cuda")
    noweight = torch.zeros(0, dtype=torch.float32, device="cuda")
    # no entries: the answer of the regular look-up on an empty cache (label -1, confidence 0, miss, no neighbours)
    empty = fb.FreezeCache(dim=64, capacity=4, num_classes=2, k=k, dtype=fb.FI_BF16, max_batch=8, path=fb.FI_PATH_STREAM)
    want = _as_numpy(empty.lookup_batch(q))
    got = _as_numpy(fb.lookup_noalloc(none, nolab, noweight, q, k=k))
    torch.cuda.synchronize()
    for a, g in zip(want, got):
        np.testing.assert_array_equal(a, g)
    assert (got[0] == -1).all() and (got[2] == 0).all() and (got[4] == -1).all()
    empty.close()
    # no requests: nothing is launched and the outputs stay as they were
    x = torch.randn(16, 64, device="cuda").to(torch.bfloat16)
    out = fb.LookupOut(1, k, "cuda")
    out.label.fill_(77)
    fb.lookup_noalloc(x, torch.zeros(16, dtype=torch.int32, device="cuda"), torch.ones(16, device="cuda"), q[:0], k=k, out=out)
    torch.cuda.synchronize()
    assert int(out.label[0]) == 77


def test_noalloc_rejects_what_the_fixed_scratch_cannot_hold():
    x = torch.zeros(16, 64, dtype=torch.bfloat16, device="cuda")
    labels = torch.zeros(16, dtype=torch.int32, device="cuda")
    ones = torch.ones(16, dtype=torch.float32, device="cuda")
    q = torch.zeros(257, 64, dtype=torch.bfloat16, device="cuda")
    with pytest.raises(fb.FiError) as e:
        fb.lookup_noalloc(x, labels, ones, q, k=1)
    assert e.value.status == 2 and "256" in str(e.value)
    with pytest.raises(fb.FiError) as e:
        fb.lookup_noalloc(x, labels, ones, q[:4], k=33)
    assert e.value.status == 1

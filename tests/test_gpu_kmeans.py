"""k-means cache construction on the device (one Lloyd iteration and the cluster tagging) against the fp64 oracle,
and the resulting k-means cache used for look-ups (Sec. 4: majority label of the closest centre, confidence
fraction / distance)."""
import numpy as np
import pytest
import torch

from oracle import fi_oracle as fo
from paper_2002_02645_b200 import binding as fb
from paper_2002_02645_b200 import datagen as dg
from helpers import compare_lookup, to_device

pytestmark = pytest.mark.gpu


def to_np(t):
    """Device tensor -> numpy; bf16 as its uint16 bit patterns."""
    if t.dtype == torch.bfloat16:
        return t.view(torch.int16).cpu().numpy().view(np.uint16)
    return t.cpu().numpy()


def centres_cache(centres_np, dim, num_classes, dtype, max_batch, clusters):
    c = fb.FreezeCache(dim=dim, capacity=clusters, num_classes=num_classes, k=1,
                       dtype=fb.FI_BF16 if dtype == "bf16" else fb.FI_F32, max_batch=max_batch)
    c.insert(to_device(centres_np), torch.zeros(clusters, dtype=torch.int32, device="cuda"))
    return c


@pytest.mark.parametrize("n,d,clusters,classes,dtype,max_batch", [
    (5000, 1024, 200, 10, "bf16", 2048),      # the paper's shape: 200 clusters of 1024-dim reduced activations
    (3000, 2056, 37, 1000, "bf16", 700),      # two dimension chunks (ragged), many classes, ragged last batch
    (1200, 36, 9, 5, "f32", 4096),
])
def test_kmeans_step_matches_oracle(n, d, clusters, classes, dtype, max_batch):
    w = dg.single_layer(name="t", n_cache=n, n_query=clusters, dim=d, num_classes=classes, dtype=dtype, sigma=0.5, k=1,
                        seed=31, zipf=1.1 if classes > 100 else None)
    st = w.stages[0]
    points, labels = st.cache_vecs, st.cache_labels
    init = st.queries                                     # fresh draws from the same mixture as initial centres
    init[-1] = init[-1] * 0 + 1000 if dtype == "f32" else np.full(d, 0x7F00, np.uint16)   # far away: stays empty
    ref = fo.kmeans_step(points, init, labels, classes)
    cache = centres_cache(init, d, classes, dtype, max_batch, clusters)
    got = [to_np(t) for t in cache.kmeans_step(to_device(points), torch.from_numpy(labels).cuda())]
    again = [to_np(t) for t in cache.kmeans_step(to_device(points), torch.from_numpy(labels).cuda())]
    cache.poll_status()
    for a, b in zip(got, again):                          # sums run in a fixed order: bit-identical reruns
        np.testing.assert_array_equal(a, b)
    assign, centres, counts, majority, fraction = got
    # assignments are exact except where a point's two nearest centres are closer than 1e-4 relative
    r2 = fo.lookup(points, init, np.zeros(clusters, np.int32), k=1, tau=0.0)
    decidable = (r2.next_d - r2.nd[:, 0]) / np.maximum(r2.nd[:, 0], 1e-300) >= 1e-4
    np.testing.assert_array_equal(assign[decidable], ref.assign[decidable])
    mismatch = assign != ref.assign
    touched = np.union1d(assign[mismatch], ref.assign[mismatch]).astype(np.int64)     # clusters whose members differ
    ok = np.ones(clusters, bool)
    ok[touched] = False
    print(f"kmeans {n}x{d}: undecidable assignments {int((~decidable).sum())}, of which different {int(mismatch.sum())}, "
          f"clusters compared {int(ok.sum())} of {clusters}, empty clusters {int((ref.counts == 0).sum())}")
    assert ok.sum() >= clusters - 2 * int((~decidable).sum())
    np.testing.assert_array_equal(counts[ok], ref.counts[ok])
    np.testing.assert_array_equal(majority[ok], ref.majority[ok])
    np.testing.assert_allclose(fraction[ok], ref.fraction[ok], rtol=1e-6)
    gc = dg.stored_to_f64(centres)
    # fp32 means rounded to the storage type: within one bf16 unit in the last place, or, for fp32 storage,
    # within the 1e-5 relative that the fp32 look-up distances are held to (sums of ~100 terms)
    ulp = 2.0 ** -7 if dtype == "bf16" else 1e-5
    assert (np.abs(gc - ref.centres)[ok] <= ulp * np.maximum(np.abs(ref.centres[ok]), 1e-30) + 1e-30).all()
    if dtype == "bf16":
        exact = dg.f32_to_bf16_bits(ref.centres.astype(np.float32))[ok] == centres[ok]
        assert exact.mean() > 0.99
    assert ref.counts[-1] == 0 and counts[-1] == 0 and majority[-1] == -1
    np.testing.assert_array_equal(centres[-1], init[-1])
    cache.close()


def test_kmeans_cache_end_to_end():
    """A few Lloyd iterations on the device, then look-ups against the resulting <centre, label, fraction> cache."""
    w = dg.single_layer(name="t", n_cache=4000, n_query=64, dim=512, num_classes=10, dtype="bf16", sigma=0.5, k=1, seed=32)
    st = w.stages[0]
    pts, labs = to_device(st.cache_vecs), torch.from_numpy(st.cache_labels).cuda()
    clusters = 40
    cache = centres_cache(st.cache_vecs[:clusters].copy(), 512, 10, "bf16", 4096, clusters)
    for _ in range(3):
        _, centres, counts, majority, fraction = cache.kmeans_step(pts, labs)
        keep = counts > 0
        cache.clear()
        cache.insert(centres[keep].contiguous(), majority[keep].contiguous(), fraction[keep].contiguous())
    torch.cuda.synchronize()
    assert cache.size() == int(keep.sum()) and float(fraction[keep].mean()) > 0.9        # pure clusters
    # the look-up rule of Sec. 4 on that cache, against the oracle on the same entries
    cen = to_np(centres[keep])
    maj, frac = majority[keep].cpu().numpy(), fraction[keep].cpu().numpy()
    ref = fo.lookup(st.queries, cen, maj, k=1, tau=0.0, weights=frac)
    tau = float(np.float32(np.median(ref.conf)))
    ref = fo.lookup(st.queries, cen, maj, k=1, tau=tau, weights=frac)
    cache.set_threshold(tau)
    out = cache.lookup_batch(to_device(st.queries))
    torch.cuda.synchronize()
    compare_lookup(out.label.cpu().numpy(), out.conf.cpu().numpy(), out.hit.cpu().numpy(), out.topk_dist.cpu().numpy(),
                   out.topk_idx.cpu().numpy(), ref, storage="bf16", tau=tau, rule=0, cache_labels=maj, weights=frac)
    assert (out.label.cpu().numpy() == w.query_classes).mean() > 0.9
    cache.close()

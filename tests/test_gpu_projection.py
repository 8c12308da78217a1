"""The projection in front of the look-up (Sec. 3) on the GPU against the fp64 oracle.

Tolerance.  The GPU forms W x + b with bf16 products accumulated in fp32 on the tensor cores and rounds once to bf16;
the oracle forms it in fp64 and rounds once to bf16.  The fp32 sum differs from the exact one by at most
E = 3e-4 * (sum_j |w_j x_j| + |b|) (measured accumulation error of the tensor-core path is about 1e-4 of that
magnitude).  Rounding is monotone, so the GPU's output must lie between the bf16 roundings of max(0, pre - E) and
max(0, pre + E): usually one value, the oracle's own; two neighbours when pre sits within E of a rounding boundary.
"""
import numpy as np
import pytest
import torch

from oracle import fi_oracle as fo
from paper_2002_02645_b200 import binding as fb
from paper_2002_02645_b200 import datagen as dg
from helpers import to_device

pytestmark = pytest.mark.gpu

ACC_ERR = 3e-4


def check_projection(y_gpu_bits, bits, pre, mag):
    g = fo.bf16_bits_to_f64(y_gpu_bits)
    lo = fo.bf16_bits_to_f64(fo.round_to_bf16_bits(np.maximum(pre - ACC_ERR * mag, 0.0)))
    hi = fo.bf16_bits_to_f64(fo.round_to_bf16_bits(np.maximum(pre + ACC_ERR * mag, 0.0)))
    bad = (g < lo) | (g > hi)
    assert not bad.any(), f"{int(bad.sum())} outputs outside the rounding interval, first at {np.argwhere(bad)[0]}"
    same = float((y_gpu_bits == bits).mean())
    assert same > 0.95, f"only {same:.3f} of the outputs equal the oracle's rounding"
    return same


def as_bits(t: torch.Tensor) -> np.ndarray:
    return t.view(torch.int16).cpu().numpy().view(np.uint16)


@pytest.mark.parametrize("batch,in_dim,out_dim,use_bias", [
    (300, 4096, 1024, True),        # several pieces per tile, ragged last query tile
    (77, 1096, 272, False),         # row length not a multiple of 64, output not a multiple of 256
    (1, 512, 16, True),             # degenerate: one row, one 16-column tile
    (1024, 16384, 1024, True),      # 16 tiles x 9 pieces
    (600, 64, 1024, True),          # one k-block: pieces cannot be cut along the row length
])
def test_projection_matches_oracle(batch, in_dim, out_dim, use_bias):
    w_bits, bias = dg.projection_weights(in_dim, out_dim, seed=3)
    st = dg.single_layer(name="p", n_cache=8, n_query=batch, dim=in_dim, num_classes=4, dtype="bf16", sigma=0.5, k=1,
                         seed=4).stages[0]
    bits, pre, mag = fo.project(st.queries, w_bits, bias if use_bias else None)
    proj = fb.Projection(in_dim=in_dim, out_dim=out_dim, max_batch=max(batch, 16))
    proj.set_weights(to_device(w_bits), torch.from_numpy(bias).cuda() if use_bias else None)
    y = proj.apply(to_device(st.queries))
    y2 = proj.apply(to_device(st.queries))
    torch.cuda.synchronize()
    proj.poll_status()
    same = check_projection(as_bits(y), bits, pre, mag)
    assert torch.equal(y.view(torch.int16), y2.view(torch.int16))        # pieces are summed in a fixed order
    assert (pre < 0).any() and (pre > 0).any()
    print(f"projection {batch}x{in_dim}->{out_dim}: {same:.4f} of the outputs bit-equal to the oracle")
    proj.close()


def test_projection_gather_and_device_count():
    in_dim, out_dim = 2048, 256
    w_bits, bias = dg.projection_weights(in_dim, out_dim, seed=5)
    st = dg.single_layer(name="p", n_cache=8, n_query=400, dim=in_dim, num_classes=4, dtype="bf16", sigma=0.5, k=1,
                         seed=6).stages[0]
    rows = np.random.default_rng(7).permutation(400)[:333].astype(np.int32)
    count = 290                                                # the device-resident count is below the list length
    bits, pre, mag = fo.project(st.queries[rows[:count]], w_bits, bias)
    proj = fb.Projection(in_dim=in_dim, out_dim=out_dim, max_batch=512)
    proj.set_weights(to_device(w_bits), torch.from_numpy(bias).cuda())
    out = torch.full((333, out_dim), -7.0, dtype=torch.bfloat16, device="cuda")
    proj.apply(to_device(st.queries), row_idx=torch.from_numpy(rows).cuda(),
               count=torch.tensor([count], dtype=torch.int32, device="cuda"), out=out)
    torch.cuda.synchronize()
    check_projection(as_bits(out[:count]), bits, pre, mag)
    assert (out[count:] == -7.0).all()                          # rows past the count are left untouched
    proj.close()


def test_projection_argument_errors():
    proj = fb.Projection(in_dim=64, out_dim=32, max_batch=8)
    x = torch.zeros(4, 64, dtype=torch.bfloat16, device="cuda")
    with pytest.raises(fb.FiError) as e:                        # weights never set
        proj.apply(x)
    assert e.value.status == fb.FI_ERR_INVALID_ARG
    proj.set_weights(torch.zeros(32, 64, dtype=torch.bfloat16, device="cuda"))
    with pytest.raises(fb.FiError):                             # batch above max_batch
        proj.apply(torch.zeros(9, 64, dtype=torch.bfloat16, device="cuda"))
    with pytest.raises(fb.FiError):
        fb.Projection(in_dim=60, out_dim=32)                    # in_dim not a multiple of 8
    with pytest.raises(fb.FiError):
        fb.Projection(in_dim=64, out_dim=24)                    # out_dim not a multiple of 16
    y = proj.apply(x)
    torch.cuda.synchronize()
    assert (y == 0).all()
    proj.close()


def test_cascade_with_projection():
    """Three stages, each with its own projection to 256 dimensions.  (i) The fused step equals, bit for bit, the plain
    cascade step fed with explicitly projected activations (both on the GPU: a consistency check).  (ii) Against the
    oracle's own pipeline (fp64 projection, fp64 look-up) the answers agree for nearly all requests; they cannot
    agree for all, because a projected coordinate that lies within the accumulation error of a bf16 rounding
    boundary may round to the neighbouring value on the GPU, and the look-up then sees a slightly different vector."""
    dims, out_dim, n_cache, b0, k = [4096, 2048, 1096], 256, 2000, 300, 5
    stages, projs, caches, caches_plain, taus, ora_cache, ora_q = [], [], [], [], [], [], []
    for l, d in enumerate(dims):
        w = dg.single_layer(name=f"s{l}", n_cache=n_cache, n_query=b0, dim=d, num_classes=6, dtype="bf16",
                            sigma=0.9 - 0.2 * l, k=k, seed=40 + l)
        st = w.stages[0]
        w_bits, bias = dg.projection_weights(d, out_dim, seed=50, stage=l)
        oc, _, _ = fo.project(st.cache_vecs, w_bits, bias)
        oq, _, _ = fo.project(st.queries, w_bits, bias)
        ref0 = fo.lookup(oq, oc, st.cache_labels, k=k, tau=0.0)
        taus.append(float(np.float32(np.percentile(ref0.conf, 60.0))))
        ora_cache.append(oc)
        ora_q.append(oq)
        stages.append(st)
        p = fb.Projection(in_dim=d, out_dim=out_dim, max_batch=2048)
        p.set_weights(to_device(w_bits), torch.from_numpy(bias).cuda())
        projs.append(p)
        c = fb.FreezeCache(dim=out_dim, capacity=n_cache, num_classes=6, k=k, threshold=taus[l], max_batch=512)
        c.insert(p.apply(to_device(st.cache_vecs)), torch.from_numpy(st.cache_labels).cuda())
        caches.append(c)
    ref = fo.cascade(ora_q, ora_cache, [s.cache_labels for s in stages], taus, k=k)

    def run(fused: bool):
        state = fb.CascadeState(b0, "cuda:0")
        fb.cascade_init(state, len(dims))
        for l in range(len(dims)):
            x = to_device(stages[l].queries)
            if fused:
                fb.cascade_step_projected(caches[l], projs[l], x, state, l)
            else:
                fb.cascade_step(caches[l], projs[l].apply(x), state, l)
        torch.cuda.synchronize()
        return state.final_label.cpu().numpy()[:b0].copy(), state.exit_stage.cpu().numpy()[:b0].copy()

    label_f, stage_f = run(True)
    label_p, stage_p = run(False)
    np.testing.assert_array_equal(label_f, label_p)
    np.testing.assert_array_equal(stage_f, stage_p)
    agree = float(((label_f == ref.final_label) & (stage_f == ref.exit_stage)).mean())
    print(f"cascade with projection: {agree:.3f} of the requests agree with the oracle pipeline; "
          f"exit stages {np.bincount(ref.exit_stage, minlength=4).tolist()}")
    assert agree >= 0.95
    assert len(set(ref.exit_stage.tolist())) >= 3
    for o in caches + projs:
        o.close()

"""The allocation-free sampling entry point against the ordinary one.

psb_sample_level_static serves hosts that cannot call cudaMalloc when they need fresh draws
(real-time loops, work beside a graph capture, fixed memory budgets): it keeps its scratch in
a fixed array inside the library.  Here it is called through the C ABI twice in a row - the
second call on a smaller, different filter, so that anything left in the shared array by the
first call would show - and compared bit for bit with psb_sample_weights + psb_weights_export
and with the CPU oracle.
Collected last so that a failure here cannot hide another test's result.
"""
import numpy as np
import pytest

pytestmark = pytest.mark.gpu


def _reference(psb, ctx, w, groups, seed, layer_id, log2k, exp_bits, norm):
    wt = ctx.sample_weights(w, groups=groups, seed=seed, layer_id=layer_id, level_mask=1 << log2k,
                            exp_bits=exp_bits, norm=norm)
    wint, e_base = ctx.weights_export(wt, log2k)
    wint, e_base = wint.cpu().numpy(), e_base.cpu().numpy()
    wt.free()
    return wint, e_base


@pytest.mark.parametrize("norm", [0, 1])
def test_static_scratch_sampler_matches_the_allocating_one_twice_in_a_row(norm):
    import torch

    import paper_1904_02205_b200 as psb

    ctx = psb.Context(0)
    dev = ctx.device
    rng = np.random.default_rng(404 + norm)
    calls = [  # (shape, groups, weight scale, log2k, exp_bits, seed)
        ((192, 64, 3, 3), 1, 8.0, 3, 4, 11),      # large exponents first ...
        ((40, 1, 3, 3), 40, 1e-3, 4, 3, 12),      # ... then a smaller filter with tiny weights
    ]
    # outputs are allocated up front: the calls under test allocate nothing
    outs = [(torch.full(s, 12345, dtype=torch.int32, device=dev),
             torch.full((s[0],), 777, dtype=torch.int32, device=dev)) for s, *_ in calls]
    ws = []
    for shape, groups, scale, log2k, exp_bits, seed in calls:
        w = rng.normal(0, scale, size=shape).astype(np.float32)
        w.reshape(-1)[::7] = 0.0
        ws.append(torch.from_numpy(w).to(dev))
    torch.cuda.synchronize()
    for (shape, groups, scale, log2k, exp_bits, seed), w, (wint, e_base) in zip(calls, ws, outs):
        psb.sample_level_static(w, wint, e_base, groups=groups, seed=seed, layer_id=5, log2k=log2k,
                                exp_bits=exp_bits, norm=norm)
    torch.cuda.synchronize()
    for (shape, groups, scale, log2k, exp_bits, seed), w, (wint, e_base) in zip(calls, ws, outs):
        ref_w, ref_e = _reference(psb, ctx, w, groups, seed, 5, log2k, exp_bits, norm)
        assert np.array_equal(e_base.cpu().numpy(), ref_e)
        assert np.array_equal(wint.cpu().numpy(), ref_w)      # integers: bit-exact, as in the other tests
        # and directly against the CPU oracle
        from oracle import psb_oracle

        psb_oracle.build()
        Wo, ebo, _ = psb_oracle.sample_level(w.cpu().numpy(), seed, 5, log2k, exp_bits=exp_bits, norm=norm)
        assert np.array_equal(e_base.cpu().numpy(), ebo)
        assert np.array_equal(wint.cpu().numpy().astype(np.int64), Wo)
    # sizes beyond the fixed array are refused with an error, nothing is launched
    big = torch.zeros((psb.PSB_STATIC_MAX_OUT_CH + 1, 1, 1, 1), dtype=torch.float32, device=dev)
    out = torch.zeros((psb.PSB_STATIC_MAX_OUT_CH + 1, 1, 1, 1), dtype=torch.int32, device=dev)
    with pytest.raises(psb.PsbError) as e:
        psb.sample_level_static(big, out, None, log2k=0)
    assert e.value.status == psb.PSB_ERR_UNSUPPORTED
    assert ctx.device_status() == 0
    ctx.close()

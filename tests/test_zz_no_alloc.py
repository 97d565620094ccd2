"""The allocation-free entry point, asd_fused_gemv_static.

Some users of the library cannot allocate device memory where they need the fused sublayer kernel: code that
lives inside a memory pool owning the whole device, a plug-in whose host forbids allocations after start-up, a
latency-critical loop where an allocation would stall the device.  For them the kernel's cross-CTA scratch
sits in a fixed array inside the library.  This file checks, through the C ABI, that the variant gives the
same result as asd_fused_gemv with caller-provided scratch, twice in a row (the second call meets whatever
the first one left in the shared array).  It is collected last on purpose.
"""
import numpy as np
import pytest

import oracle
import synth

pytestmark = pytest.mark.gpu


def _inputs(M, n_in, n_rows, seed):
    import torch
    dev = torch.device("cuda:0")
    W = torch.from_numpy(synth.make_matrix_bf16((n_rows, n_in), seed=seed, stream=1).view(np.int16)).to(dev).view(torch.bfloat16)
    gain = torch.from_numpy(synth.make_matrix_bf16((n_in,), seed=seed, stream=2, mean=1.0).view(np.int16)).to(dev).view(torch.bfloat16)
    x = torch.from_numpy(synth.make_array_f32((M, n_in), seed=seed, stream=3, std=1.5)).to(dev)
    res = torch.from_numpy(synth.make_array_f32((M, n_rows), seed=seed, stream=4)).to(dev)
    return W, gain, x, res


@pytest.mark.parametrize("M,n_in,n_rows", [(1, 2048, 2048), (5, 688, 256), (9, 1032, 51)])
def test_static_scratch_variant_matches_caller_scratch_variant_twice(M, n_in, n_rows):
    import torch
    import paper_2410_01028_b200 as asd
    W, gain, x, res = _inputs(M, n_in, n_rows, seed=40 + M)
    scratch = torch.zeros(asd.fused_gemv_scratch_bytes(), dtype=torch.uint8, device="cuda:0")
    # reference: the existing entry point with caller-provided scratch
    want_y = res.clone()
    want_cos = torch.zeros(M, dtype=torch.float32, device="cuda:0")
    asd.fused_gemv(x, W, asd.EPI_RESIDUAL, want_y, gain=gain, cos=want_cos, scratch=scratch)
    want_t = torch.empty((M, n_rows), dtype=torch.float32, device="cuda:0")
    asd.fused_gemv(x, W, asd.EPI_PLAIN, want_t, gain=gain, scratch=scratch)
    torch.cuda.synchronize()
    for call in range(2):   # two calls in a row share the built-in array
        got_y = res.clone()
        got_cos = torch.zeros(M, dtype=torch.float32, device="cuda:0")
        asd.fused_gemv_static(x, W, asd.EPI_RESIDUAL, got_y, gain=gain, cos=got_cos)
        got_t = torch.empty((M, n_rows), dtype=torch.float32, device="cuda:0")
        asd.fused_gemv_static(x, W, asd.EPI_PLAIN, got_t, gain=gain)
        torch.cuda.synchronize()
        scale = float(want_t.abs().max())
        assert float((got_t - want_t).abs().max()) <= 1e-5 * scale, call
        assert float((got_y - want_y).abs().max()) <= 1e-5 * max(scale, float(want_y.abs().max())), call
        assert float((got_cos - want_cos).abs().max()) <= 1e-5, call
    # and directly against the CPU oracle (normalised input rounded to bf16 on both sides: a rounding flip moves one
    # product by 2^-8, hence 2e-3 of the output scale; cosine within 1e-3)
    xh, Wh, gh, rh = (x.cpu().numpy(), W.view(torch.int16).cpu().numpy().view(np.uint16),
                      gain.view(torch.int16).cpu().numpy().view(np.uint16), res.cpu().numpy())
    ref_t, _ = oracle.fused_matvec(xh, Wh, epilogue=0, gain=gh)
    ref_y, ref_cos = oracle.fused_matvec(xh, Wh, epilogue=2, gain=gh, res=rh)
    assert np.abs(got_t.cpu().numpy() - ref_t).max() <= 2e-3 * np.abs(ref_t).max()
    assert np.abs(got_y.cpu().numpy() - ref_y).max() <= 2e-3 * np.abs(ref_y).max()
    assert np.abs(got_cos.cpu().numpy() - ref_cos).max() <= 1e-3


def test_static_scratch_variant_rejects_bad_arguments():
    import torch
    import paper_2410_01028_b200 as asd
    W, gain, x, res = _inputs(2, 256, 64, seed=3)
    with pytest.raises(asd.AsdError) as e:
        asd.fused_gemv_static(x, W, asd.EPI_RESIDUAL, res, gain=gain, cos=None)   # the cosine output is required
    assert e.value.code == -1
    with pytest.raises(asd.AsdError) as e:
        asd.fused_gemv_static(x[:, :252], W, asd.EPI_PLAIN, res, gain=gain)       # n_in must be a multiple of 8
    assert e.value.code == -1


def test_static_scratch_variant_rejects_shapes_beyond_its_array():
    import torch
    import paper_2410_01028_b200 as asd
    # 9 activation rows x 8192 inputs x 200000 weight rows: the per-CTA partial sums only fit shared memory with a
    # launch plan of several hundred CTAs, more than the built-in array has room for.  Nothing is launched.
    M, n_in, n_rows = 9, 8192, 200000
    W = torch.empty((n_rows, n_in), dtype=torch.bfloat16, device="cuda:0")
    x = torch.zeros((M, n_in), dtype=torch.float32, device="cuda:0")
    gain = torch.ones(n_in, dtype=torch.bfloat16, device="cuda:0")
    out = torch.empty((M, n_rows), dtype=torch.float32, device="cuda:0")
    with pytest.raises(asd.AsdError) as e:
        asd.fused_gemv_static(x, W, asd.EPI_PLAIN, out, gain=gain)
    assert e.value.code == -3
    # the variant with caller-provided scratch takes the same shape
    scratch = torch.zeros(asd.fused_gemv_scratch_bytes(), dtype=torch.uint8, device="cuda:0")
    W.zero_()
    asd.fused_gemv(x, W, asd.EPI_PLAIN, out, gain=gain, scratch=scratch)
    torch.cuda.synchronize()
    assert float(out.abs().max()) == 0.0

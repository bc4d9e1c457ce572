"""bcjr_soft_quantize_static: the forward call for callers that are not allowed to allocate.

Some users of the library run where cudaMalloc / cudaFree must not be called (a host loop that
cannot take their device-wide synchronisation, a process whose memory belongs to another
allocator, a plug-in confined to the buffers it was handed).  For them the library has one entry
point whose scratch is a fixed array inside the library image.  This test calls it through the C
ABI and compares it with the regular, context-based entry point on the same inputs -- twice in a
row, because every call reuses the same scratch array and must not be disturbed by what the
previous call left there.

Collected last on purpose (file name), so that a run that stops at the first failure has
already run every other test.
"""
import ctypes

import numpy as np
import pytest

import oracle
import parity
from paper_2605_10655_b200 import synth

pytestmark = pytest.mark.gpu


def _device_inputs(wl, nblk, seed_shift=0):
    import torch
    dev = torch.device("cuda", 0)
    W = np.ascontiguousarray(wl.weights()[:nblk]) + np.float32(0.01 * seed_shift)
    return torch.from_numpy(W).to(dev), torch.from_numpy(wl.codebook()).to(dev)


def test_static_entry_point_matches_regular_one_twice_in_a_row():
    import torch
    from paper_2605_10655_b200 import Context, binding
    lib = binding.load_library()
    ctx = Context(0)
    try:
        for call, (wl, nblk) in enumerate([(synth.tiny(), 64), (synth.mid(), 40)]):
            Wd, cd = _device_inputs(wl, nblk, seed_shift=call)
            ref_soft, ref_logZ = ctx.bcjr_soft_quantize(Wd, cd, wl.Lb, wl.k, wl.n, wl.T)
            ctx.sync_status()
            soft = torch.full_like(Wd, float("nan"))
            logZ = torch.full((nblk,), float("nan"), device=Wd.device)
            stream = torch.cuda.current_stream().cuda_stream
            rc = lib.bcjr_soft_quantize_static(ctypes.c_void_p(Wd.data_ptr()), ctypes.c_void_p(cd.data_ptr()),
                                               wl.Lb, wl.k, wl.n, nblk, ctypes.c_float(wl.T),
                                               ctypes.c_void_p(soft.data_ptr()), ctypes.c_void_p(logZ.data_ptr()),
                                               ctypes.c_void_p(stream))
            assert rc == 0, binding.status_string(rc)
            torch.cuda.synchronize()
            assert parity.rel_inf(soft.cpu().numpy(), ref_soft.cpu().numpy()) <= parity.SOFT_TOL
            np.testing.assert_allclose(logZ.cpu().numpy(), ref_logZ.cpu().numpy(), rtol=1e-5, atol=1e-3)
            # and against the float64 oracle, which shares nothing with either CUDA entry point
            ref = oracle.soft_quantize(Wd.cpu().numpy(), cd.cpu().numpy(), wl.Lb, wl.k, wl.T)
            assert parity.rel_inf(soft.cpu().numpy(), ref["soft"]) <= parity.SOFT_TOL
            np.testing.assert_allclose(logZ.cpu().numpy(), ref["logZ"], rtol=1e-5, atol=1e-3)
        # the same inputs again, straight after a different problem has used the scratch
        wl = synth.tiny()
        Wd, cd = _device_inputs(wl, 64)
        a, _ = binding.bcjr_soft_quantize_static(Wd, cd, wl.Lb, wl.k, wl.n, wl.T)
        b, _ = binding.bcjr_soft_quantize_static(Wd, cd, wl.Lb, wl.k, wl.n, wl.T)
        torch.cuda.synchronize()
        assert torch.equal(a, b)
        ref, _ = ctx.bcjr_soft_quantize(Wd, cd, wl.Lb, wl.k, wl.n, wl.T)
        ctx.sync_status()
        assert parity.rel_inf(a.cpu().numpy(), ref.cpu().numpy()) <= parity.SOFT_TOL
    finally:
        ctx.close()


def test_static_entry_point_largest_trellis_one_resident_block_and_no_allocation():
    # Lb = 16, k = 2, n = 256: one block's history is 16 MiB, so the 32 MiB scratch holds exactly one
    # thread block, which must work through all three weight blocks reusing the same history slot.
    # The regular call runs a different (tensor-memory) kernel here, so this also compares two
    # implementations; the oracle decides.  With caller-supplied outputs the second call must leave
    # the device's free memory untouched.
    import torch
    from paper_2605_10655_b200 import Context, binding
    wl = synth.q_proj()
    nblk = 3
    Wd, cd = _device_inputs(wl, nblk)
    soft = torch.full_like(Wd, float("nan"))
    logZ = torch.full((nblk,), float("nan"), device=Wd.device)
    binding.bcjr_soft_quantize_static(Wd, cd, wl.Lb, wl.k, wl.n, wl.T, soft=soft, logZ=logZ)
    torch.cuda.synchronize()
    first = soft.clone()
    free0, _ = torch.cuda.mem_get_info()
    binding.bcjr_soft_quantize_static(Wd, cd, wl.Lb, wl.k, wl.n, wl.T, soft=soft, logZ=logZ)
    torch.cuda.synchronize()
    free1, _ = torch.cuda.mem_get_info()
    assert free1 == free0, "the static entry point changed the device's free memory"
    assert torch.equal(first, soft)
    ref = oracle.soft_quantize(Wd.cpu().numpy(), cd.cpu().numpy(), wl.Lb, wl.k, wl.T)
    assert parity.rel_inf(soft.cpu().numpy(), ref["soft"]) <= parity.SOFT_TOL
    np.testing.assert_allclose(logZ.cpu().numpy(), ref["logZ"], rtol=1e-5, atol=1e-3)
    ctx = Context(0)
    try:
        reg, _ = ctx.bcjr_soft_quantize(Wd, cd, wl.Lb, wl.k, wl.n, wl.T)
        assert ctx.sync_status().last_path == 1
        assert parity.rel_inf(soft.cpu().numpy(), reg.cpu().numpy()) <= parity.SOFT_TOL
    finally:
        ctx.close()


def test_static_entry_point_refuses_what_does_not_fit():
    import torch
    from paper_2605_10655_b200 import binding
    lib = binding.load_library()
    assert lib.bcjr_static_scratch_bytes() == 32 << 20
    dev = torch.device("cuda", 0)
    # one block of 2^16 states and 1024 steps needs 64 MiB of history: more than the fixed scratch
    W = torch.zeros((1, 1024), device=dev); c = torch.zeros(1 << 16, device=dev)
    with pytest.raises(binding.BcjrError) as ei:
        binding.bcjr_soft_quantize_static(W, c, 16, 2, 1024, 0.5)
    assert ei.value.code == -8
    with pytest.raises(binding.BcjrError) as ei:
        binding.bcjr_soft_quantize_static(W, c, 16, 2, 1024, -1.0)
    assert ei.value.code == -1

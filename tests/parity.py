"""Helpers of the GPU parity tests: run the CUDA path through the C ABI, run the oracle on the
same seeded inputs, and compare with the stated tolerances.

Tolerances (fp32 results against the float64 oracle):
  soft codeword   max |x - r| / max |r|  <= 1e-4
  gradients       max |x - r| / max |r|  <= 1e-3
  log Z           |x - r| <= 1e-5 |r| + 1e-3
  Viterbi         states, path bits and hard codeword bit-exact
"""
import numpy as np

SOFT_TOL = 1e-4
GRAD_TOL = 1e-3


def rel_inf(x, r):
    x = np.asarray(x, dtype=np.float64); r = np.asarray(r, dtype=np.float64)
    den = np.abs(r).max()
    return float(np.abs(x - r).max() / (den if den > 0 else 1.0))


def gpu_forward_backward(ctx, W, c, g, Lb, k, T):
    import torch
    dev = torch.device("cuda", ctx.device)
    n = W.shape[1]
    Wd = torch.from_numpy(np.ascontiguousarray(W)).to(dev)
    cd = torch.from_numpy(np.ascontiguousarray(c)).to(dev)
    soft, logZ = ctx.bcjr_soft_quantize(Wd, cd, Lb, k, n, T)
    out = {}
    if g is not None:
        gd = torch.from_numpy(np.ascontiguousarray(g)).to(dev)
        gW, gc = ctx.bcjr_backward(gd)
        out["grad_W"] = gW.cpu().numpy(); out["grad_codebook"] = gc.cpu().numpy()
    diag = ctx.sync_status()
    out["soft"] = soft.cpu().numpy(); out["logZ"] = logZ.cpu().numpy(); out["diag"] = diag
    return out


def gpu_viterbi(ctx, W, c, Lb, k):
    import torch
    dev = torch.device("cuda", ctx.device)
    n = W.shape[1]
    Wd = torch.from_numpy(np.ascontiguousarray(W)).to(dev)
    cd = torch.from_numpy(np.ascontiguousarray(c)).to(dev)
    bits, states, hard = ctx.viterbi_hard(Wd, cd, Lb, k, n)
    ctx.sync_status()
    return {"path_bits": bits.cpu().numpy(), "states": states.cpu().numpy().view(np.uint16),
            "hard": hard.cpu().numpy()}


def assert_forward_backward(got, ref_f, ref_b=None, what=""):
    e = rel_inf(got["soft"], ref_f["soft"])
    assert e <= SOFT_TOL, f"{what}: soft codeword rel err {e:.3e}"
    lz = np.abs(got["logZ"] - ref_f["logZ"])
    assert np.all(lz <= 1e-5 * np.abs(ref_f["logZ"]) + 1e-3), f"{what}: logZ err {lz.max():.3e}"
    if ref_b is not None:
        e = rel_inf(got["grad_W"], ref_b["grad_W"])
        assert e <= GRAD_TOL, f"{what}: grad_W rel err {e:.3e}"
        e = rel_inf(got["grad_codebook"], ref_b["grad_codebook"])
        assert e <= GRAD_TOL, f"{what}: grad_codebook rel err {e:.3e}"


def assert_viterbi(got, ref, what=""):
    np.testing.assert_array_equal(got["states"], ref["states"], err_msg=what + ": states")
    np.testing.assert_array_equal(got["path_bits"], ref["path_bits"], err_msg=what + ": path bits")
    np.testing.assert_array_equal(got["hard"].view(np.uint32), ref["hard"].view(np.uint32), err_msg=what + ": hard")

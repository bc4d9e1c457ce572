"""Thin ctypes binding of the C ABI in include/bcjr_b200.h.

Argument marshalling only: every step of the method runs in the CUDA kernels behind the
shared library.  torch is used for device memory and streams.  There is no CPU fallback:
a missing library raises at load time, a failing call raises BcjrError.
"""
from __future__ import annotations

import ctypes
from pathlib import Path

_PKG = Path(__file__).resolve().parent
LIB_PATH = _PKG / "libbcjr_b200.so"

EXPORTS = ["bcjr_create", "bcjr_destroy", "bcjr_set_option", "bcjr_soft_quantize", "bcjr_backward",
           "viterbi_hard", "bcjr_soft_quantize_vec", "viterbi_hard_vec", "bcjr_ste_forward", "bcjr_temperature", "bcjr_gaussian_codebook", "bcjr_adam_update",
           "bcjr_backward_adam", "bcjr_rht", "bcjr_group_scale", "bcjr_group_unscale", "bcjr_step_host", "bcjr_sync_status", "bcjr_block_defects", "bcjr_workspace_bytes",
           "bcjr_last_cuda_error", "bcjr_status_string", "bcjr_soft_quantize_static",
           "bcjr_static_scratch_bytes", "bcjr_measure_pipe_peaks"]


class BcjrError(RuntimeError):
    def __init__(self, code, where, detail=""):
        self.code = code
        super().__init__(f"{where}: {status_string(code)} ({code}){(' - ' + detail) if detail else ''}")


class PipePeaks(ctypes.Structure):
    """Mirror of bcjr_pipe_peaks (include/bcjr_microbench.h)."""
    _fields_ = [("num_sms", ctypes.c_int32), ("pad", ctypes.c_int32)] + [(n, ctypes.c_double) for n in (
        "sm_clock_mhz", "ex2_per_clk_sm", "lg2_per_clk_sm", "fma_f32_per_clk_sm",
        "fma_f32x2_per_clk_sm", "ex2_gops", "fma_f32x2_gops", "st_async_bytes_per_clk_sm", "cta_barrier_clk",
        "mbarrier_round_clk", "fma_f32x2_with_alu_per_clk_sm", "fma_f32x2_with_max_per_clk_sm",
        "fma_f32x2_with_ex2_per_clk_sm", "fma_f32x2_with_f64_per_clk_sm")]


class Diag(ctypes.Structure):
    _fields_ = [("device_status", ctypes.c_int32), ("max_posterior_defect", ctypes.c_float),
                ("max_logz_mismatch", ctypes.c_float), ("kernel_launches", ctypes.c_int32),
                ("last_path", ctypes.c_int32)]


_lib = None


def load_library() -> ctypes.CDLL:
    """Loads the in-tree CUDA library; raises if it has not been built."""
    global _lib
    if _lib is not None:
        return _lib
    if not LIB_PATH.exists():
        raise ImportError(f"{LIB_PATH} is missing: build it with `python -m paper_2605_10655_b200.build` "
                          "(there is no CPU fallback)")
    lib = ctypes.CDLL(str(LIB_PATH))
    vp, i, i64, f = ctypes.c_void_p, ctypes.c_int, ctypes.c_int64, ctypes.c_float
    lib.bcjr_create.restype = i; lib.bcjr_create.argtypes = [ctypes.POINTER(vp), i]
    lib.bcjr_destroy.restype = i; lib.bcjr_destroy.argtypes = [vp]
    lib.bcjr_set_option.restype = i; lib.bcjr_set_option.argtypes = [vp, ctypes.c_char_p, i64]
    lib.bcjr_soft_quantize.restype = i
    lib.bcjr_soft_quantize.argtypes = [vp, vp, vp, i, i, i, i64, f, vp, vp, vp]
    lib.bcjr_backward.restype = i; lib.bcjr_backward.argtypes = [vp, vp, vp, vp, vp]
    lib.viterbi_hard.restype = i; lib.viterbi_hard.argtypes = [vp, vp, vp, i, i, i, i64, vp, i64, vp, vp, vp]
    lib.bcjr_soft_quantize_vec.restype = i
    lib.bcjr_soft_quantize_vec.argtypes = [vp, vp, vp, i, i, i, i, i64, f, vp, vp, vp]
    lib.viterbi_hard_vec.restype = i
    lib.viterbi_hard_vec.argtypes = [vp, vp, vp, i, i, i, i, i64, vp, i64, vp, vp, vp]
    lib.bcjr_ste_forward.restype = i
    lib.bcjr_ste_forward.argtypes = [vp, vp, vp, i, i, i, i64, f, vp, vp, vp, vp]
    lib.bcjr_temperature.restype = ctypes.c_double
    lib.bcjr_temperature.argtypes = [ctypes.c_double, ctypes.c_double, i, i]
    lib.bcjr_gaussian_codebook.restype = i; lib.bcjr_gaussian_codebook.argtypes = [vp, i, vp, vp]
    lib.bcjr_adam_update.restype = i
    lib.bcjr_adam_update.argtypes = [vp, vp, vp, vp, vp, i64, i, f, f, f, f, vp]
    lib.bcjr_backward_adam.restype = i
    lib.bcjr_backward_adam.argtypes = [vp, vp, vp, vp, vp, vp, vp, vp, i, f, f, f, f, f, vp]
    lib.bcjr_rht.restype = i; lib.bcjr_rht.argtypes = [vp, vp, vp, i, i, vp, vp, i, vp]
    lib.bcjr_group_scale.restype = i; lib.bcjr_group_scale.argtypes = [vp, vp, vp, vp, i64, vp]
    lib.bcjr_group_unscale.restype = i; lib.bcjr_group_unscale.argtypes = [vp, vp, vp, vp, i64, vp]
    lib.bcjr_step_host.restype = i
    lib.bcjr_step_host.argtypes = [vp, vp, vp, vp, i, i, i, i64, f, vp, vp, vp, vp]
    lib.bcjr_sync_status.restype = i; lib.bcjr_sync_status.argtypes = [vp, vp, ctypes.POINTER(Diag)]
    lib.bcjr_block_defects.restype = i; lib.bcjr_block_defects.argtypes = [vp, vp, i64, vp]
    lib.bcjr_workspace_bytes.restype = i64; lib.bcjr_workspace_bytes.argtypes = [vp]
    lib.bcjr_last_cuda_error.restype = ctypes.c_char_p; lib.bcjr_last_cuda_error.argtypes = [vp]
    lib.bcjr_status_string.restype = ctypes.c_char_p; lib.bcjr_status_string.argtypes = [i]
    lib.bcjr_soft_quantize_static.restype = i
    lib.bcjr_soft_quantize_static.argtypes = [vp, vp, i, i, i, i64, f, vp, vp, vp]
    lib.bcjr_static_scratch_bytes.restype = i64; lib.bcjr_static_scratch_bytes.argtypes = []
    lib.bcjr_measure_pipe_peaks.restype = i; lib.bcjr_measure_pipe_peaks.argtypes = [i, ctypes.POINTER(PipePeaks), vp]
    _lib = lib
    return lib


def measure_pipe_peaks(device: int = 0, stream=None) -> dict:
    """Measured special-function, FP32 and cluster-exchange rates of the device (see include/bcjr_microbench.h)."""
    pk = PipePeaks()
    rc = load_library().bcjr_measure_pipe_peaks(int(device), ctypes.byref(pk), _stream_ptr(stream))
    if rc != 0:
        raise BcjrError(rc, "bcjr_measure_pipe_peaks")
    return {name: getattr(pk, name) for name, _ in PipePeaks._fields_ if name != "pad"}


def temperature(T0: float, T_end: float, t: int, n_steps: int) -> float:
    """Annealing schedule of Section 3.6 (library routine)."""
    return float(load_library().bcjr_temperature(T0, T_end, t, n_steps))


def status_string(code: int) -> str:
    return load_library().bcjr_status_string(int(code)).decode()


def path_bytes(Lb: int, k: int, n: int) -> int:
    return (Lb + k * (n - 1) + 7) // 8


def _stream_ptr(stream):
    import torch
    s = stream if stream is not None else torch.cuda.current_stream()
    return ctypes.c_void_p(s.cuda_stream)


def _dev(t, dtype, numel=None, name="tensor"):
    import torch
    if t is None:
        return None
    if not (isinstance(t, torch.Tensor) and t.is_cuda and t.is_contiguous() and t.dtype == dtype):
        raise TypeError(f"{name}: expected a contiguous CUDA tensor of dtype {dtype}")
    if numel is not None and t.numel() != numel:
        raise ValueError(f"{name}: expected {numel} elements, got {t.numel()}")
    return ctypes.c_void_p(t.data_ptr())


def bcjr_soft_quantize_static(W, codebook, Lb, k, n, T, soft=None, logZ=None, stream=None):
    """Forward call for callers that may not allocate device memory: no context, no cudaMalloc;
    the scratch is a fixed array inside the library (see include/bcjr_b200.h for the limits).
    The output tensors are the caller's: pass `soft` / `logZ` to avoid torch allocating them here.
    All calls on a device share that scratch, so keep them ordered on one stream."""
    import torch
    lib = load_library()
    B = W.numel() // n
    if B * n != W.numel():
        raise ValueError("W.numel() must be a multiple of n")
    if soft is None:
        soft = torch.empty_like(W)
    if logZ is None:
        logZ = torch.empty(B, dtype=torch.float32, device=W.device)
    with torch.cuda.device(W.device):
        rc = lib.bcjr_soft_quantize_static(_dev(W, torch.float32, name="W"),
                                           _dev(codebook, torch.float32, 1 << Lb, "codebook"), Lb, k, n, B,
                                           float(T), _dev(soft, torch.float32, B * n, "soft"),
                                           _dev(logZ, torch.float32, B, "logZ"), _stream_ptr(stream))
    if rc != 0:
        raise BcjrError(rc, "bcjr_soft_quantize_static")
    return soft, logZ


class Context:
    """Owns one bcjr_ctx (scratch memory + the state saved between forward and backward)."""

    def __init__(self, device: int = 0):
        self._lib = load_library()
        self._h = ctypes.c_void_p()
        rc = self._lib.bcjr_create(ctypes.byref(self._h), int(device))
        if rc != 0:
            raise BcjrError(rc, "bcjr_create")
        self.device = int(device)
        self._saved = None

    def close(self):
        if getattr(self, "_h", None) is not None and self._h:
            self._lib.bcjr_destroy(self._h)
            self._h = None

    def __del__(self):
        try:
            self.close()
        except Exception:
            pass

    def _check(self, rc, where):
        if rc != 0:
            raise BcjrError(rc, where, self._lib.bcjr_last_cuda_error(self._h).decode())

    def set_option(self, name: str, value: int):
        self._check(self._lib.bcjr_set_option(self._h, name.encode(), int(value)), "bcjr_set_option")

    def bcjr_soft_quantize(self, W, codebook, Lb, k, n, T, soft=None, logZ=None, stream=None):
        """W: [num_blocks*n] (any shape with that many elements) float32 CUDA.  Returns (soft, logZ).
        codebook=None selects the computed Gaussian emission of Section 3.1 (no table)."""
        import torch
        B = W.numel() // n
        if B * n != W.numel():
            raise ValueError("W.numel() must be a multiple of n")
        if soft is None:
            soft = torch.empty_like(W)
        if logZ is None:
            logZ = torch.empty(B, dtype=torch.float32, device=W.device)
        rc = self._lib.bcjr_soft_quantize(self._h, _dev(W, torch.float32, name="W"),
                                          _dev(codebook, torch.float32, 1 << Lb, "codebook"), Lb, k, n, B,
                                          float(T), _dev(soft, torch.float32, B * n, "soft"),
                                          _dev(logZ, torch.float32, B, "logZ"), _stream_ptr(stream))
        self._check(rc, "bcjr_soft_quantize")
        self._saved = (W, codebook, Lb, B * n)       # keep the borrowed tensors alive
        return soft, logZ

    def bcjr_backward(self, grad_soft, grad_W=None, grad_codebook=None, stream=None, want_grad_codebook=True):
        """Returns (grad_W, grad_codebook); with want_grad_codebook=False the table's gradient is not formed
        (NULL is passed; the second value is None)."""
        import torch
        if self._saved is None:
            raise BcjrError(-4, "bcjr_backward")
        W, codebook, Lb, numel = self._saved
        if grad_W is None:
            grad_W = torch.empty_like(W)
        if codebook is None:                          # computed emission: there is no table to differentiate
            want_grad_codebook = False
        if grad_codebook is None and want_grad_codebook:
            grad_codebook = torch.empty(codebook.numel(), dtype=torch.float32, device=W.device)
        rc = self._lib.bcjr_backward(self._h, _dev(grad_soft, torch.float32, numel, "grad_soft"),
                                     _dev(grad_W, torch.float32, numel, "grad_W"),
                                     _dev(grad_codebook, torch.float32, name="grad_codebook")
                                     if grad_codebook is not None else None,
                                     _stream_ptr(stream))
        self._check(rc, "bcjr_backward")
        return grad_W, grad_codebook

    def viterbi_hard(self, W, codebook, Lb, k, n, want_states=True, want_hard=True, stream=None):
        """Returns (path_bits [B, nbytes] uint8, states [B, n] int16-as-uint16 bits or None, hard [B, n] or None)."""
        import torch
        B = W.numel() // n
        nb = path_bytes(Lb, k, n)
        bits = torch.empty((B, nb), dtype=torch.uint8, device=W.device)
        states = torch.empty((B, n), dtype=torch.int16, device=W.device) if want_states else None
        hard = torch.empty((B, n), dtype=torch.float32, device=W.device) if want_hard else None
        rc = self._lib.viterbi_hard(self._h, _dev(W, torch.float32, name="W"),
                                    _dev(codebook, torch.float32, 1 << Lb, "codebook"), Lb, k, n, B,
                                    ctypes.c_void_p(bits.data_ptr()), nb,
                                    ctypes.c_void_p(states.data_ptr()) if want_states else None,
                                    ctypes.c_void_p(hard.data_ptr()) if want_hard else None, _stream_ptr(stream))
        self._check(rc, "viterbi_hard")
        return bits, states, hard

    def bcjr_soft_quantize_vec(self, W, codebook, Lb, k, V, n, T, soft=None, logZ=None, stream=None):
        """Vector emissions: codebook [2^Lb, V], a step consumes V weights.  Returns (soft, logZ)."""
        import torch
        B = W.numel() // n
        if B * n != W.numel():
            raise ValueError("W.numel() must be a multiple of n")
        if soft is None:
            soft = torch.empty_like(W)
        if logZ is None:
            logZ = torch.empty(B, dtype=torch.float32, device=W.device)
        rc = self._lib.bcjr_soft_quantize_vec(self._h, _dev(W, torch.float32, name="W"),
                                              _dev(codebook, torch.float32, (1 << Lb) * V, "codebook"), Lb, k, V, n, B,
                                              float(T), _dev(soft, torch.float32, B * n, "soft"),
                                              _dev(logZ, torch.float32, B, "logZ"), _stream_ptr(stream))
        self._check(rc, "bcjr_soft_quantize_vec")
        self._saved = (W, codebook, Lb, B * n)
        return soft, logZ

    def viterbi_hard_vec(self, W, codebook, Lb, k, V, n, want_states=True, want_hard=True, stream=None):
        """Returns (path_bits [B, nbytes], states [B, n/V] or None, hard [B, n] or None)."""
        import torch
        B = W.numel() // n
        nb = path_bytes(Lb, k * V, n // V)
        bits = torch.empty((B, nb), dtype=torch.uint8, device=W.device)
        states = torch.empty((B, n // V), dtype=torch.int16, device=W.device) if want_states else None
        hard = torch.empty((B, n), dtype=torch.float32, device=W.device) if want_hard else None
        rc = self._lib.viterbi_hard_vec(self._h, _dev(W, torch.float32, name="W"),
                                        _dev(codebook, torch.float32, (1 << Lb) * V, "codebook"), Lb, k, V, n, B,
                                        ctypes.c_void_p(bits.data_ptr()), nb,
                                        ctypes.c_void_p(states.data_ptr()) if want_states else None,
                                        ctypes.c_void_p(hard.data_ptr()) if want_hard else None, _stream_ptr(stream))
        self._check(rc, "viterbi_hard_vec")
        return bits, states, hard

    def bcjr_ste_forward(self, W, codebook, Lb, k, n, T, want_states=False, want_soft=False, stream=None):
        """Hard Viterbi codeword forward, finite-T state saved for bcjr_backward.  Returns (hard, states, soft)."""
        import torch
        B = W.numel() // n
        if B * n != W.numel():
            raise ValueError("W.numel() must be a multiple of n")
        hard = torch.empty((B, n), dtype=torch.float32, device=W.device)
        states = torch.empty((B, n), dtype=torch.int16, device=W.device) if want_states else None
        soft = torch.empty((B, n), dtype=torch.float32, device=W.device) if want_soft else None
        rc = self._lib.bcjr_ste_forward(self._h, _dev(W, torch.float32, name="W"),
                                        _dev(codebook, torch.float32, 1 << Lb, "codebook"), Lb, k, n, B, float(T),
                                        ctypes.c_void_p(hard.data_ptr()),
                                        ctypes.c_void_p(states.data_ptr()) if want_states else None,
                                        ctypes.c_void_p(soft.data_ptr()) if want_soft else None, _stream_ptr(stream))
        self._check(rc, "bcjr_ste_forward")
        self._saved = (W, codebook, Lb, B * n)
        return hard, states, soft

    def bcjr_gaussian_codebook(self, Lb, device=None, stream=None):
        """Table of the computed Gaussian emission c(s) = Phi^-1((s + 1/2) / 2^Lb)."""
        import torch
        out = torch.empty(1 << Lb, dtype=torch.float32, device=torch.device("cuda", self.device) if device is None else device)
        self._check(self._lib.bcjr_gaussian_codebook(self._h, Lb, ctypes.c_void_p(out.data_ptr()), _stream_ptr(stream)),
                    "bcjr_gaussian_codebook")
        return out

    def bcjr_adam_update(self, param, grad, m, v, t, lr, beta1=0.9, beta2=0.999, eps=1e-8, stream=None):
        """One Adam step on `param` in place (m, v: moment buffers of the same size)."""
        import torch
        n = param.numel()
        rc = self._lib.bcjr_adam_update(self._h, _dev(param, torch.float32, n, "param"), _dev(grad, torch.float32, n, "grad"),
                                        _dev(m, torch.float32, n, "m"), _dev(v, torch.float32, n, "v"), n, int(t),
                                        float(lr), float(beta1), float(beta2), float(eps), _stream_ptr(stream))
        self._check(rc, "bcjr_adam_update")

    def bcjr_backward_adam(self, grad_soft, m_W, v_W, t, lr_W, m_c=None, v_c=None, lr_c=0.0,
                           beta1=0.9, beta2=0.999, eps=1e-8, stream=None):
        """Backward pass + Adam on the W (and, with m_c/v_c, the codebook) of the last forward call, in place."""
        import torch
        if self._saved is None:
            raise BcjrError(-4, "bcjr_backward_adam")
        W, codebook, Lb, numel = self._saved
        upd_c = m_c is not None
        rc = self._lib.bcjr_backward_adam(
            self._h, _dev(grad_soft, torch.float32, numel, "grad_soft"), _dev(W, torch.float32, numel, "W"),
            _dev(m_W, torch.float32, numel, "m_W"), _dev(v_W, torch.float32, numel, "v_W"),
            _dev(codebook, torch.float32, codebook.numel(), "codebook") if upd_c else None,
            _dev(m_c, torch.float32, codebook.numel(), "m_c") if upd_c else None,
            _dev(v_c, torch.float32, codebook.numel(), "v_c") if upd_c else None,
            int(t), float(lr_W), float(lr_c), float(beta1), float(beta2), float(eps), _stream_ptr(stream))
        self._check(rc, "bcjr_backward_adam")
        self._saved = None

    def bcjr_rht(self, W, sign_rows, sign_cols, inverse=False, out=None, stream=None):
        """Random-sign Hadamard rotation on both sides of W [m, n] (or its inverse); returns `out`."""
        import torch
        m, n = W.shape
        if out is None:
            out = torch.empty_like(W)
        rc = self._lib.bcjr_rht(self._h, _dev(W, torch.float32, m * n, "W"), _dev(out, torch.float32, m * n, "out"), m, n,
                                _dev(sign_rows, torch.float32, m, "sign_rows"), _dev(sign_cols, torch.float32, n, "sign_cols"),
                                1 if inverse else 0, _stream_ptr(stream))
        self._check(rc, "bcjr_rht")
        return out

    def bcjr_group_scale(self, W, stream=None):
        """Per-16 scales (root mean square) of W; returns (scales [numel/16], W / scales)."""
        import torch
        numel = W.numel()
        scales = torch.empty(numel // 16, dtype=torch.float32, device=W.device)
        out = torch.empty_like(W)
        rc = self._lib.bcjr_group_scale(self._h, _dev(W, torch.float32, numel, "W"), ctypes.c_void_p(scales.data_ptr()),
                                        _dev(out, torch.float32, numel, "W_scaled"), numel, _stream_ptr(stream))
        self._check(rc, "bcjr_group_scale")
        return scales, out

    def bcjr_group_unscale(self, W_scaled, scales, stream=None):
        import torch
        numel = W_scaled.numel()
        out = torch.empty_like(W_scaled)
        rc = self._lib.bcjr_group_unscale(self._h, _dev(W_scaled, torch.float32, numel, "W_scaled"),
                                          _dev(scales, torch.float32, numel // 16, "scales"),
                                          _dev(out, torch.float32, numel, "W"), numel, _stream_ptr(stream))
        self._check(rc, "bcjr_group_unscale")
        return out

    def bcjr_step_host(self, W, codebook, grad_soft, Lb, k, n, T, soft=None, grad_W=None, grad_codebook=None,
                       stream=None):
        """Host (CPU, ideally pinned) float32 tensors in, host tensors out; synchronous."""
        import torch

        def hp(t, name):
            if t is None:
                return None
            if t.is_cuda or not t.is_contiguous() or t.dtype != torch.float32:
                raise TypeError(f"{name}: expected a contiguous float32 CPU tensor")
            return ctypes.c_void_p(t.data_ptr())
        B = W.numel() // n
        rc = self._lib.bcjr_step_host(self._h, hp(W, "W"), hp(codebook, "codebook"), hp(grad_soft, "grad_soft"),
                                      Lb, k, n, B, float(T), hp(soft, "soft"), hp(grad_W, "grad_W"),
                                      hp(grad_codebook, "grad_codebook"), _stream_ptr(stream))
        self._check(rc, "bcjr_step_host")
        self._saved = None

    def sync_status(self, stream=None, check=True) -> Diag:
        d = Diag()
        rc = self._lib.bcjr_sync_status(self._h, _stream_ptr(stream), ctypes.byref(d))
        if check:
            self._check(rc, "bcjr_sync_status")
        return d

    def block_defects(self, count: int, stream=None):
        """Per-block posterior defect of the last forward call made with option record_block_defect = 1
        (numpy float32 array of `count` values)."""
        import numpy as np
        out = np.empty(int(count), dtype=np.float32)
        rc = self._lib.bcjr_block_defects(self._h, out.ctypes.data_as(ctypes.c_void_p), int(count), _stream_ptr(stream))
        self._check(rc, "bcjr_block_defects")
        return out

    def workspace_bytes(self) -> int:
        return int(self._lib.bcjr_workspace_bytes(self._h))

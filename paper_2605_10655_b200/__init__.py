"""B200-native BCJR soft quantisation (forward-backward over a bitshift trellis), its backward
pass and the Viterbi hard code, behind the C ABI of include/bcjr_b200.h.

    from paper_2605_10655_b200 import Context
    ctx = Context(device=0)
    soft, logZ = ctx.bcjr_soft_quantize(W, codebook, Lb=16, k=2, n=256, T=0.1)
    grad_W, grad_codebook = ctx.bcjr_backward(grad_soft)
    path_bits, states, hard = ctx.viterbi_hard(W, codebook, Lb=16, k=2, n=256)

The CUDA library is loaded on first use; there is no CPU fallback.
"""
from .binding import (BcjrError, Context, Diag, bcjr_soft_quantize_static, load_library,  # noqa: F401
                      path_bytes, status_string)

"""CPU oracle for the steps on either side of the trellis pass in the paper's QAT loop.

TEST INFRASTRUCTURE ONLY (same rules as the trellis oracle): plain float64 numpy written from the
definitions, never imported by the CUDA package.

  temperature(T0, T_end, t, n_steps)   Section 3.6: T_t = T_0 (T_end / T_0)^(t / N_steps)
  gaussian_codebook(Lb)                Section 3.1: c(s) = Phi^-1((s + 1/2) / S), no permutation
  adam_update(...)                     the Adam rule Algorithm 1 applies to the continuous pre-image
                                       (Kingma & Ba 2015, Algorithm 1 there): with g the gradient at step t,
                                         m <- b1 m + (1 - b1) g,   v <- b2 v + (1 - b2) g^2,
                                         p <- p - lr * (m / (1 - b1^t)) / (sqrt(v / (1 - b2^t)) + eps)

  hadamard / rht_forward / rht_inverse / group_scales   the incoherence rotation and the per-16 scales
                                       that precede the trellis in the paper's pipeline (see below)

Pins (tests/test_qat_oracle_pins.py): end points and constant ratio of the schedule; Phi(c(s)) =
(s + 1/2)/S through an independent routine, antisymmetry, monotonicity; Adam's closed forms (first
step, constant gradient for any number of steps, zero gradient); the Hadamard matrix against scipy's
and H H = n I, the rotation's inverse, norm preservation, a spike spread flat, W x reproduced from the
rotated quantities; unit mean square of every scaled group.  Nothing here is unpinned.
"""
import numpy as np
from scipy.special import ndtri


def temperature(T0, T_end, t, n_steps):
    return float(T0) * (float(T_end) / float(T0)) ** (t / n_steps)


def gaussian_codebook(Lb):
    S = 1 << Lb
    return ndtri((np.arange(S, dtype=np.float64) + 0.5) / S)


def adam_update(p, g, m, v, t, lr, beta1=0.9, beta2=0.999, eps=1e-8):
    """Returns (p, m, v) after step t (1-based); inputs are not modified."""
    p = np.asarray(p, dtype=np.float64); g = np.asarray(g, dtype=np.float64)
    m = beta1 * np.asarray(m, dtype=np.float64) + (1.0 - beta1) * g
    v = beta2 * np.asarray(v, dtype=np.float64) + (1.0 - beta2) * g * g
    mhat = m / (1.0 - beta1 ** t)
    vhat = v / (1.0 - beta2 ** t)
    return p - lr * mhat / (np.sqrt(vhat) + eps), m, v


# ---- incoherence processing (Section 3.1 / Section 4 "Quantization configuration"): a random-sign
# Hadamard rotation on both sides of the weight matrix, and a scale per group of 16 elements.
# The paper names both and gives no formula; the forms fixed here are the
# QuIP#-style ones:  W~ = H_m diag(sL) W diag(sR) H_n / sqrt(m n)  with the Sylvester-ordered
# Walsh-Hadamard matrices H (entries +-1, H H = size * I), so that the inverse is
# W = diag(sL) H_m W~ H_n diag(sR) / sqrt(m n);  scale of a group = root mean square of its 16 elements.
def hadamard(n):
    """Sylvester construction H_{2n} = [[H, H], [H, -H]] written out; n a power of two."""
    H = np.ones((1, 1))
    while H.shape[0] < n:
        H = np.block([[H, H], [H, -H]])
    assert H.shape[0] == n, "size must be a power of two"
    return H


def rht_forward(W, sL, sR):
    W = np.asarray(W, dtype=np.float64)
    m, n = W.shape
    return hadamard(m) @ (np.asarray(sL, dtype=np.float64)[:, None] * W * np.asarray(sR, dtype=np.float64)[None, :]) @ hadamard(n) / np.sqrt(m * n)


def rht_inverse(Wt, sL, sR):
    Wt = np.asarray(Wt, dtype=np.float64)
    m, n = Wt.shape
    return np.asarray(sL, dtype=np.float64)[:, None] * (hadamard(m) @ Wt @ hadamard(n)) * np.asarray(sR, dtype=np.float64)[None, :] / np.sqrt(m * n)


def group_scales(W, group=16):
    """Root mean square of every `group` consecutive elements of each row; returns (scales, W / scales)."""
    W = np.asarray(W, dtype=np.float64)
    m, n = W.shape
    g = W.reshape(m, n // group, group)
    s = np.sqrt((g * g).mean(axis=2))
    scaled = np.divide(g, s[:, :, None], out=np.zeros_like(g), where=s[:, :, None] > 0)      # an all-zero group stays zero
    return s, scaled.reshape(m, n)

"""CPU oracle for the steps on either side of the trellis pass in the paper's QAT loop.

TEST INFRASTRUCTURE ONLY (same rules as the trellis oracle): plain float64 numpy written from the
definitions, never imported by the CUDA package.

  temperature(T0, T_end, t, n_steps)   Section 3.6: T_t = T_0 (T_end / T_0)^(t / N_steps)
  gaussian_codebook(Lb)                Section 3.1: c(s) = Phi^-1((s + 1/2) / S), no permutation
  adam_update(...)                     the Adam rule Algorithm 1 applies to the continuous pre-image
                                       (Kingma & Ba 2015, Algorithm 1 there): with g the gradient at step t,
                                         m <- b1 m + (1 - b1) g,   v <- b2 v + (1 - b2) g^2,
                                         p <- p - lr * (m / (1 - b1^t)) / (sqrt(v / (1 - b2^t)) + eps)

Pins (tests/test_qat_oracle_pins.py): end points and constant ratio of the schedule; Phi(c(s)) =
(s + 1/2)/S through an independent routine, antisymmetry, monotonicity; Adam's closed forms (first
step, constant gradient for any number of steps, zero gradient).  Nothing here is unpinned.
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

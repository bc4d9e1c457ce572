"""Best path, runner-up margin and nearest-entry decoding in float64 numpy.

Used to state the cold-limit comparison (Section 3.3, identity 1: as T -> 0 the soft codeword
tends to the Viterbi hard code) precisely.  At any finite T the two differ wherever a second
path comes within a few T of the best one, so the comparison is made on the blocks whose
path-energy margin -- squared error of the best path that differs from the Viterbi path
somewhere, minus that of the Viterbi path -- exceeds a stated multiple of T.

Independent of the oracle's dynamic programmes: min-sum forward and backward tables over the
bitshift trellis (Section 3.1), written with array reshapes instead of predecessor tables.
For every step t and state s, F_t(s) + B_t(s) is the squared error of the best path through
(t, s); a path other than the best one leaves it at some step, so the runner-up's error is
the minimum of F_t(s) + B_t(s) over all (t, s) off the best path.
"""
import numpy as np


def best_and_margin(w, c, Lb, k):
    """Returns (states [n] of the best path, its squared error, margin to the best other path)."""
    w = np.asarray(w, dtype=np.float64); c = np.asarray(c, dtype=np.float64)
    n, S, K = len(w), 1 << Lb, 1 << k
    Q = S // K
    e = (w[:, None] - c[None, :]) ** 2                                   # [n, S]
    F = np.empty((n, S)); B = np.empty((n, S))
    F[0] = e[0]
    for t in range(1, n):
        # predecessors of s: (s >> k) + j*Q, j < K  ->  min over the leading axis of [K, Q], indexed by s >> k
        F[t] = e[t] + np.repeat(F[t - 1].reshape(K, Q).min(axis=0), K)
    B[n - 1] = 0.0
    for t in range(n - 2, -1, -1):
        # successors of s: ((s << k) | b) mod S, b < K  ->  min over the trailing axis of [Q, K], indexed by s mod Q
        B[t] = np.tile((e[t + 1] + B[t + 1]).reshape(Q, K).min(axis=1), K)
    through = F + B
    total = through[0].min()
    states = through.argmin(axis=1)                                      # lowest state on ties, like the oracle
    masked = through.copy()
    masked[np.arange(n), states] = np.inf
    return states, float(total), float(masked.min() - total)


def decode_nearest(values, c):
    """Nearest table entry (by value) to each element of `values`; returns the entry values."""
    c = np.asarray(c, dtype=np.float64)
    order = np.sort(c)
    v = np.asarray(values, dtype=np.float64)
    i = np.clip(np.searchsorted(order, v), 1, len(order) - 1)
    lo, hi = order[i - 1], order[i]
    return np.where(v - lo <= hi - v, lo, hi)

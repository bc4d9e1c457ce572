"""Exhaustive enumeration of every legal trellis path: the definition of last resort.

Independent of the oracle's dynamic programmes: it lists all S * K^(n-1) paths of the
bitshift trellis (Section 3.1), weighs each with the Boltzmann factor of Eq. 4 and
takes expectations directly (Eq. 3).  Only usable on tiny trellises.
"""
import itertools

import numpy as np


def enumerate_paths(Lb, k, n):
    """All legal state sequences as an int array [num_paths, n]."""
    S, K = 1 << Lb, 1 << k
    first = np.arange(S, dtype=np.int64)
    paths = first[:, None]
    for _ in range(n - 1):
        last = paths[:, -1]
        nxt = ((last[:, None] << k) | np.arange(K)[None, :]) & (S - 1)     # [P, K]
        paths = np.concatenate([np.repeat(paths, K, axis=0), nxt.reshape(-1, 1)], axis=1)
    return paths


def path_energy(paths, w, c):
    """sum_t 1/2 (w_t - c[s_t])^2 per path (Eq. 4's exponent times T)."""
    return 0.5 * ((w[None, :] - c[paths]) ** 2).sum(axis=1)


def soft_codeword(w, c, Lb, k, T, paths=None):
    """Returns (soft [n], logZ, gamma [n,S]) by direct summation over paths."""
    w = np.asarray(w, dtype=np.float64); c = np.asarray(c, dtype=np.float64)
    n = len(w)
    if paths is None:
        paths = enumerate_paths(Lb, k, n)
    E = path_energy(paths, w, c)
    m = (-E / T).max()
    p = np.exp(-E / T - m)
    Z = p.sum()
    p = p / Z
    soft = (p[:, None] * c[paths]).sum(axis=0)
    gamma = np.zeros((n, 1 << Lb))
    for t in range(n):
        np.add.at(gamma[t], paths[:, t], p)
    return soft, m + np.log(Z), gamma


def loss(w, c, g, Lb, k, T, paths=None):
    soft, _, _ = soft_codeword(w, c, Lb, k, T, paths)
    return float(np.dot(g, soft))


def fd_gradients(w, c, g, Lb, k, T, h=1e-6):
    """Central finite differences of loss() w.r.t. every weight and every table entry."""
    w = np.asarray(w, dtype=np.float64).copy(); c = np.asarray(c, dtype=np.float64).copy()
    paths = enumerate_paths(Lb, k, len(w))
    gw = np.zeros_like(w); gc = np.zeros_like(c)
    for i in range(len(w)):
        wp = w.copy(); wp[i] += h; wm = w.copy(); wm[i] -= h
        gw[i] = (loss(wp, c, g, Lb, k, T, paths) - loss(wm, c, g, Lb, k, T, paths)) / (2 * h)
    for u in range(len(c)):
        cp = c.copy(); cp[u] += h; cm = c.copy(); cm[u] -= h
        gc[u] = (loss(w, cp, g, Lb, k, T, paths) - loss(w, cm, g, Lb, k, T, paths)) / (2 * h)
    return gw, gc


def best_path(w, c, Lb, k):
    """Exhaustive argmin of sum_t (w_t - c[s_t])^2; returns (states [n], cost, gap to runner-up)."""
    w = np.asarray(w, dtype=np.float64); c = np.asarray(c, dtype=np.float64)
    paths = enumerate_paths(Lb, k, len(w))
    cost = ((w[None, :] - c[paths]) ** 2).sum(axis=1)
    order = np.argsort(cost, kind="stable")
    return paths[order[0]], cost[order[0]], cost[order[1]] - cost[order[0]]


def pack_path_bits(states, Lb, k):
    """Reference packing: s_1 in Lb bits then k new bits per step, MSB first."""
    bits = [(int(states[0]) >> i) & 1 for i in range(Lb - 1, -1, -1)]
    for s in states[1:]:
        bits += [(int(s) >> i) & 1 for i in range(k - 1, -1, -1)]
    out = np.zeros((len(bits) + 7) // 8, dtype=np.uint8)
    for i, b in enumerate(bits):
        if b:
            out[i >> 3] |= 1 << (7 - (i & 7))
    return out


# ---------------------------------------------------------------- vector emissions (V numbers per step)
def vec_soft_codeword(w, c, Lb, kb, V, T, paths=None):
    """w: [n], c: [S, V]; a step consumes V weights and kb bits.  Returns (soft [n], logZ)."""
    w = np.asarray(w, dtype=np.float64).reshape(-1, V); c = np.asarray(c, dtype=np.float64)
    nt = w.shape[0]
    if paths is None:
        paths = enumerate_paths(Lb, kb, nt)
    emitted = c[paths]                                        # [P, nt, V]
    E = 0.5 * ((w[None] - emitted) ** 2).sum(axis=(1, 2))
    m = (-E / T).max()
    p = np.exp(-E / T - m)
    Z = p.sum()
    soft = (p[:, None, None] * emitted).sum(axis=0) / Z
    return soft.reshape(-1), m + np.log(Z)


def vec_fd_gradients(w, c, g, Lb, kb, V, T, h=1e-6):
    w = np.asarray(w, dtype=np.float64).copy(); c = np.asarray(c, dtype=np.float64).copy()
    g = np.asarray(g, dtype=np.float64)
    paths = enumerate_paths(Lb, kb, len(w) // V)
    f = lambda ww, cc: float(np.dot(g, vec_soft_codeword(ww, cc, Lb, kb, V, T, paths)[0]))
    gw = np.zeros_like(w); gc = np.zeros_like(c)
    for i in range(len(w)):
        wp = w.copy(); wp[i] += h; wm = w.copy(); wm[i] -= h
        gw[i] = (f(wp, c) - f(wm, c)) / (2 * h)
    for u in range(c.shape[0]):
        for v in range(V):
            cp = c.copy(); cp[u, v] += h; cm = c.copy(); cm[u, v] -= h
            gc[u, v] = (f(w, cp) - f(w, cm)) / (2 * h)
    return gw, gc


def vec_best_path(w, c, Lb, kb, V):
    w = np.asarray(w, dtype=np.float64).reshape(-1, V); c = np.asarray(c, dtype=np.float64)
    paths = enumerate_paths(Lb, kb, w.shape[0])
    cost = ((w[None] - c[paths]) ** 2).sum(axis=(1, 2))
    order = np.argsort(cost, kind="stable")
    return paths[order[0]], cost[order[0]], cost[order[1]] - cost[order[0]]

"""Pins for the float64 CPU oracle (no GPU needed).

The paper prints no numeric worked example of a soft codeword, a gradient or a path, so
the oracle is pinned to what the mathematics fixes:
  P1  exhaustive enumeration of every legal path (Eq. 3-4 taken literally),
  P2  central finite differences of the enumerated loss, and the shift identity,
  P3  marginals sum to one, log Z is the same at every t (Eq. 6, "any t"),
  P4  an independent Viterbi (exhaustive argmin; a second, "push"-style DP), the
      T -> 0 limit of the soft codeword, idempotence of the hard code,
  P5  special cases that reduce to library routines (scipy softmax / logsumexp,
      dense transfer-matrix products).
"""
import numpy as np
import pytest
from scipy.special import logsumexp, softmax

import bruteforce as bf
import oracle

TINY = [(6, 4, 2), (5, 3, 1), (4, 5, 3), (4, 2, 2), (4, 3, 2), (3, 4, 4), (5, 4, 1)]  # (n, Lb, k)


def _inputs(n, Lb, seed, B=1):
    rng = np.random.default_rng(seed)
    c = rng.standard_normal(1 << Lb).astype(np.float32)
    W = rng.standard_normal((B, n)).astype(np.float32)
    g = rng.standard_normal((B, n)).astype(np.float32)
    return W, c, g


# ---------------------------------------------------------------- P1: every path enumerated
@pytest.mark.parametrize("n,Lb,k", TINY)
@pytest.mark.parametrize("T", [1.0, 0.5, 0.05])
def test_soft_codeword_matches_enumeration(n, Lb, k, T):
    W, c, _ = _inputs(n, Lb, seed=100 + n + Lb + k, B=3)
    out = oracle.soft_quantize(W, c, Lb, k, T, want_gamma_of=1)
    for b in range(3):
        soft, logZ, gamma = bf.soft_codeword(W[b], c, Lb, k, T)
        np.testing.assert_allclose(out["soft"][b], soft, rtol=0, atol=1e-12)
        np.testing.assert_allclose(out["logZ"][b], logZ, rtol=0, atol=1e-11)
        if b == 1:
            np.testing.assert_allclose(out["gamma"], gamma, rtol=0, atol=1e-13)


def test_path_count_and_legality():
    paths = bf.enumerate_paths(4, 2, 6)
    assert paths.shape == (16 * 4 ** 5, 6)              # 16384 paths
    assert len({tuple(p) for p in paths}) == len(paths)
    assert np.all((paths[:, 1:] >> 2) == (paths[:, :-1] & 3))   # new state keeps the old low bits


# ---------------------------------------------------------------- P2: gradients
@pytest.mark.parametrize("n,Lb,k", [(6, 4, 2), (5, 3, 1), (4, 5, 3), (4, 2, 2), (4, 3, 2)])
@pytest.mark.parametrize("T", [1.0, 0.3])
def test_gradients_match_finite_differences_of_enumeration(n, Lb, k, T):
    W, c, g = _inputs(n, Lb, seed=200 + n + Lb + k)
    out = oracle.backward(W, c, g, Lb, k, T)
    gw, gc = bf.fd_gradients(W[0], c, g[0].astype(np.float64), Lb, k, T, h=1e-6)
    np.testing.assert_allclose(out["grad_W"][0], gw, rtol=0, atol=5e-8)
    np.testing.assert_allclose(out["grad_codebook"], gc, rtol=0, atol=5e-8)


def test_grad_codebook_sums_over_blocks():
    n, Lb, k, T = 5, 4, 2, 0.4
    W, c, g = _inputs(n, Lb, seed=7, B=4)
    whole = oracle.backward(W, c, g, Lb, k, T)
    parts = [oracle.backward(W[i:i + 1], c, g[i:i + 1], Lb, k, T) for i in range(4)]
    np.testing.assert_allclose(whole["grad_codebook"], sum(p["grad_codebook"] for p in parts), atol=1e-13)
    np.testing.assert_allclose(whole["grad_W"], np.concatenate([p["grad_W"] for p in parts]), atol=1e-14)


@pytest.mark.parametrize("Lb,k,n,T", [(8, 2, 64, 0.5), (9, 3, 40, 0.1), (7, 1, 30, 0.05), (8, 4, 20, 0.2)])
def test_shift_identity(Lb, k, n, T):
    # soft(w + a, c + a) = soft(w, c) + a  =>  sum grad_W + sum grad_c = sum g
    W, c, g = _inputs(n, Lb, seed=300 + Lb, B=3)
    out = oracle.backward(W, c, g, Lb, k, T)
    total = out["grad_W"].sum() + out["grad_codebook"].sum()
    np.testing.assert_allclose(total, g.astype(np.float64).sum(), rtol=0, atol=1e-9)


def test_gradient_finite_differences_of_oracle_medium():
    # larger than enumeration allows: differentiate the oracle's own forward pass numerically
    Lb, k, n, T = 8, 2, 12, 0.2
    W, c, g = _inputs(n, Lb, seed=17)
    g64 = g.astype(np.float64)
    out = oracle.backward(W, c, g, Lb, k, T)
    W64 = W.astype(np.float64); c64 = c.astype(np.float64)
    h = 1e-6
    for i in [0, 5, n - 1]:
        Wp = W64.copy(); Wp[0, i] += h; Wm = W64.copy(); Wm[0, i] -= h
        fd = (np.sum(g64 * oracle.soft_quantize(Wp, c64, Lb, k, T)["soft"])
              - np.sum(g64 * oracle.soft_quantize(Wm, c64, Lb, k, T)["soft"])) / (2 * h)
        assert abs(fd - out["grad_W"][0, i]) < 1e-7
    for u in [0, 37, 255]:
        cp = c64.copy(); cp[u] += h; cm = c64.copy(); cm[u] -= h
        fd = (np.sum(g64 * oracle.soft_quantize(W64, cp, Lb, k, T)["soft"])
              - np.sum(g64 * oracle.soft_quantize(W64, cm, Lb, k, T)["soft"])) / (2 * h)
        assert abs(fd - out["grad_codebook"][u]) < 1e-7


# ---------------------------------------------------------------- P3: invariants
@pytest.mark.parametrize("Lb,k,n,T", [(8, 2, 64, 0.5), (10, 2, 32, 0.01), (9, 3, 48, 0.001), (6, 1, 50, 0.1)])
def test_marginals_sum_to_one_and_logZ_any_t(Lb, k, n, T):
    rng = np.random.default_rng(5)
    c = rng.standard_normal(1 << Lb).astype(np.float32)
    W = (rng.standard_t(4, size=(2, n)) / np.sqrt(2.0)).astype(np.float32)
    out = oracle.soft_quantize(W, c, Lb, k, T, want_gamma_of=1)
    np.testing.assert_allclose(out["gamma"].sum(axis=1), 1.0, rtol=0, atol=1e-12)
    assert np.all(np.isfinite(out["soft"]))
    # Z = sum_s alpha_t(s) beta_t(s) for any t
    np.testing.assert_allclose(out["logZ_t"], out["logZ"][1], rtol=0, atol=1e-9 * max(1.0, abs(out["logZ"][1])))
    # consecutive marginals are consistent with the trellis: the mass on the states that share
    # their low Lb-k bits at t-1 equals the mass on the states sharing those as high bits at t
    S, K = 1 << Lb, 1 << k
    gam = out["gamma"]
    left = gam[:-1].reshape(n - 1, K, S // K).sum(axis=1)      # sum over the k bits shifted out
    right = gam[1:].reshape(n - 1, S // K, K).sum(axis=2)      # sum over the k bits shifted in
    np.testing.assert_allclose(left, right, rtol=0, atol=1e-12)


# ---------------------------------------------------------------- P4: Viterbi
@pytest.mark.parametrize("n,Lb,k", TINY)
def test_viterbi_matches_exhaustive_argmin(n, Lb, k):
    W, c, _ = _inputs(n, Lb, seed=400 + n + Lb + k, B=5)
    out = oracle.viterbi(W, c, Lb, k)
    for b in range(5):
        states, cost, gap = bf.best_path(W[b], c, Lb, k)
        assert gap > 1e-9                                   # unique minimiser on these seeds
        np.testing.assert_array_equal(out["states"][b], states)
        np.testing.assert_allclose(out["cost"][b], cost, rtol=0, atol=1e-12)
        np.testing.assert_array_equal(out["hard"][b], c[states])
        np.testing.assert_array_equal(out["path_bits"][b], bf.pack_path_bits(states, Lb, k))


def _push_viterbi(w, c, Lb, k):
    """Second, independent DP: relax every edge out of every state ("push" form)."""
    S, K = 1 << Lb, 1 << k
    w = w.astype(np.float64); c = c.astype(np.float64)
    m = (w[0] - c) ** 2
    back = []
    for t in range(1, len(w)):
        new = np.full(S, np.inf); frm = np.zeros(S, dtype=np.int64)
        for s in range(S):                      # ascending s: lowest predecessor wins ties
            for b in range(K):
                s2 = ((s << k) | b) & (S - 1)
                if m[s] < new[s2]:
                    new[s2] = m[s]; frm[s2] = s
        m = new + (w[t] - c) ** 2
        back.append(frm)
    s = int(np.argmin(m)); cost = m[s]
    states = [s]
    for frm in reversed(back):
        s = int(frm[s]); states.append(s)
    return np.array(states[::-1]), cost


@pytest.mark.parametrize("Lb,k,n", [(8, 2, 24), (7, 3, 16), (6, 1, 30), (8, 4, 10)])
def test_viterbi_matches_independent_push_dp(Lb, k, n):
    W, c, _ = _inputs(n, Lb, seed=500 + Lb + k, B=2)
    out = oracle.viterbi(W, c, Lb, k)
    for b in range(2):
        states, cost = _push_viterbi(W[b], c, Lb, k)
        np.testing.assert_array_equal(out["states"][b], states)
        np.testing.assert_allclose(out["cost"][b], cost, rtol=1e-14)


def test_viterbi_is_idempotent_on_its_own_output():
    Lb, k, n = 8, 2, 40
    W, c, _ = _inputs(n, Lb, seed=9, B=3)
    first = oracle.viterbi(W, c, Lb, k)
    again = oracle.viterbi(first["hard"], c, Lb, k)
    np.testing.assert_array_equal(again["hard"], first["hard"])
    np.testing.assert_allclose(again["cost"], 0.0, atol=0)


def test_soft_codeword_tends_to_viterbi_as_T_to_zero():
    # Section 3.3, identity 1.  Checked on blocks whose runner-up path is well separated.
    n, Lb, k = 6, 4, 2
    W, c, _ = _inputs(n, Lb, seed=21, B=6)
    hard = oracle.viterbi(W, c, Lb, k)
    T = 1e-4
    soft = oracle.soft_quantize(W, c, Lb, k, T)["soft"]
    checked = 0
    for b in range(6):
        _, _, gap = bf.best_path(W[b], c, Lb, k)        # gap in sum (w-c)^2 units = 2 * energy gap
        if 0.5 * gap > 20 * T:
            np.testing.assert_allclose(soft[b], hard["hard"][b].astype(np.float64), atol=1e-6)
            checked += 1
    assert checked >= 3
    # and the distance shrinks monotonically with T on every block
    err = [np.abs(oracle.soft_quantize(W, c, Lb, k, t)["soft"] - hard["hard"]).max() for t in (1.0, 0.1, 0.01, 0.001)]
    assert err[0] > err[1] > err[2] > err[3]


# ---------------------------------------------------------------- P5: reductions to library routines
def test_fully_connected_trellis_decouples_into_softmax():
    # Lb = k: every state follows every state, so the steps are independent:
    # gamma_t = softmax_s(-(w_t - c)^2 / 2T), grad_W[t] = g_t Var_gamma(c) / T
    Lb = k = 3; n = 7; T = 0.3
    W, c, g = _inputs(n, Lb, seed=31)
    c64 = c.astype(np.float64); w64 = W[0].astype(np.float64)
    gam = softmax(-(w64[:, None] - c64[None, :]) ** 2 / (2 * T), axis=1)
    out = oracle.soft_quantize(W, c, Lb, k, T, want_gamma_of=0)
    np.testing.assert_allclose(out["gamma"], gam, atol=1e-14)
    np.testing.assert_allclose(out["soft"][0], gam @ c64, atol=1e-14)
    np.testing.assert_allclose(out["logZ"][0], logsumexp(-(w64[:, None] - c64[None, :]) ** 2 / (2 * T), axis=1).sum(), atol=1e-12)
    var = gam @ c64 ** 2 - (gam @ c64) ** 2
    grads = oracle.backward(W, c, g, Lb, k, T)
    np.testing.assert_allclose(grads["grad_W"][0], g[0].astype(np.float64) * var / T, atol=1e-12)


def test_single_step_block_is_a_softmax():
    Lb, k, T = 6, 2, 0.2
    W, c, _ = _inputs(1, Lb, seed=41, B=4)
    c64 = c.astype(np.float64)
    out = oracle.soft_quantize(W, c, Lb, k, T)
    for b in range(4):
        p = softmax(-(float(W[b, 0]) - c64) ** 2 / (2 * T))
        np.testing.assert_allclose(out["soft"][b, 0], p @ c64, atol=1e-14)


def test_infinite_temperature_gives_table_mean():
    Lb, k, n = 6, 2, 9
    W, c, _ = _inputs(n, Lb, seed=51)
    out = oracle.soft_quantize(W, c, Lb, k, 1e12)
    np.testing.assert_allclose(out["soft"][0], c.astype(np.float64).mean(), atol=1e-9)


@pytest.mark.parametrize("Lb,k", [(6, 2), (8, 2), (6, 3), (5, 1)])
def test_matches_dense_transfer_matrix_product(Lb, k):
    # Section 3.4: alpha_t = (alpha_{t-1} M) * exp(e_t) with the 0/1 transfer matrix M; the
    # marginal is alpha_t beta_t / Z.  Linear domain, dense S x S matrix products.
    n, T = 10, 0.7
    S, K = 1 << Lb, 1 << k
    W, c, _ = _inputs(n, Lb, seed=61 + Lb)
    c64 = c.astype(np.float64); w = W[0].astype(np.float64)
    M = np.zeros((S, S))
    for s in range(S):
        for b in range(K):
            M[s, ((s << k) | b) & (S - 1)] = 1.0
    phi = np.exp(-(w[:, None] - c64[None, :]) ** 2 / (2 * T))          # [n, S]
    alpha = [phi[0]]
    for t in range(1, n):
        alpha.append((alpha[-1] @ M) * phi[t])
    beta = [np.ones(S)]
    for t in range(n - 2, -1, -1):
        beta.append(M @ (phi[t + 1] * beta[-1]))
    beta = beta[::-1]
    Z = alpha[-1].sum()
    soft = np.array([(alpha[t] * beta[t] / Z) @ c64 for t in range(n)])
    out = oracle.soft_quantize(W, c, Lb, k, T)
    np.testing.assert_allclose(out["soft"][0], soft, atol=1e-12)
    np.testing.assert_allclose(out["logZ"][0], np.log(Z), atol=1e-11)


def test_low_temperature_stability_student_t():
    Lb, k, n = 10, 3, 64
    rng = np.random.default_rng(71)
    c = rng.standard_normal(1 << Lb).astype(np.float32)
    W = (rng.standard_t(4, size=(2, n)) / np.sqrt(2.0)).astype(np.float32)
    g = rng.standard_normal((2, n)).astype(np.float32)
    for T in (0.01, 0.001):
        out = oracle.soft_quantize(W, c, Lb, k, T, want_gamma_of=0)
        assert np.all(np.isfinite(out["soft"])) and np.all(np.isfinite(out["logZ"]))
        assert np.abs(out["gamma"].sum(axis=1) - 1).max() < 1e-12
        grads = oracle.backward(W, c, g, Lb, k, T)
        assert np.all(np.isfinite(grads["grad_W"])) and np.all(np.isfinite(grads["grad_codebook"]))
        total = grads["grad_W"].sum() + grads["grad_codebook"].sum()
        np.testing.assert_allclose(total, g.astype(np.float64).sum(), atol=1e-8)


def test_invalid_arguments_are_rejected():
    W, c, g = _inputs(4, 4, seed=1)
    with pytest.raises(RuntimeError):
        oracle.soft_quantize(W, c, 4, 2, 0.0)
    with pytest.raises(RuntimeError):
        oracle.soft_quantize(W, c[:4], 2, 3, 1.0)      # k > Lb


# ---------------------------------------------------------------- min-sum helper of the cold-limit tests
@pytest.mark.parametrize("Lb,k,n", [(4, 2, 6), (3, 1, 7), (5, 3, 4), (4, 2, 1)])
def test_minsum_margin_against_enumeration_and_oracle_viterbi(Lb, k, n):
    import minsum
    rng = np.random.default_rng(900 + Lb + n)
    c = rng.standard_normal(1 << Lb).astype(np.float32)
    for trial in range(4):
        w = rng.standard_normal(n).astype(np.float32)
        states, cost, gap = bf.best_path(w, c, Lb, k)
        s2, cost2, margin = minsum.best_and_margin(w, c, Lb, k)
        np.testing.assert_array_equal(s2, states)
        assert abs(cost2 - cost) < 1e-12 and abs(margin - gap) < 1e-12
        ref = oracle.viterbi(w[None], c, Lb, k)
        np.testing.assert_array_equal(ref["states"][0], states)
        assert abs(ref["cost"][0] - cost) < 1e-12


def test_nearest_entry_decoding():
    import minsum
    c = np.array([0.5, -1.0, 2.0, 0.75], dtype=np.float32)
    np.testing.assert_array_equal(minsum.decode_nearest([0.6, 0.7, -3.0, 9.0, 1.3, 1.4], c), [0.5, 0.75, -1.0, 2.0, 0.75, 2.0])

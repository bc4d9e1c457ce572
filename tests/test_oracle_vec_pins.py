"""Pins of the vector-emission oracle (V numbers per state and step) against things other than itself."""
import numpy as np
import pytest
from scipy.special import logsumexp, softmax

import bruteforce as bf
import oracle


def _case(Lb, V, nt, B, seed):
    rng = np.random.default_rng(seed)
    c = rng.standard_normal((1 << Lb, V)).astype(np.float32)
    W = rng.standard_normal((B, nt * V)).astype(np.float32)
    g = rng.standard_normal((B, nt * V)).astype(np.float32)
    return W, c, g


@pytest.mark.parametrize("Lb,kb,V,nt,T", [(4, 2, 2, 5, 0.7), (3, 1, 2, 6, 0.2), (4, 4, 2, 3, 1.3), (5, 2, 3, 4, 0.5)])
def test_soft_codeword_and_logz_equal_enumeration_of_every_path(Lb, kb, V, nt, T):
    W, c, _ = _case(Lb, V, nt, 2, seed=70 + Lb + V)
    ref = oracle.soft_quantize_vec(W, c, Lb, kb, V, T)
    for b in range(2):
        soft, logZ = bf.vec_soft_codeword(W[b], c, Lb, kb, V, T)
        np.testing.assert_allclose(ref["soft"][b], soft, rtol=0, atol=1e-12)
        assert abs(ref["logZ"][b] - logZ) < 1e-11


@pytest.mark.parametrize("Lb,kb,V,nt,T", [(4, 2, 2, 4, 0.6), (3, 1, 2, 5, 0.25)])
def test_gradients_equal_finite_differences_of_the_enumeration(Lb, kb, V, nt, T):
    W, c, g = _case(Lb, V, nt, 1, seed=90 + Lb)
    ref = oracle.backward_vec(W, c, g, Lb, kb, V, T)
    gw, gc = bf.vec_fd_gradients(W[0], c, g[0], Lb, kb, V, T)
    np.testing.assert_allclose(ref["grad_W"][0], gw, rtol=0, atol=2e-8)
    np.testing.assert_allclose(ref["grad_codebook"], gc, rtol=0, atol=2e-8)


def test_table_gradient_sums_over_blocks():
    Lb, kb, V, nt, T = 4, 2, 2, 4, 0.5
    W, c, g = _case(Lb, V, nt, 3, seed=5)
    tot = oracle.backward_vec(W, c, g, Lb, kb, V, T)
    parts = [oracle.backward_vec(W[b:b + 1], c, g[b:b + 1], Lb, kb, V, T) for b in range(3)]
    np.testing.assert_allclose(tot["grad_codebook"], sum(p["grad_codebook"] for p in parts), atol=1e-13)
    for b in range(3):
        np.testing.assert_allclose(tot["grad_W"][b], parts[b]["grad_W"][0], atol=0)


@pytest.mark.parametrize("Lb,k,n,T", [(6, 2, 7, 0.4), (5, 3, 5, 1.0)])
def test_single_emission_reduces_to_the_scalar_oracle(Lb, k, n, T):
    W, c, g = _case(Lb, 1, n, 3, seed=11)
    a = oracle.soft_quantize_vec(W, c, Lb, k, 1, T); b = oracle.soft_quantize(W, c[:, 0], Lb, k, T)
    np.testing.assert_allclose(a["soft"], b["soft"], atol=1e-14); np.testing.assert_allclose(a["logZ"], b["logZ"], atol=1e-13)
    ga = oracle.backward_vec(W, c, g, Lb, k, 1, T); gb = oracle.backward(W, c[:, 0], g, Lb, k, T)
    np.testing.assert_allclose(ga["grad_W"], gb["grad_W"], atol=1e-13)
    np.testing.assert_allclose(ga["grad_codebook"][:, 0], gb["grad_codebook"], atol=1e-13)
    va = oracle.viterbi_vec(W, c, Lb, k, 1); vb = oracle.viterbi(W, c[:, 0], Lb, k)
    for key in ("states", "hard", "path_bits", "cost"):
        np.testing.assert_array_equal(va[key], vb[key])


def test_constant_second_column_leaves_a_scalar_problem():
    # c[s, 1] = const: the second weight of every step adds a state-independent energy, so the
    # first components follow the scalar trellis on W[:, 0::2] and the second ones equal the constant
    Lb, kb, nt, T = 6, 2, 6, 0.3
    W, c, g = _case(Lb, 2, nt, 2, seed=21)
    c[:, 1] = 0.625
    a = oracle.soft_quantize_vec(W, c, Lb, kb, 2, T)
    b = oracle.soft_quantize(W[:, 0::2], c[:, 0], Lb, kb, T)
    np.testing.assert_allclose(a["soft"][:, 0::2], b["soft"], atol=1e-13)
    np.testing.assert_allclose(a["soft"][:, 1::2], 0.625, atol=1e-13)
    shift = -0.5 * ((W[:, 1::2].astype(np.float64) - 0.625) ** 2).sum(axis=1) / T
    np.testing.assert_allclose(a["logZ"], b["logZ"] + shift, atol=1e-11)
    # gradient w.r.t. the second weights vanishes (they only shift log Z); the first ones match
    g2 = g.copy(); g2[:, 1::2] = 0.0
    ga = oracle.backward_vec(W, c, g2, Lb, kb, 2, T); gb = oracle.backward(W[:, 0::2], c[:, 0], g[:, 0::2], Lb, kb, T)
    np.testing.assert_allclose(ga["grad_W"][:, 0::2], gb["grad_W"], atol=1e-12)
    np.testing.assert_allclose(ga["grad_W"][:, 1::2], 0.0, atol=1e-12)
    np.testing.assert_allclose(ga["grad_codebook"][:, 0], gb["grad_codebook"], atol=1e-12)


def test_memoryless_trellis_is_one_softmax_per_step():
    # Lb = kb: every state follows every state, the steps are independent
    Lb = kb = 3; V = 2; nt = 5; T = 0.45
    W, c, _ = _case(Lb, V, nt, 2, seed=31)
    ref = oracle.soft_quantize_vec(W, c, Lb, kb, V, T)
    c64 = c.astype(np.float64)
    for b in range(2):
        w = W[b].astype(np.float64).reshape(nt, V)
        e = -0.5 * ((w[:, None, :] - c64[None]) ** 2).sum(axis=2) / T          # [nt, S]
        soft = softmax(e, axis=1) @ c64
        np.testing.assert_allclose(ref["soft"][b], soft.reshape(-1), atol=1e-13)
        assert abs(ref["logZ"][b] - logsumexp(e, axis=1).sum()) < 1e-11


@pytest.mark.parametrize("Lb,kb,V,nt", [(4, 2, 2, 5), (3, 1, 2, 6), (4, 4, 2, 3)])
def test_viterbi_equals_exhaustive_search(Lb, kb, V, nt):
    W, c, _ = _case(Lb, V, nt, 4, seed=41 + kb)
    ref = oracle.viterbi_vec(W, c, Lb, kb, V)
    for b in range(4):
        states, cost, gap = bf.vec_best_path(W[b], c, Lb, kb, V)
        assert gap > 1e-9
        np.testing.assert_array_equal(ref["states"][b], states)
        assert abs(ref["cost"][b] - cost) < 1e-12
        np.testing.assert_array_equal(ref["hard"][b], c[states].reshape(-1))
        np.testing.assert_array_equal(ref["path_bits"][b], bf.pack_path_bits(states, Lb, kb))


def test_cold_limit_of_the_soft_codeword_is_the_viterbi_codeword():
    Lb, kb, V, nt = 6, 2, 2, 6
    W, c, _ = _case(Lb, V, nt, 3, seed=51)
    soft = oracle.soft_quantize_vec(W, c, Lb, kb, V, 1e-5)["soft"]
    hard = oracle.viterbi_vec(W, c, Lb, kb, V)["hard"]
    np.testing.assert_allclose(soft, hard, atol=1e-6)


def test_bad_arguments_are_rejected():
    W, c, _ = _case(4, 2, 3, 1, seed=1)
    with pytest.raises(RuntimeError):
        oracle.soft_quantize_vec(W[:, :5], c, 4, 2, 2, 0.5)        # n not a multiple of V
    with pytest.raises(RuntimeError):
        oracle.soft_quantize_vec(W, c, 4, 5, 2, 0.5)               # more than 4 bits per step

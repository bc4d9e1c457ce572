"""The oracle reproduces the stored expected values of the seeded tiny workload.

The stored file is written by tests/golden/make_golden.py from the oracle alone; this test
guards the oracle (and the seeded generators) against silent drift.
"""
import json
from pathlib import Path

import numpy as np

import oracle
from paper_2605_10655_b200 import synth

GOLD = json.loads((Path(__file__).parent / "golden" / "tiny_expected.json").read_text())


def test_oracle_reproduces_stored_tiny_values():
    wl = synth.tiny()
    W, c, g = wl.weights(), wl.codebook(), wl.upstream()
    assert GOLD["workload"] == {"name": wl.name, "Lb": wl.Lb, "k": wl.k, "n": wl.n, "T": wl.T, "blocks": 64}
    fwd = oracle.soft_quantize(W, c, wl.Lb, wl.k, wl.T)
    bwd = oracle.backward(W, c, g, wl.Lb, wl.k, wl.T)
    vit = oracle.viterbi(W, c, wl.Lb, wl.k)
    np.testing.assert_allclose(fwd["soft"][0], GOLD["soft_block0"], atol=1e-13)
    np.testing.assert_allclose(fwd["soft"][63], GOLD["soft_block63"], atol=1e-13)
    np.testing.assert_allclose(fwd["logZ"], GOLD["logZ"], atol=1e-10)
    np.testing.assert_allclose(bwd["grad_W"][0], GOLD["grad_W_block0"], atol=1e-12)
    np.testing.assert_allclose(bwd["grad_W"][63], GOLD["grad_W_block63"], atol=1e-12)
    np.testing.assert_allclose(bwd["grad_codebook"], GOLD["grad_codebook"], atol=1e-11)
    assert vit["states"][0].tolist() == GOLD["viterbi_states_block0"]
    assert [bytes(r).hex() for r in vit["path_bits"]] == GOLD["viterbi_path_bits_hex"]


def test_oracle_reproduces_stored_vector_emission_values():
    import importlib.util
    spec = importlib.util.spec_from_file_location("make_golden", Path(__file__).parent / "golden" / "make_golden.py")
    mg = importlib.util.module_from_spec(spec); spec.loader.exec_module(mg)
    gold = json.loads((Path(__file__).parent / "golden" / "vec_expected.json").read_text())
    Lb, k, V, T, W, c, g = mg.vec_case()
    assert gold["case"] == {"Lb": Lb, "k": k, "V": V, "n": 32, "blocks": 8, "T": T, "seed": 20605}
    fwd = oracle.soft_quantize_vec(W, c, Lb, k * V, V, T)
    bwd = oracle.backward_vec(W, c, g, Lb, k * V, V, T)
    vit = oracle.viterbi_vec(W, c, Lb, k * V, V)
    np.testing.assert_allclose(fwd["soft"][0], gold["soft_block0"], atol=1e-13)
    np.testing.assert_allclose(fwd["logZ"], gold["logZ"], atol=1e-10)
    np.testing.assert_allclose(bwd["grad_W"][0], gold["grad_W_block0"], atol=1e-12)
    np.testing.assert_allclose(bwd["grad_codebook"][:8], gold["grad_codebook_rows_0_7"], atol=1e-11)
    np.testing.assert_allclose(bwd["grad_codebook"].sum(axis=0), gold["grad_codebook_sum"], atol=1e-10)
    assert vit["states"][0].tolist() == gold["viterbi_states_block0"]
    assert [bytes(r).hex() for r in vit["path_bits"]] == gold["viterbi_path_bits_hex"]

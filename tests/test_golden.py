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

"""Writes tests/golden/tiny_expected.json and vec_expected.json from the float64 CPU oracle alone.

Run from the repository root:  python tests/golden/make_golden.py
The paper prints no numeric worked example (no soft codeword, gradient or path appears in
its text), so these stored values are the oracle's, on the seeded "tiny" workload
(64 blocks of 64 weights, Lb=8, k=2, T=0.5), after the oracle itself has been pinned to
path enumeration and finite differences by tests/test_oracle_pins.py.
"""
import json
import sys
from pathlib import Path

import numpy as np

ROOT = Path(__file__).resolve().parents[2]
sys.path.insert(0, str(ROOT))

import oracle  # noqa: E402
from paper_2605_10655_b200 import synth  # noqa: E402


def main():
    wl = synth.tiny()
    W, c, g = wl.weights(), wl.codebook(), wl.upstream()
    fwd = oracle.soft_quantize(W, c, wl.Lb, wl.k, wl.T)
    bwd = oracle.backward(W, c, g, wl.Lb, wl.k, wl.T)
    vit = oracle.viterbi(W, c, wl.Lb, wl.k)
    out = {
        "workload": {"name": wl.name, "Lb": wl.Lb, "k": wl.k, "n": wl.n, "T": wl.T, "blocks": wl.num_blocks()},
        "soft_block0": fwd["soft"][0].tolist(),
        "soft_block63": fwd["soft"][63].tolist(),
        "logZ": fwd["logZ"].tolist(),
        "grad_W_block0": bwd["grad_W"][0].tolist(),
        "grad_W_block63": bwd["grad_W"][63].tolist(),
        "grad_codebook": bwd["grad_codebook"].tolist(),
        "viterbi_states_block0": vit["states"][0].tolist(),
        "viterbi_path_bits_hex": [bytes(r).hex() for r in vit["path_bits"]],
        "viterbi_cost": vit["cost"].tolist(),
    }
    path = Path(__file__).with_name("tiny_expected.json")
    path.write_text(json.dumps(out, indent=0))
    print("wrote", path, path.stat().st_size, "bytes")
    write_vec()


def vec_case():
    """Seeded vector-emission case: 8 blocks of 32 weights, Lb=8, 2 bits per weight, 2 weights per step."""
    rng = np.random.default_rng(20605)
    Lb, k, V, n, B, T = 8, 2, 2, 32, 8, 0.4
    c = rng.standard_normal((1 << Lb, V)).astype(np.float32)
    W = rng.standard_normal((B, n)).astype(np.float32)
    g = rng.standard_normal((B, n)).astype(np.float32)
    return Lb, k, V, T, W, c, g


def write_vec():
    Lb, k, V, T, W, c, g = vec_case()
    fwd = oracle.soft_quantize_vec(W, c, Lb, k * V, V, T)
    bwd = oracle.backward_vec(W, c, g, Lb, k * V, V, T)
    vit = oracle.viterbi_vec(W, c, Lb, k * V, V)
    out = {
        "case": {"Lb": Lb, "k": k, "V": V, "n": int(W.shape[1]), "blocks": int(W.shape[0]), "T": T, "seed": 20605},
        "soft_block0": fwd["soft"][0].tolist(),
        "logZ": fwd["logZ"].tolist(),
        "grad_W_block0": bwd["grad_W"][0].tolist(),
        "grad_codebook_rows_0_7": bwd["grad_codebook"][:8].tolist(),
        "grad_codebook_sum": bwd["grad_codebook"].sum(axis=0).tolist(),
        "viterbi_states_block0": vit["states"][0].tolist(),
        "viterbi_path_bits_hex": [bytes(r).hex() for r in vit["path_bits"]],
    }
    path = Path(__file__).with_name("vec_expected.json")
    path.write_text(json.dumps(out, indent=0))
    print("wrote", path, path.stat().st_size, "bytes")


if __name__ == "__main__":
    main()

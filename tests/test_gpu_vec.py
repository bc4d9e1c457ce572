"""GPU parity of the vector-emission calls (V weights per trellis step) against the float64 oracle."""
import numpy as np
import pytest

import oracle
import parity

pytestmark = pytest.mark.gpu


@pytest.fixture(scope="module")
def ctx():
    from paper_2605_10655_b200 import Context
    c = Context(0)
    yield c
    c.close()


def _case(Lb, V, nt, B, seed):
    rng = np.random.default_rng(seed)
    c = rng.standard_normal((1 << Lb, V)).astype(np.float32)
    W = rng.standard_normal((B, nt * V)).astype(np.float32)
    g = rng.standard_normal((B, nt * V)).astype(np.float32)
    return W, c, g


def _run(ctx, W, c, g, Lb, k, V, T, viterbi=True):
    import torch
    dev = torch.device("cuda", ctx.device)
    n = W.shape[1]
    Wd, cd, gd = (torch.from_numpy(np.ascontiguousarray(a)).to(dev) for a in (W, c, g))
    soft, logZ = ctx.bcjr_soft_quantize_vec(Wd, cd, Lb, k, V, n, T)
    fwd_path = ctx.sync_status().last_path
    gW, gc = ctx.bcjr_backward(gd)
    diag = ctx.sync_status()
    out = {"soft": soft.cpu().numpy(), "logZ": logZ.cpu().numpy(), "grad_W": gW.cpu().numpy(),
           "grad_codebook": gc.cpu().numpy().reshape(1 << Lb, V), "diag": diag, "fwd_path": fwd_path}
    if viterbi:
        bits, states, hard = ctx.viterbi_hard_vec(Wd, cd, Lb, k, V, n)
        ctx.sync_status()
        out.update(path_bits=bits.cpu().numpy(), states=states.cpu().numpy().view(np.uint16), hard=hard.cpu().numpy())
    return out


def _check(ctx, Lb, k, V, nt, B, T, seed, what):
    W, c, g = _case(Lb, V, nt, B, seed)
    got = _run(ctx, W, c, g, Lb, k, V, T)
    kb = k * V
    ref_f = oracle.soft_quantize_vec(W, c, Lb, kb, V, T)
    ref_b = oracle.backward_vec(W, c, g, Lb, kb, V, T)
    parity.assert_forward_backward(got, ref_f, ref_b, what)
    assert got["diag"].device_status == 0 and got["diag"].max_posterior_defect < 1e-3, what
    parity.assert_viterbi(got, oracle.viterbi_vec(W, c, Lb, kb, V), what)
    return got


@pytest.mark.parametrize("Lb,k,nt,B,T", [
    (4, 2, 5, 3, 0.7),        # the enumerable case of the oracle's pins
    (4, 1, 6, 2, 0.3),
    (8, 2, 32, 24, 0.5),
    (8, 1, 33, 5, 0.1),
    (12, 2, 64, 9, 0.2),
    (12, 1, 17, 300, 1.0),    # more blocks than resident thread blocks, odd step count
    (5, 2, 7, 4, 0.05),       # Lb not a multiple of the 4 bits per step
])
def test_two_weights_per_step_small_and_mid_trellises(ctx, Lb, k, nt, B, T):
    _check(ctx, Lb, k, 2, nt, B, T, seed=8000 + Lb * 10 + k, what=f"V=2 Lb={Lb} k={k} nt={nt} B={B} T={T}")


@pytest.mark.parametrize("path", [0, 1], ids=["cluster", "generic"])
@pytest.mark.parametrize("T", [0.3, 0.05])
def test_sixteen_bit_state_sixteen_predecessors(ctx, T, path):
    # the paper's own configuration: Lb = 16, 2 bits per weight, 2 weights per step; on the
    # cluster kernels (default) and on the one-CTA-per-block kernels
    ctx.set_option("path", path)
    try:
        got = _check(ctx, 16, 2, 2, 24, 3, T, seed=8100, what=f"V=2 Lb=16 k=2 T={T} path={path}")
        assert got["fwd_path"] == (1 if path == 0 else 0)
    finally:
        ctx.set_option("path", 0)


@pytest.mark.parametrize("nt,B", [(1, 2), (2, 5), (3, 1), (37, 70)])
def test_cluster_kernels_ragged_step_counts_and_more_blocks_than_clusters(ctx, nt, B):
    _check(ctx, 16, 2, 2, nt, B, 0.2, seed=8500 + nt, what=f"V=2 Lb=16 nt={nt} B={B}")


@pytest.mark.parametrize("fwd_variant", [0, 1], ids=["clusters_of_two", "clusters_of_four"])
def test_cluster_forward_kernels_several_batches_per_cluster(ctx, fwd_variant):
    # both forward kernels (two-CTA clusters, the default, and four-CTA clusters) with the resident CTAs capped so
    # that every cluster works through several batches of blocks in flight, the last one ragged
    ctx.set_option("fwd_variant", fwd_variant)
    ctx.set_option("max_ctas", 8)
    try:
        got = _check(ctx, 16, 2, 2, 9, 19, 0.15, seed=8600 + fwd_variant, what=f"V=2 Lb=16 B=19 capped, fwd_variant={fwd_variant}")
        assert got["fwd_path"] == 1
    finally:
        ctx.set_option("fwd_variant", 0)
        ctx.set_option("max_ctas", 0)


def test_sixteen_bit_state_one_bit_per_weight(ctx):
    _check(ctx, 16, 1, 2, 20, 2, 0.2, seed=8200, what="V=2 Lb=16 k=1")


def test_full_block_length_sampled_blocks(ctx):
    # 256-weight blocks (128 steps) as the paper cuts them; the oracle checks a few blocks
    Lb, k, V, nt, T = 16, 2, 2, 128, 0.1
    W, c, g = _case(Lb, V, nt, 150, seed=8300)
    got = _run(ctx, W, c, g, Lb, k, V, T, viterbi=True)
    pick = [0, 17, 38, 71, 99, 120, 133, 149]
    ref_f = oracle.soft_quantize_vec(W[pick], c, Lb, k * V, V, T)
    assert parity.rel_inf(got["soft"][pick], ref_f["soft"]) <= parity.SOFT_TOL
    ref_b = oracle.backward_vec(W[pick], c, g[pick], Lb, k * V, V, T)
    assert parity.rel_inf(got["grad_W"][pick], ref_b["grad_W"]) <= parity.GRAD_TOL
    # grad_codebook sums over the blocks of a call: compare it on a call of its own over the picked blocks
    sub = _run(ctx, W[pick], c, g[pick], Lb, k, V, T)
    assert parity.rel_inf(sub["grad_codebook"], ref_b["grad_codebook"]) <= parity.GRAD_TOL
    assert parity.rel_inf(sub["grad_W"], ref_b["grad_W"]) <= parity.GRAD_TOL
    ref_v = oracle.viterbi_vec(W[pick], c, Lb, k * V, V)
    np.testing.assert_array_equal(got["states"][pick], ref_v["states"])
    np.testing.assert_array_equal(got["hard"][pick].view(np.uint32), ref_v["hard"].view(np.uint32))
    np.testing.assert_array_equal(got["path_bits"][pick], ref_v["path_bits"])
    # properties that hold for every block: the hard codeword is made of table rows along a legal path
    st = got["states"].astype(np.int64)
    assert np.all((st[:, 1:] >> 4) == (st[:, :-1] & 0xFFF))
    np.testing.assert_array_equal(got["hard"].reshape(150, nt, V), c[st])
    assert got["diag"].max_posterior_defect < 1e-3


def test_long_blocks_fall_back_to_the_one_cta_kernels(ctx):
    # 1030 weights per block: the cluster forward kernel still takes it (<= 2048), the cluster
    # backward kernel does not (<= 1024) and hands over to the one-CTA kernel; 2100 exceeds both
    for nt in (515, 1050):
        got = _check(ctx, 16, 2, 2, nt, 1, 0.3, seed=8600 + nt, what=f"V=2 Lb=16 nt={nt}")
        assert got["diag"].device_status == 0


def test_stored_vector_emission_values(ctx):
    import importlib.util
    import json
    from pathlib import Path
    here = Path(__file__).parent
    spec = importlib.util.spec_from_file_location("make_golden", here / "golden" / "make_golden.py")
    mg = importlib.util.module_from_spec(spec); spec.loader.exec_module(mg)
    gold = json.loads((here / "golden" / "vec_expected.json").read_text())
    Lb, k, V, T, W, c, g = mg.vec_case()
    got = _run(ctx, W, c, g, Lb, k, V, T)
    assert parity.rel_inf(got["soft"][0], gold["soft_block0"]) <= parity.SOFT_TOL
    assert parity.rel_inf(got["grad_W"][0], gold["grad_W_block0"]) <= parity.GRAD_TOL
    assert parity.rel_inf(got["grad_codebook"].sum(axis=0), gold["grad_codebook_sum"]) <= parity.GRAD_TOL
    assert got["states"][0].tolist() == gold["viterbi_states_block0"]
    assert [bytes(r).hex() for r in got["path_bits"]] == gold["viterbi_path_bits_hex"]


def test_single_emission_forwards_to_the_scalar_call_and_bad_arguments(ctx):
    import torch
    from paper_2605_10655_b200 import BcjrError
    dev = torch.device("cuda", ctx.device)
    W, c, g = _case(8, 1, 16, 4, seed=8400)
    Wd, cd = torch.from_numpy(W).to(dev), torch.from_numpy(c).to(dev)
    a, _ = ctx.bcjr_soft_quantize_vec(Wd, cd, 8, 2, 1, 16, 0.5)
    b, _ = ctx.bcjr_soft_quantize(Wd, cd.reshape(-1), 8, 2, 16, 0.5)
    ctx.sync_status()
    assert torch.equal(a, b)
    c2 = torch.from_numpy(np.repeat(c, 2, axis=1)).to(dev)
    with pytest.raises(BcjrError) as e:                       # n not a multiple of V
        ctx.bcjr_soft_quantize_vec(Wd[:, :15].contiguous(), c2, 8, 2, 2, 15, 0.5)
    assert e.value.code == -1
    with pytest.raises(BcjrError) as e:                       # 3 bits per weight x 2 weights: more than 4 bits per step
        ctx.bcjr_soft_quantize_vec(Wd, c2, 8, 3, 2, 16, 0.5)
    assert e.value.code == -5
    with pytest.raises(BcjrError) as e:                       # a pointer that is not 8-byte aligned
        ctx.bcjr_soft_quantize_vec(Wd.reshape(-1)[1:33], c2, 8, 2, 2, 16, 0.5)
    assert e.value.code == -1

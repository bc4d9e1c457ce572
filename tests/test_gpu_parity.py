"""GPU parity: the CUDA path (called through the C ABI) against the float64 CPU oracle,
element by element, on the same seeded inputs."""
import json
from pathlib import Path

import numpy as np
import pytest

import bruteforce as bf
import oracle
import parity
from oracle import qat_oracle as qo
from paper_2605_10655_b200 import synth

pytestmark = pytest.mark.gpu

GENERIC, CLUSTER = 1, 2


@pytest.fixture(scope="module")
def ctx():
    from paper_2605_10655_b200 import Context
    c = Context(0)
    yield c
    c.close()


def _rand(n, Lb, B, seed, student=False):
    rng = np.random.default_rng(seed)
    c = rng.standard_normal(1 << Lb).astype(np.float32)
    W = (rng.standard_t(4, size=(B, n)) / np.sqrt(2.0)).astype(np.float32) if student \
        else rng.standard_normal((B, n)).astype(np.float32)
    g = rng.standard_normal((B, n)).astype(np.float32)
    return W, c, g


def _check_all(ctx, W, c, g, Lb, k, T, what, viterbi=True):
    got = parity.gpu_forward_backward(ctx, W, c, g, Lb, k, T)
    ref_f = oracle.soft_quantize(W, c, Lb, k, T)
    ref_b = oracle.backward(W, c, g, Lb, k, T)
    parity.assert_forward_backward(got, ref_f, ref_b, what)
    assert got["diag"].max_posterior_defect < 1e-3, what
    if viterbi:
        parity.assert_viterbi(parity.gpu_viterbi(ctx, W, c, Lb, k), oracle.viterbi(W, c, Lb, k), what)
    return got


# ------------------------------------------------------------------ tiny workload, all blocks
def test_tiny_workload_all_blocks(ctx):
    ctx.set_option("path", 0)
    wl = synth.tiny()
    W, c, g = wl.weights(), wl.codebook(), wl.upstream()
    got = _check_all(ctx, W, c, g, wl.Lb, wl.k, wl.T, "tiny")
    gold = json.loads((Path(__file__).parent / "golden" / "tiny_expected.json").read_text())
    assert parity.rel_inf(got["soft"][0], gold["soft_block0"]) <= parity.SOFT_TOL
    assert parity.rel_inf(got["grad_codebook"], gold["grad_codebook"]) <= parity.GRAD_TOL


def test_enumerable_case_against_every_path(ctx):
    wl = synth.brute()
    W, c, g = wl.weights(), wl.codebook(), wl.upstream()
    got = parity.gpu_forward_backward(ctx, W, c, g, wl.Lb, wl.k, wl.T)
    vit = parity.gpu_viterbi(ctx, W, c, wl.Lb, wl.k)
    for b in range(W.shape[0]):
        soft, logZ, _ = bf.soft_codeword(W[b], c, wl.Lb, wl.k, wl.T)
        assert parity.rel_inf(got["soft"][b], soft) <= parity.SOFT_TOL
        assert abs(got["logZ"][b] - logZ) < 1e-4
        states, _, gap = bf.best_path(W[b], c, wl.Lb, wl.k)
        assert gap > 1e-6
        np.testing.assert_array_equal(vit["states"][b], states)
        np.testing.assert_array_equal(vit["path_bits"][b], bf.pack_path_bits(states, wl.Lb, wl.k))
    gw, gc = bf.fd_gradients(W[0], c, g[0].astype(np.float64), wl.Lb, wl.k, wl.T)
    one = parity.gpu_forward_backward(ctx, W[:1], c, g[:1], wl.Lb, wl.k, wl.T)
    assert parity.rel_inf(one["grad_W"][0], gw) <= parity.GRAD_TOL
    assert parity.rel_inf(one["grad_codebook"], gc) <= parity.GRAD_TOL


# ------------------------------------------------------------------ shapes, ragged sizes, edge cases
SHAPES = [  # (Lb, k, n, B, T)
    (4, 2, 6, 5, 0.5), (2, 2, 7, 3, 0.3), (3, 2, 9, 4, 0.4), (5, 3, 11, 3, 0.2), (4, 4, 5, 2, 1.0),
    (6, 1, 33, 7, 0.1), (8, 2, 64, 301, 0.5), (9, 3, 40, 10, 0.05), (10, 4, 17, 9, 0.2), (7, 1, 1, 6, 0.3),
    (8, 2, 2, 4, 0.2), (11, 2, 100, 13, 0.02), (13, 3, 30, 5, 0.1), (15, 1, 12, 2, 0.3),
]


@pytest.mark.parametrize("Lb,k,n,B,T", SHAPES)
def test_shapes_generic_path(ctx, Lb, k, n, B, T):
    ctx.set_option("path", GENERIC)
    try:
        W, c, g = _rand(n, Lb, B, seed=1000 + Lb * 10 + k)
        _check_all(ctx, W, c, g, Lb, k, T, f"Lb={Lb} k={k} n={n}")
    finally:
        ctx.set_option("path", 0)


@pytest.mark.parametrize("Lb,n,B,T", [(11, 33, 37, 0.3), (12, 1, 3, 0.5), (12, 2, 70, 0.2), (12, 256, 40, 0.1), (13, 50, 9, 0.05),
                                      (13, 7, 1, 0.3), (12, 1500, 2, 0.2), (11, 64, 300, 0.02)])
def test_one_warp_per_block_kernels(ctx, Lb, n, B, T):
    # Lb = 11..13, k = 2: a warp runs a block alone (no CTA barrier in the sweeps), sixteen or eight blocks per CTA;
    # ragged block counts leave warps without work, long blocks exercise the history stream
    k = 2
    W, c, g = _rand(n, Lb, B, seed=1300 + Lb + n)
    got = _check_all(ctx, W, c, g, Lb, k, T, f"warp per block Lb={Lb} n={n} B={B}")
    assert got["diag"].last_path == 2 and got["diag"].device_status == 0
    ctx.set_option("max_ctas", 2)                       # fewer CTAs than the work needs: every warp loops over blocks
    try:
        again = parity.gpu_forward_backward(ctx, W, c, g, Lb, k, T)
    finally:
        ctx.set_option("max_ctas", 0)
    np.testing.assert_array_equal(again["soft"], got["soft"])
    np.testing.assert_array_equal(again["grad_W"], got["grad_W"])
    assert parity.rel_inf(again["grad_codebook"], got["grad_codebook"]) < 1e-5
    if Lb >= 12:
        # with grad_codebook the default at Lb = 12, 13 gives a block to two warps; the one-warp kernel stays selectable
        ctx.set_option("bwd_variant", 1)
        try:
            one = _check_all(ctx, W, c, g, Lb, k, T, f"one warp per block (backward) Lb={Lb} n={n} B={B}", viterbi=False)
        finally:
            ctx.set_option("bwd_variant", 0)
        assert one["diag"].last_path == 2 and parity.rel_inf(one["grad_W"], got["grad_W"]) < 2e-5


def test_more_blocks_than_resident_ctas(ctx):
    # the persistent loop must visit every block exactly once, whatever the grid size
    Lb, k, n, T = 8, 2, 16, 0.3
    W, c, g = _rand(n, Lb, 37, seed=77)
    ref = parity.gpu_forward_backward(ctx, W, c, g, Lb, k, T)
    ctx.set_option("max_ctas", 5)
    try:
        got = parity.gpu_forward_backward(ctx, W, c, g, Lb, k, T)
        vit = parity.gpu_viterbi(ctx, W, c, Lb, k)
    finally:
        ctx.set_option("max_ctas", 0)
    np.testing.assert_array_equal(got["soft"], ref["soft"])
    np.testing.assert_array_equal(got["grad_W"], ref["grad_W"])
    assert parity.rel_inf(got["grad_codebook"], ref["grad_codebook"]) < 1e-5
    parity.assert_viterbi(vit, oracle.viterbi(W, c, Lb, k), "max_ctas=5")


def test_empty_input_and_argument_errors(ctx):
    import torch
    from paper_2605_10655_b200 import BcjrError, Context
    dev = torch.device("cuda", 0)
    c = torch.zeros(256, device=dev)
    W = torch.zeros((0, 64), device=dev)
    soft, logZ = ctx.bcjr_soft_quantize(W, c, 8, 2, 64, 0.5)
    assert soft.numel() == 0
    gW, gc = ctx.bcjr_backward(torch.zeros((0, 64), device=dev))
    ctx.sync_status()
    assert float(gc.abs().max()) == 0.0
    W = torch.zeros((2, 64), device=dev)
    for bad in [dict(Lb=8, k=2, T=0.0), dict(Lb=8, k=2, T=float("nan")), dict(Lb=8, k=5, T=1.0),
                dict(Lb=8, k=0, T=1.0)]:
        with pytest.raises(BcjrError) as ei:
            ctx.bcjr_soft_quantize(W, c, bad["Lb"], bad["k"], 64, bad["T"])
        assert ei.value.code == -1
    with pytest.raises(BcjrError) as ei:
        ctx.bcjr_soft_quantize(torch.zeros((1, 4), device=dev), torch.zeros(1 << 16, device=dev), 16, 1, 4, 1.0)
    assert ei.value.code == -5
    fresh = Context(0)
    try:
        rc = fresh._lib.bcjr_backward(fresh._h, W.data_ptr(), W.data_ptr(), None, None)  # noqa
        assert rc == -4                                 # backward before any forward
    finally:
        fresh.close()


# ------------------------------------------------------------------ mid trellis (S = 4096)
@pytest.mark.parametrize("T", [1.0, 0.1, 0.01])
def test_mid_trellis_temperature_sweep(ctx, T):
    wl = synth.mid()
    idx = synth.sample_blocks(wl.num_blocks(), 512)
    W, c, g = wl.weights()[idx], wl.codebook(), wl.upstream()[idx]
    _check_all(ctx, W, c, g, wl.Lb, wl.k, T, f"mid T={T}", viterbi=(T == 1.0))


def _cold_limit_statistics(soft_gpu, soft_ref, W, c, Lb, k, T, what):
    """Section 3.3, identity 1 (as T -> 0 the soft codeword tends to the Viterbi hard code), stated for a
    finite T.  A block has converged when no other path comes close to the best one: its margin
    (squared error of the best path that leaves the Viterbi path somewhere, minus the Viterbi path's)
    exceeds 20 T / kappa with kappa = 1/2, so that every other path carries less than e^-20 of the
    Viterbi path's weight.  On those blocks the soft codeword, decoded to the nearest table entry, must
    BE the hard code at every position, for the oracle and for the GPU alike.  Over all blocks the
    agreement is reported as the fraction of positions within 1e-3 of the hard code."""
    import minsum
    B = W.shape[0]
    margin = np.empty(B); hard = np.empty(W.shape)
    for b in range(B):
        st, _, margin[b] = minsum.best_and_margin(W[b], c, Lb, k)
        hard[b] = c.astype(np.float64)[st]
    conv = margin > 20.0 * T / 0.5
    dec_ref = np.stack([minsum.decode_nearest(soft_ref[b], c) for b in range(B)])
    dec_gpu = np.stack([minsum.decode_nearest(soft_gpu[b], c) for b in range(B)])
    ref_blocks_differ = [int(b) for b in range(B) if not np.array_equal(dec_ref[b], hard[b])]
    frac_ref = float((np.abs(soft_ref - hard) <= 1e-3).mean())
    frac_gpu = float((np.abs(soft_gpu - hard) <= 1e-3).mean())
    worst_conv = float(np.abs(soft_gpu[conv] - hard[conv]).max()) if conv.any() else 0.0
    print(f"\n{what}: T={T}: {int(conv.sum())}/{B} blocks past the margin 20T/kappa; positions within 1e-3 of the hard "
          f"code: oracle {frac_ref:.4f}, GPU {frac_gpu:.4f}; max |soft - hard| on converged blocks {worst_conv:.2e}; "
          f"blocks whose decoded oracle soft codeword differs from the hard code: {len(ref_blocks_differ)} "
          f"(none of them converged: {not any(conv[b] for b in ref_blocks_differ)})")
    assert not any(conv[b] for b in ref_blocks_differ), what + ": the oracle itself disagrees on a converged block"
    for b in np.nonzero(conv)[0]:
        np.testing.assert_array_equal(dec_gpu[b], hard[b], err_msg=f"{what}: block {b} (margin {margin[b]:.3g})")
    assert worst_conv <= 1e-3
    assert abs(frac_gpu - frac_ref) <= 2e-3
    return conv


def test_mid_trellis_cold_limit_matches_viterbi(ctx):
    wl = synth.mid()
    idx = synth.sample_blocks(wl.num_blocks(), 256, seed=5)
    W, c = wl.weights()[idx], wl.codebook()
    T = 1e-4
    got = parity.gpu_forward_backward(ctx, W, c, None, wl.Lb, wl.k, T)
    ref = oracle.soft_quantize(W, c, wl.Lb, wl.k, T)
    assert parity.rel_inf(got["soft"], ref["soft"]) <= parity.SOFT_TOL
    conv = _cold_limit_statistics(got["soft"], ref["soft"], W, c, wl.Lb, wl.k, T, "mid trellis")
    assert conv.mean() > 0.5                       # at T = 1e-4 most blocks have a clear winner
    vit = oracle.viterbi(W, c, wl.Lb, wl.k)
    gvit = parity.gpu_viterbi(ctx, W, c, wl.Lb, wl.k)
    parity.assert_viterbi(gvit, vit, "mid viterbi")


# ------------------------------------------------------------------ S = 2^16
@pytest.mark.parametrize("variant", ["tmem", "tmem_fused", "tmem_one_barrier", "cluster_registers", "generic"])
def test_q_proj_shape_sampled_blocks(ctx, variant):
    # the same sampled blocks through every implementation of the 2^16-state path
    wl = synth.q_proj()
    idx = synth.sample_blocks(wl.num_blocks(), 6 if variant != "generic" else 3)
    W, c, g = wl.weights()[idx], wl.codebook(), wl.upstream()[idx]
    opts = {"tmem": dict(path=0, fwd_variant=0, bwd_variant=0),
            "tmem_fused": dict(path=0, fwd_variant=0, bwd_variant=3),
            "tmem_one_barrier": dict(path=0, fwd_variant=0, bwd_variant=2),
            "cluster_registers": dict(path=2, fwd_variant=1, bwd_variant=1),
            "generic": dict(path=1, fwd_variant=0, bwd_variant=0)}[variant]
    try:
        for k_, v_ in opts.items():
            ctx.set_option(k_, v_)
        got = _check_all(ctx, W, c, g, wl.Lb, wl.k, wl.T, f"q_proj sample [{variant}]", viterbi=(variant == "tmem"))
        assert got["diag"].last_path == (0 if variant == "generic" else 1)
    finally:
        for k_ in opts:
            ctx.set_option(k_, 0)


@pytest.fixture(scope="module")
def decoder_sample():
    # four blocks (first, last, two seeded) from each of the seven matrices of the decoder-layer workload
    wl = synth.decoder_layer()
    Ws = []
    for i in range(len(wl.matrices)):
        Wm = wl.weights(i)
        Ws.append(Wm[synth.sample_blocks(Wm.shape[0], 4, seed=40 + i)])
    W = np.ascontiguousarray(np.concatenate(Ws))
    g = np.random.default_rng(4242).standard_normal(W.shape).astype(np.float32)
    return wl, W, wl.codebook(), g


@pytest.mark.parametrize("T", [0.3, 0.03, 0.01])
def test_decoder_layer_temperature_range_sampled_blocks(ctx, decoder_sample, T):
    # the annealing range of the decoder-layer workload (0.3 -> 0.01) on its kernels
    wl, W, c, g = decoder_sample
    assert W.shape[0] == 28
    got = _check_all(ctx, W, c, g, wl.Lb, wl.k, T, f"decoder layer sample, T={T}", viterbi=False)
    assert got["diag"].last_path == 1


@pytest.mark.parametrize("k", [2, 3])
def test_large_trellis_viterbi_full_length_many_blocks(ctx, k):
    # 256 blocks of 256 weights: near-ties between paths are what a wrong metric precision or
    # operation order would flip, and they only show in a sample of this size
    wl = synth.q_proj() if k == 2 else synth.gate_k3()
    idx = synth.sample_blocks(wl.num_blocks(), 256, seed=60 + k)
    W, c = wl.weights()[idx], wl.codebook()
    ref = oracle.viterbi(W, c, wl.Lb, k)
    got = parity.gpu_viterbi(ctx, W, c, wl.Lb, k)
    parity.assert_viterbi(got, ref, f"viterbi 256 blocks k={k}")


@pytest.mark.parametrize("n,B", [(1, 3), (2, 2), (3, 1), (7, 5), (64, 2), (255, 1), (15, 151)])
@pytest.mark.parametrize("variant", ["tmem", "tmem_fused", "cluster_registers"])
def test_large_trellis_ragged_lengths_and_block_counts(ctx, variant, n, B):
    # odd and tiny n exercise the buffer-parity and history-ring bookkeeping of the 2^16-state
    # kernels; B below the number of resident clusters leaves most of the grid without work
    Lb, k, T = 16, 2, 0.2
    W, c, g = _rand(n, Lb, B, seed=4000 + n)
    opts = dict(path=2, fwd_variant=int(variant == "cluster_registers"),
                bwd_variant={"tmem": 0, "tmem_fused": 3, "cluster_registers": 1}[variant])
    if B > 100 and variant != "tmem":
        pytest.skip("the many-block case is about the two-kernel backward call (more blocks than one chunk)")
    try:
        for k_, v_ in opts.items():
            ctx.set_option(k_, v_)
        got = _check_all(ctx, W, c, g, Lb, k, T, f"Lb=16 n={n} B={B} [{variant}]", viterbi=(variant == "tmem"))
        assert got["diag"].last_path == 1 and got["diag"].device_status == 0
    finally:
        for k_ in opts:
            ctx.set_option(k_, 0)


@pytest.mark.parametrize("k,n", [(2, 12), (3, 17)])
def test_large_trellis_viterbi_many_blocks_per_cta(ctx, k, n):
    # more blocks than thread blocks: every CTA runs several blocks, alternating its two
    # backpointer buffers while the trace warp lags one block behind the dynamic programme
    # (n = 17 at k = 3 takes the metric addresses once round their 13-step rotation period)
    Lb = 16
    W, c, _ = _rand(n, Lb, 450, seed=4200 + k)
    ref = oracle.viterbi(W, c, Lb, k)
    got = parity.gpu_viterbi(ctx, W, c, Lb, k)
    parity.assert_viterbi(got, ref, "viterbi 450 blocks")
    ctx.set_option("max_ctas", 3)
    try:
        parity.assert_viterbi(parity.gpu_viterbi(ctx, W[:40], c, Lb, k), oracle.viterbi(W[:40], c, Lb, k), "3 CTAs")
    finally:
        ctx.set_option("max_ctas", 0)
    ctx.set_option("path", GENERIC)
    try:
        parity.assert_viterbi(parity.gpu_viterbi(ctx, W[:6], c, Lb, k), oracle.viterbi(W[:6], c, Lb, k), "generic")
    finally:
        ctx.set_option("path", 0)


def test_large_trellis_long_blocks_fall_back_cleanly(ctx):
    # n = 1100 exceeds the backward TMEM kernel's step table (1024): it must take the next kernel
    # that covers the shape and still match; n = 2100 exceeds every large-trellis kernel
    Lb, k, T = 16, 2, 0.3
    for n in (1100, 2100):
        W, c, g = _rand(n, Lb, 1, seed=4100 + n)
        got = _check_all(ctx, W, c, g, Lb, k, T, f"Lb=16 n={n}", viterbi=False)
        assert got["diag"].device_status == 0


def test_non_finite_input_is_reported_not_fatal(ctx):
    # a NaN weight poisons its own block only; the call completes, the status says so, and the
    # context keeps working
    import torch
    from paper_2605_10655_b200 import BcjrError
    for Lb, n in ((8, 16), (16, 8)):
        W, c, g = _rand(n, Lb, 3, seed=77)
        W[1, n // 2] = np.nan
        dev = torch.device("cuda", 0)
        Wd, cd = torch.from_numpy(W).to(dev), torch.from_numpy(c).to(dev)
        soft, _ = ctx.bcjr_soft_quantize(Wd, cd, Lb, 2, n, 0.5)
        with pytest.raises(BcjrError) as ei:
            ctx.sync_status()
        assert ei.value.code == -7
        soft = soft.cpu().numpy()
        ref = oracle.soft_quantize(W[[0, 2]], c, Lb, 2, 0.5)["soft"]
        assert parity.rel_inf(soft[[0, 2]], ref) <= parity.SOFT_TOL       # the other blocks are intact
        assert ctx.sync_status().device_status == 0                          # cleared by the query


def test_device_wait_that_runs_out_is_reported_and_survivable(ctx):
    # No GPU fault is provoked: a history chunk is simply never requested, the consumer's bounded
    # wait gives up after its (shortened) budget, the kernel runs to its end and the host reads
    # BCJR_ETIMEOUT.  Afterwards the same context computes correct results again.
    from paper_2605_10655_b200 import BcjrError
    Lb, k, n, T = 16, 2, 6, 0.3
    W, c, g = _rand(n, Lb, 2, seed=4400)
    ref = oracle.soft_quantize(W, c, Lb, k, T)
    try:
        ctx.set_option("wait_limit_ms", 20)
        ctx.set_option("debug_drop_history_load", 1)
        with pytest.raises(BcjrError) as ei:
            parity.gpu_forward_backward(ctx, W, c, g, Lb, k, T)
        assert ei.value.code == -6
    finally:
        ctx.set_option("debug_drop_history_load", 0)
        ctx.set_option("wait_limit_ms", 2000)
    got = parity.gpu_forward_backward(ctx, W, c, g, Lb, k, T)
    assert got["diag"].device_status == 0
    assert parity.rel_inf(got["soft"], ref["soft"]) <= parity.SOFT_TOL


@pytest.mark.parametrize("Lb,k,n,B,T", [(8, 2, 64, 16, 0.5), (16, 2, 48, 3, 0.1), (16, 3, 40, 2, 0.05)])
def test_ste_forward_emits_hard_codeword_and_keeps_the_soft_gradient(ctx, Lb, k, n, B, T):
    # BCJR-STE: hard Viterbi codeword forward, gradient of the temperature-T relaxation backward
    import torch
    W, c, g = _rand(n, Lb, B, seed=5100 + Lb + k)
    dev = torch.device("cuda", ctx.device)
    Wd, cd, gd = (torch.from_numpy(a).to(dev) for a in (W, c, g))
    hard, states, soft = ctx.bcjr_ste_forward(Wd, cd, Lb, k, n, T, want_states=True, want_soft=True)
    gW, gc = ctx.bcjr_backward(gd)
    assert ctx.sync_status().device_status == 0
    ref_v = oracle.viterbi(W, c, Lb, k)
    np.testing.assert_array_equal(hard.cpu().numpy().view(np.uint32), ref_v["hard"].view(np.uint32))
    np.testing.assert_array_equal(states.cpu().numpy().view(np.uint16), ref_v["states"])
    ref_f, ref_b = oracle.soft_quantize(W, c, Lb, k, T), oracle.backward(W, c, g, Lb, k, T)
    assert parity.rel_inf(soft.cpu().numpy(), ref_f["soft"]) <= parity.SOFT_TOL
    assert parity.rel_inf(gW.cpu().numpy(), ref_b["grad_W"]) <= parity.GRAD_TOL
    assert parity.rel_inf(gc.cpu().numpy(), ref_b["grad_codebook"]) <= parity.GRAD_TOL
    # without the optional outputs the saved state is the same
    hard2, _, _ = ctx.bcjr_ste_forward(Wd, cd, Lb, k, n, T)
    gW2, gc2 = ctx.bcjr_backward(gd)
    ctx.sync_status()
    assert torch.equal(hard, hard2) and torch.equal(gW, gW2) and torch.equal(gc, gc2)


@pytest.mark.parametrize("k,n,B,m", [(2, 256, 5, 2), (2, 256, 5, 4), (2, 37, 3, 3), (2, 5, 2, 16), (2, 1, 2, 2), (2, 150, 151, 8),
                                     (2, 512, 1, 4), (3, 40, 3, 4)])
def test_checkpointed_history_matches_the_oracle(ctx, k, n, B, m):
    # history_every_m: the forward messages are kept for every m-th step and recomputed in between; the
    # soft codeword, log Z and (through the saved soft codeword) the gradients must not change
    Lb, T = 16, 0.1
    W, c, g = _rand(n, Lb, B, seed=4500 + 10 * k + m)
    ctx.set_option("history_every_m", m)
    try:
        got = _check_all(ctx, W, c, g, Lb, k, T, f"history_every_m={m} k={k} n={n}", viterbi=False)
        assert got["diag"].last_path == 1 and got["diag"].device_status == 0
    finally:
        ctx.set_option("history_every_m", 1)
    plain = parity.gpu_forward_backward(ctx, W, c, g, Lb, k, T)
    assert parity.rel_inf(got["soft"], plain["soft"]) <= 1e-5


@pytest.mark.parametrize("Lb,k,n,B", [(16, 2, 64, 5), (16, 3, 40, 3), (16, 2, 1100, 1), (8, 2, 64, 9), (12, 3, 30, 4), (12, 2, 30, 21)])
def test_computed_gaussian_emission(ctx, Lb, k, n, B):
    """codebook = NULL: the emission of Section 3.1, c(s) = Phi^-1((s + 1/2) / S), evaluated by the kernels
    themselves (2^16 states) or read from a table the context writes (other shapes).  For the soft codeword, log Z
    and the gradient the oracle is fed its own table (the inverse normal CDF in double, rounded to float32); an entry
    may differ from the device's by an ulp, far inside the tolerances.  Path bits are compared exactly, and an ulp can
    flip a near-tie, so for Viterbi alone the oracle decodes with the table bcjr_gaussian_codebook writes (the same
    device routine the kernels evaluate; the QAT tests compare it with the inverse normal CDF)."""
    import torch
    from paper_2605_10655_b200 import BcjrError
    T = 0.1
    rng = np.random.default_rng(4700 + Lb + k)
    W = rng.standard_normal((B, n)).astype(np.float32)
    g = rng.standard_normal((B, n)).astype(np.float32)
    dev = torch.device("cuda", ctx.device)
    c = qo.gaussian_codebook(Lb).astype(np.float32)
    c_dev = ctx.bcjr_gaussian_codebook(Lb).cpu().numpy()
    Wd, gd = torch.from_numpy(W).to(dev), torch.from_numpy(g).to(dev)
    soft, logZ = ctx.bcjr_soft_quantize(Wd, None, Lb, k, n, T)
    gW, none = ctx.bcjr_backward(gd)
    assert none is None
    bits, states, hard = ctx.viterbi_hard(Wd, None, Lb, k, n)
    assert ctx.sync_status().device_status == 0
    ref_f, ref_b, ref_v = oracle.soft_quantize(W, c, Lb, k, T), oracle.backward(W, c, g, Lb, k, T), oracle.viterbi(W, c_dev, Lb, k)
    assert parity.rel_inf(soft.cpu().numpy(), ref_f["soft"]) <= parity.SOFT_TOL
    np.testing.assert_allclose(logZ.cpu().numpy(), ref_f["logZ"], rtol=1e-5, atol=1e-3)
    assert parity.rel_inf(gW.cpu().numpy(), ref_b["grad_W"]) <= parity.GRAD_TOL
    parity.assert_viterbi({"path_bits": bits.cpu().numpy(), "states": states.cpu().numpy().view(np.uint16),
                           "hard": hard.cpu().numpy()}, ref_v, "computed emission")
    # a computed emission has no table to differentiate
    ctx.bcjr_soft_quantize(Wd, None, Lb, k, n, T)
    rc = ctx._lib.bcjr_backward(ctx._h, gd.data_ptr(), gW.data_ptr(), gW.data_ptr(), None)   # noqa
    assert rc == -1


@pytest.mark.parametrize("variant,max_ctas", [(0, 0), (0, 2), (4, 0), (3, 0)],
                         ids=["one_cta", "one_cta_several_blocks_each", "two_kernels", "fused_cluster"])
def test_backward_without_codebook_gradient(ctx, variant, max_ctas):
    # grad_codebook = NULL: the table is fixed (as in the paper's experiments) and only grad_W is formed.  At 2^16
    # states and k = 2 the call then runs both sweeps on one CTA per block (messages in place in both sweeps); the
    # cluster kernels without their accumulator half stay selectable.  grad_W must be the same either way.
    import torch
    wl = synth.q_proj()
    idx = synth.sample_blocks(wl.num_blocks(), 5, seed=17)
    W, c, g = wl.weights()[idx], wl.codebook(), wl.upstream()[idx]
    W = W.copy()
    W[3, 40] = 7.5                                            # one block outside the table's range: re-centred energies
    dev = torch.device("cuda", ctx.device)
    Wd, cd, gd = (torch.from_numpy(np.ascontiguousarray(a)).to(dev) for a in (W, c, g))
    ctx.set_option("bwd_variant", variant)
    ctx.set_option("max_ctas", max_ctas)
    try:
        for (Lb, k, Wd_, cd_, gd_) in ((wl.Lb, wl.k, Wd, cd, gd), (8, 2, Wd[:, :64].contiguous(), cd[:256].contiguous(), gd[:, :64].contiguous())):
            n = Wd_.shape[1]
            ctx.bcjr_soft_quantize(Wd_, cd_, Lb, k, n, wl.T)
            gW_full, gc = ctx.bcjr_backward(gd_)
            ctx.bcjr_soft_quantize(Wd_, cd_, Lb, k, n, wl.T)
            gW_only, none = ctx.bcjr_backward(gd_, want_grad_codebook=False)
            st = ctx.sync_status()
            assert st.device_status == 0 and none is None and st.max_posterior_defect < 1e-3
            ref = oracle.backward(Wd_.cpu().numpy(), cd_.cpu().numpy(), gd_.cpu().numpy(), Lb, k, wl.T)
            assert parity.rel_inf(gW_only.cpu().numpy(), ref["grad_W"]) <= parity.GRAD_TOL
            assert parity.rel_inf(gW_full.cpu().numpy(), ref["grad_W"]) <= parity.GRAD_TOL
            assert parity.rel_inf(gW_only.cpu().numpy(), gW_full.cpu().numpy()) <= 2e-5   # two kernels, two summation orders
    finally:
        ctx.set_option("bwd_variant", 0)
        ctx.set_option("max_ctas", 0)


def test_backward_without_codebook_gradient_three_bits(ctx):
    # k = 3 has no accumulator-free kernel: the call runs the two-kernel path and drops the partial sums
    import torch
    W, c, g = _rand(40, 16, 3, seed=77, student=True)
    dev = torch.device("cuda", ctx.device)
    Wd, cd, gd = (torch.from_numpy(a).to(dev) for a in (W, c, g))
    ctx.bcjr_soft_quantize(Wd, cd, 16, 3, 40, 0.1)
    gW, none = ctx.bcjr_backward(gd, want_grad_codebook=False)
    assert ctx.sync_status().device_status == 0 and none is None
    ref = oracle.backward(W, c, g, 16, 3, 0.1)
    assert parity.rel_inf(gW.cpu().numpy(), ref["grad_W"]) <= parity.GRAD_TOL
    ctx.bcjr_soft_quantize(Wd, None, 16, 3, 40, 0.1)                   # computed emission: no table to differentiate
    gW2, none = ctx.bcjr_backward(gd, want_grad_codebook=False)
    ref2 = oracle.backward(W, qo.gaussian_codebook(16).astype(np.float32), g, 16, 3, 0.1)
    assert ctx.sync_status().device_status == 0
    assert parity.rel_inf(gW2.cpu().numpy(), ref2["grad_W"]) <= parity.GRAD_TOL


@pytest.mark.parametrize("n,T", [(1, 0.3), (2, 0.3), (37, 0.05), (256, 0.02)])
def test_one_cta_backward_lengths_and_temperatures(ctx, n, T):
    # the one-CTA backward call at the block lengths where its history ring and slot rotation wrap differently
    # (n = 1, 2: fewer steps than the ring is deep; 37: not a multiple of the 7 rotations), and at a cold T
    import torch
    W, c, g = _rand(n, 16, 3, seed=300 + n)
    dev = torch.device("cuda", ctx.device)
    Wd, cd, gd = (torch.from_numpy(a).to(dev) for a in (W, c, g))
    ctx.bcjr_soft_quantize(Wd, cd, 16, 2, n, T)
    gW, none = ctx.bcjr_backward(gd, want_grad_codebook=False)
    st = ctx.sync_status()
    assert st.device_status == 0 and st.max_posterior_defect < 1e-3
    ref = oracle.backward(W, c, g, 16, 2, T)
    assert parity.rel_inf(gW.cpu().numpy(), ref["grad_W"]) <= parity.GRAD_TOL


def test_results_do_not_depend_on_what_ran_before(ctx):
    # scratch (history, partial sums, tensor memory) is reused between calls and between
    # blocks: the same input must give bit-identical output regardless of the previous call
    wl = synth.q_proj()
    W, c, g = wl.weights()[:5], wl.codebook(), wl.upstream()[:5]
    first = parity.gpu_forward_backward(ctx, W, c, g, wl.Lb, wl.k, wl.T)
    other = _rand(33, 16, 3, seed=9)
    parity.gpu_forward_backward(ctx, other[0], other[1], other[2], 16, 2, 0.7)
    again = parity.gpu_forward_backward(ctx, W, c, g, wl.Lb, wl.k, wl.T)
    for key in ("soft", "logZ", "grad_W", "grad_codebook"):
        np.testing.assert_array_equal(first[key], again[key], err_msg=key)


def test_q_proj_full_size_sampled_outputs_and_invariants(ctx):
    """The full 2048 x 2048 matrix (16384 blocks) in the launch configuration the benchmark times.
    soft and grad_W of a block depend on that block alone, so sampled blocks are compared with
    the oracle one by one; grad_codebook sums over all blocks and is checked through the shift
    identity  sum grad_W + sum grad_codebook = sum g  (soft(w + a, c + a) = soft(w, c) + a)."""
    import torch
    wl = synth.q_proj()
    W, c, g = wl.weights(), wl.codebook(), wl.upstream()
    got = parity.gpu_forward_backward(ctx, W, c, g, wl.Lb, wl.k, wl.T)
    assert got["diag"].last_path == 1 and got["diag"].device_status == 0
    assert got["diag"].max_posterior_defect < 1e-3
    assert np.all(np.isfinite(got["soft"])) and np.all(np.isfinite(got["grad_W"]))
    idx = synth.sample_blocks(wl.num_blocks(), 64, seed=123)
    ref_f = oracle.soft_quantize(W[idx], c, wl.Lb, wl.k, wl.T)
    ref_b = oracle.backward(W[idx], c, g[idx], wl.Lb, wl.k, wl.T)
    assert parity.rel_inf(got["soft"][idx], ref_f["soft"]) <= parity.SOFT_TOL
    assert parity.rel_inf(got["grad_W"][idx], ref_b["grad_W"]) <= parity.GRAD_TOL
    np.testing.assert_allclose(got["logZ"][idx], ref_f["logZ"], rtol=1e-5, atol=1e-3)
    total = got["grad_W"].astype(np.float64).sum() + got["grad_codebook"].astype(np.float64).sum()
    gsum = g.astype(np.float64).sum()
    assert abs(total - gsum) <= 1e-3 * np.abs(g).astype(np.float64).sum() ** 0.5 * 10
    # the soft codeword is a convex combination of table entries
    assert got["soft"].min() >= c.min() - 1e-4 and got["soft"].max() <= c.max() + 1e-4


def test_three_bit_student_t_register_variant(ctx):
    wl = synth.gate_k3()
    idx = synth.sample_blocks(wl.num_blocks(), 4)
    W, c, g = wl.weights()[idx], wl.codebook(), wl.upstream()[idx]
    try:
        ctx.set_option("fwd_variant", 1); ctx.set_option("bwd_variant", 1)
        got = _check_all(ctx, W, c, g, wl.Lb, wl.k, 0.01, "k=3 student-t T=0.01 [cluster_registers]", viterbi=False)
    finally:
        ctx.set_option("fwd_variant", 0); ctx.set_option("bwd_variant", 0)
    assert got["diag"].last_path == 1


@pytest.mark.parametrize("T", [0.01, 0.001])
def test_three_bit_student_t_low_temperature(ctx, T):
    """592 blocks of the heavy-tailed 3-bit workload in one call, the posterior defect of every block recorded.
    Compared with the oracle: the sixteen blocks with the largest defect and sixteen seeded ones, taken from
    that call (soft, log Z, grad_W depend on their block alone); grad_codebook from a second call on those
    blocks only; Viterbi on them; the cold-limit statistics."""
    wl = synth.gate_k3()
    NB = 592
    W, c, g = wl.weights()[:NB], wl.codebook(), wl.upstream()[:NB]
    ctx.set_option("record_block_defect", 1)
    try:
        got = parity.gpu_forward_backward(ctx, W, c, g, wl.Lb, wl.k, T)
        defects = ctx.block_defects(NB)
    finally:
        ctx.set_option("record_block_defect", 0)
    assert got["diag"].last_path == 1 and got["diag"].device_status == 0
    assert np.all(np.isfinite(defects)) and np.all(np.isfinite(got["soft"])) and np.all(np.isfinite(got["grad_W"]))
    worst = np.argsort(defects)[::-1][:16]
    print(f"\nk=3 student-t T={T}: posterior defect max {defects.max():.2e} (block {int(defects.argmax())}, "
          f"max |w| there {np.abs(W[defects.argmax()]).max():.1f}), median {np.median(defects):.2e}; "
          f"largest |w| of the call {np.abs(W).max():.1f} (table range {c.min():.2f} .. {c.max():.2f})")
    assert defects.max() < 1e-3
    idx = np.array(sorted(set(worst.tolist()) | set(synth.sample_blocks(NB, 16, seed=7).tolist())), dtype=np.int64)
    ref_f = oracle.soft_quantize(W[idx], c, wl.Lb, wl.k, T)
    ref_b = oracle.backward(W[idx], c, g[idx], wl.Lb, wl.k, T)
    # block by block as well, so that a block with large values cannot hide one with small values.  The stated
    # metric is per output tensor; against the maximum of a single block's 256 values the same absolute error
    # reads larger, hence twice the tolerance here (the per-tensor comparison follows at the stated one)
    for j, b in enumerate(idx):
        assert parity.rel_inf(got["soft"][b], ref_f["soft"][j]) <= 2 * parity.SOFT_TOL, f"soft, block {b} (defect {defects[b]:.2e})"
        assert parity.rel_inf(got["grad_W"][b], ref_b["grad_W"][j]) <= 2 * parity.GRAD_TOL, f"grad_W, block {b}"
    assert parity.rel_inf(got["soft"][idx], ref_f["soft"]) <= parity.SOFT_TOL
    assert parity.rel_inf(got["grad_W"][idx], ref_b["grad_W"]) <= parity.GRAD_TOL
    np.testing.assert_allclose(got["logZ"][idx], ref_f["logZ"], rtol=1e-5, atol=1e-3)
    sub = parity.gpu_forward_backward(ctx, W[idx], c, g[idx], wl.Lb, wl.k, T)
    parity.assert_forward_backward(sub, ref_f, ref_b, f"k=3 student-t T={T}, sampled blocks")
    tot = got["grad_W"].astype(np.float64).sum() + got["grad_codebook"].astype(np.float64).sum()
    assert abs(tot - g.astype(np.float64).sum()) < 1e-2 * np.abs(g).sum()
    parity.assert_viterbi(parity.gpu_viterbi(ctx, W[idx], c, wl.Lb, wl.k), oracle.viterbi(W[idx], c, wl.Lb, wl.k), "k=3")
    _cold_limit_statistics(got["soft"][idx], ref_f["soft"], W[idx], c, wl.Lb, wl.k, T, "3-bit student-t")


@pytest.mark.parametrize("n,B", [(1, 2), (5, 3), (33, 1)])
def test_three_bit_ragged_lengths(ctx, n, B):
    Lb, k, T = 16, 3, 0.2
    W, c, g = _rand(n, Lb, B, seed=4300 + n)
    _check_all(ctx, W, c, g, Lb, k, T, f"Lb=16 k=3 n={n} B={B}", viterbi=(n == 5))

#!/usr/bin/env python
"""Benchmark of the BCJR hot path on B200.

    python bench.py [--gpus N] [--steps K] [--warmup W] [--workload NAME] [--impl reference]

One "step" is one QAT-style pass over the whole synthetic workload: bcjr_soft_quantize
(alpha + beta sweeps, soft codeword) followed by bcjr_backward (grad_W, grad_codebook) for
every weight matrix of the workload.  The metric is trellis-edge updates per second with
2 * blocks * n * S * K edges per step (one alpha and one beta sweep; the sweeps the backward
pass repeats are not counted as work).  viterbi_hard is timed in the same run and reported
beside it.  Prints ONE JSON line on rank 0.
"""
from __future__ import annotations

import argparse
import json
import os
import subprocess
import sys
import threading
import time
from pathlib import Path

import numpy as np

ROOT = Path(__file__).resolve().parent
sys.path.insert(0, str(ROOT))

from paper_2605_10655_b200 import shard, synth  # noqa: E402

METRIC = "bcjr_fwd_bwd_trellis_edge_updates_per_s"
UNIT = "edges/s"
WORKLOADS = {"tiny": synth.tiny, "mid": synth.mid, "q_proj": synth.q_proj, "layer": synth.decoder_layer,
             "gate_k3": synth.gate_k3, "qtip_v2": synth.qtip_v2}
# (Lb, k, kernel) -> measured DRAM bytes per weight block (n = 256), see profiles/*.md
NCU_DRAM_BYTES_PER_BLOCK = {(16, 2, "bwd"): 66.3e6, (16, 2, "fwd"): 33.1e6}
MUFU_PER_CLK_PER_SM = 16          # special-function results per clock per SM (CUDA throughput table, cc 10.0)
NUM_SMS = 148


def mufu_ops_per_state_step(k: int, kernel: str, V: int = 1, count: str = "algorithmic") -> float:
    """Special-function operations per state per step, K = 2^(kV) states per group.

    count="algorithmic": what the recursions need at the least -- one ex2 per state and one lg2 per group in
    every sweep, plus one ex2 per group for the posterior in a beta sweep; the backward call repeats both
    sweeps and reuses their exponentials for the gradient: forward 2 + 3/K, backward 2 + 3/K.
    count="with_rcp": what the backward kernels in this library issue -- the same plus one rcp per group and
    sweep (the conditional expectations carried next to the messages are normalised by the group sum)."""
    K = 1 << (k * V)
    fwd = (1 + 1 / K) + (1 + 2 / K)
    bwd = fwd if count == "algorithmic" else (1 + 2 / K) + (1 + 3 / K)
    return {"fwd": fwd, "bwd": bwd, "both": fwd + bwd}[kernel]


def anneal_schedule(T0: float, T_end: float, steps: int):
    """Geometric temperature schedule of Section 3.6, both end points hit."""
    return [T0] if steps == 1 else [T0 * (T_end / T0) ** (i / (steps - 1)) for i in range(steps)]


class ClockSampler:
    QUERY = ("index,clocks.sm,clocks.max.sm,power.draw,clocks_event_reasons.active,"
             "clocks_event_reasons.hw_slowdown,clocks_event_reasons.hw_thermal_slowdown,"
             "clocks_event_reasons.sw_thermal_slowdown,clocks_event_reasons.sw_power_cap")

    def __init__(self, gpu_index: int):
        self.gpu = gpu_index
        self.rows = []
        self.proc = None

    def start(self):
        try:
            self.proc = subprocess.Popen(["nvidia-smi", f"--id={self.gpu}", f"--query-gpu={self.QUERY}",
                                          "--format=csv,noheader,nounits", "-lms", "200"],
                                         stdout=subprocess.PIPE, stderr=subprocess.DEVNULL, text=True)
            self.thread = threading.Thread(target=self._read, daemon=True)
            self.thread.start()
        except OSError:
            self.proc = None

    def _read(self):
        for line in self.proc.stdout:
            self.rows.append((time.time(), [x.strip() for x in line.split(",")]))

    def stop(self, t0: float, t1: float):
        if self.proc is None:
            return {"sm_mhz": None, "sm_max_mhz": None, "reasons": ["nvidia-smi unavailable"]}
        time.sleep(0.25)
        self.proc.terminate()
        rows = [r for (ts, r) in self.rows if t0 <= ts <= t1 and len(r) >= 9] or [r for _, r in self.rows if len(r) >= 9]
        if not rows:
            return {"sm_mhz": None, "sm_max_mhz": None, "reasons": ["no samples"]}
        sm = sorted(float(r[1]) for r in rows)
        reasons = set()
        for r in rows:
            for name, col in (("hw_slowdown", 5), ("hw_thermal_slowdown", 6), ("sw_thermal_slowdown", 7),
                              ("sw_power_cap", 8)):
                if r[col].lower().startswith("active"):
                    reasons.add(name)
        return {"sm_mhz": sm[len(sm) // 2], "sm_max_mhz": float(rows[0][2]),
                "power_w_max": max(float(r[3]) for r in rows), "samples": len(rows), "reasons": sorted(reasons)}


def cpu_baseline(wl, blocks_per_core: int = 4):
    """The float64 oracle, as it stands, on the host cores: forward + backward of a bounded
    sample of blocks of the same workload (blocks_per_core blocks per core)."""
    import oracle
    cores = oracle.host_cores()
    # ~5 core-seconds per block at S = 2^16, n = 256 (forward + backward); four blocks per core
    # keep the sample near 20 s; smaller trellises take proportionally more blocks
    scale = max(1, int((1 << 16) * 256 / (wl.S * wl.n)))
    nblk = max(1, min(wl.num_blocks(), blocks_per_core * cores * min(scale, 64)))
    W, c, g = wl.weights(0)[:nblk], wl.codebook(), wl.upstream(0)[:nblk]
    t0 = time.time()
    if wl.V == 1:
        oracle.soft_quantize(W, c, wl.Lb, wl.k, wl.T)
        oracle.backward(W, c, g, wl.Lb, wl.k, wl.T)
    else:
        oracle.soft_quantize_vec(W, c, wl.Lb, wl.k * wl.V, wl.V, wl.T)
        oracle.backward_vec(W, c, g, wl.Lb, wl.k * wl.V, wl.V, wl.T)
    dt = time.time() - t0
    threads = oracle.num_threads()
    edges = 2 * nblk * wl.steps * wl.S * wl.K
    return {"value": edges / dt, "unit": UNIT, "cores": threads, "kind": "oracle",
            "sample": f"{nblk} blocks of {wl.name} (n={wl.n}, Lb={wl.Lb}, k={wl.k}, T={wl.T}), "
                      f"forward+backward, {dt:.1f} s"}, dt


def run_reference(args, wl):
    rank = int(os.environ.get("RANK", "0"))
    if rank != 0:
        return
    vals = []
    for _ in range(args.warmup):
        pass                                    # the oracle has no warm-up state
    base = None
    steps = max(1, args.steps)
    per_core = 4 if steps <= 6 else 2 if steps <= 12 else 1    # keeps the whole run near two minutes (~5 core-seconds per block)
    for _ in range(steps):
        base, dt = cpu_baseline(wl, per_core)
        vals.append((base["value"], dt))
    value = float(np.mean([v for v, _ in vals]))
    base["value"] = value
    out = {"impl": "reference", "metric": METRIC, "value": value, "unit": UNIT, "n_gpus": args.gpus,
           "steps": args.steps, "warmup": args.warmup, "ms_per_step": 1e3 * float(np.mean([d for _, d in vals])),
           "higher_is_better": True, "scaling": "weak", "vs_baseline": None, "dtype": "f64", "data": "synthetic",
           "config": {"workload": wl.name, "Lb": wl.Lb, "k": wl.k, "n": wl.n, "T": wl.T,
                      "note": "float64 CPU oracle on a bounded sample per step"},
           "cpu_baseline": base, "gpu_launches": 0,
           "e2e": {"value": value, "unit": UNIT, "h2d_bytes_per_step": 0, "d2h_bytes_per_step": 0}}
    print(json.dumps(out))


class Runner:
    """Device buffers of one workload and the timed forward + backward step over all its matrices."""

    def __init__(self, ctx, wl, dev, blocks_cap=0, rank=0, world=1, keep_host=False, fixed_table=False):
        import torch
        self.ctx, self.wl, self.dev, self.rank = ctx, wl, dev, rank
        self.fixed_table = fixed_table                      # backward without grad_codebook (the paper's setting: the table is not trained)
        self.cb = torch.from_numpy(wl.codebook()).to(dev)
        self.mats = []
        for i, (name, _) in enumerate(wl.matrices):
            W = wl.weights(i)
            if blocks_cap:
                W = W[:blocks_cap]
            W = np.ascontiguousarray(W)
            if world > 1:
                W = np.roll(W, rank, axis=0)
            m = {"name": name, "W": torch.from_numpy(W).to(dev)}
            if keep_host:
                m["W_host"] = torch.from_numpy(W).pin_memory()
            m["soft"] = torch.empty_like(m["W"]); m["gW"] = torch.empty_like(m["W"]); m["g"] = torch.empty_like(m["W"])
            self.mats.append(m)
        self.nblocks = sum(m["W"].shape[0] for m in self.mats)
        self.edges_per_step = 2 * self.nblocks * wl.steps * wl.S * wl.K
        self.state_steps = self.nblocks * wl.steps * wl.S
        self.gc = torch.empty(wl.S * wl.V, dtype=torch.float32, device=dev)
        self.gc_total = torch.zeros(wl.S * wl.V, dtype=torch.float32, device=dev)
        self.gen = torch.Generator(device=dev)

    def fresh_g(self, step):
        for i, m in enumerate(self.mats):
            self.gen.manual_seed(self.wl.g_seed + 7919 * step + i + 104729 * self.rank)
            m["g"].normal_(generator=self.gen)

    def step(self, T, ev=None):
        import torch
        wl, ctx = self.wl, self.ctx
        self.gc_total.zero_()
        for m in self.mats:
            if ev is not None:
                ev["f0"].append(torch.cuda.Event(enable_timing=True)); ev["f0"][-1].record()
            if wl.V == 1:
                ctx.bcjr_soft_quantize(m["W"], self.cb, wl.Lb, wl.k, wl.n, T, soft=m["soft"])
            else:
                ctx.bcjr_soft_quantize_vec(m["W"], self.cb, wl.Lb, wl.k, wl.V, wl.n, T, soft=m["soft"])
            if ev is not None:
                ev["f1"].append(torch.cuda.Event(enable_timing=True)); ev["f1"][-1].record()
            if self.fixed_table:
                ctx.bcjr_backward(m["g"], grad_W=m["gW"], want_grad_codebook=False)
            else:
                ctx.bcjr_backward(m["g"], grad_W=m["gW"], grad_codebook=self.gc)
            if ev is not None:
                ev["b1"].append(torch.cuda.Event(enable_timing=True)); ev["b1"][-1].record()
            if not self.fixed_table:
                self.gc_total.add_(self.gc)
        if not self.fixed_table:
            shard.allreduce_grad_codebook(self.gc_total)     # the one exchange of the data-parallel path

    def timed(self, temps_warm, temps_timed, flush):
        """Warm-up steps, then the timed ones (CUDA events per step on the launching stream, L2 evicted in
        between).  Returns per-step ms, summed forward / backward ms and the launch count."""
        import torch
        for s, T in enumerate(temps_warm):
            self.fresh_g(s); flush.zero_()
            self.step(T)
        d0 = self.ctx.sync_status()
        evs = []
        for s, T in enumerate(temps_timed):
            self.fresh_g(len(temps_warm) + s)
            flush.zero_()                                   # evict L2 between timed steps (not timed)
            e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
            ev = {"f0": [], "f1": [], "b1": []}
            e0.record()
            self.step(T, ev)
            e1.record()
            evs.append((e0, e1, ev))
        torch.cuda.synchronize()
        step_ms = [e0.elapsed_time(e1) for e0, e1, _ in evs]
        fwd_ms = sum(a.elapsed_time(b) for _, _, ev in evs for a, b in zip(ev["f0"], ev["f1"]))
        bwd_ms = sum(a.elapsed_time(b) for _, _, ev in evs for a, b in zip(ev["f1"], ev["b1"]))
        diag = self.ctx.sync_status()
        return step_ms, fwd_ms, bwd_ms, diag, diag.kernel_launches - d0.kernel_launches


def mufu_fractions(wl, state_steps, fwd_ms, bwd_ms, step_ms, peak_gops):
    """Fractions of the special-function peak, on both operation counts (see mufu_ops_per_state_step)."""
    out = {}
    for count, tag in (("algorithmic", "frac"), ("with_rcp", "frac_with_rcp")):
        for kern, ms in (("fwd", fwd_ms), ("bwd", bwd_ms), ("both", step_ms)):
            ops = mufu_ops_per_state_step(wl.k, kern, wl.V, count) * state_steps
            out[f"{kern}_{tag}"] = ops / (ms * 1e-3) / 1e9 / peak_gops
    return out


def workload_leg(ctx, name, blocks_cap, dev, flush, peak_gops, fixed_table=False):
    """A short measurement of another workload in the same run: one warm-up step, two timed steps."""
    import torch
    wl = WORKLOADS[name]()
    r = Runner(ctx, wl, dev, blocks_cap, fixed_table=fixed_table)
    step_ms, fwd_ms, bwd_ms, diag, _ = r.timed([wl.T], [wl.T, wl.T], flush)
    ms = float(np.mean(step_ms))
    leg = {"workload": wl.name, "blocks": r.nblocks, "Lb": wl.Lb, "k": wl.k, "V": wl.V, "n": wl.n, "T": wl.T,
           "ms_per_step": ms, "fwd_ms": fwd_ms / 2, "bwd_ms": bwd_ms / 2, "edges_per_s": r.edges_per_step / (ms * 1e-3),
           "path": {0: "generic kernels", 1: "large-trellis kernels", 2: "one warp per block"}[diag.last_path],
           "max_posterior_defect": diag.max_posterior_defect}
    if fixed_table:
        leg["backward"] = "grad_W only (table not trained)"
    leg.update(mufu_fractions(wl, r.state_steps, fwd_ms / 2, bwd_ms / 2, ms, peak_gops))
    del r
    torch.cuda.empty_cache()
    return leg


def qat_loop_leg(ctx, dev, flush, steps=4):
    """Algorithm 1 around the path, timed as a loop: at each step the forward call, a stand-in loss on the soft
    codeword (mean squared distance to the initial weights: the layer-output loss of the paper needs a model and
    calibration activations), then bcjr_backward_adam, which updates the latent weights and the table in
    place.  q_proj-shaped matrix, T annealed 0.3 -> 0.01 over the steps."""
    import torch
    wl = WORKLOADS["q_proj"]()
    W = torch.from_numpy(np.ascontiguousarray(wl.weights(0))).to(dev)
    target = W.clone()
    cb = torch.from_numpy(wl.codebook()).to(dev)
    mW, vW, mc, vc = torch.zeros_like(W), torch.zeros_like(W), torch.zeros_like(cb), torch.zeros_like(cb)
    soft = torch.empty_like(W)
    temps = anneal_schedule(0.3, 0.01, steps)
    losses, ms = [], []
    for t in range(steps + 1):                                  # the first pass is the warm-up
        T = temps[max(t - 1, 0)]
        flush.zero_()
        e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
        e0.record()
        ctx.bcjr_soft_quantize(W, cb, wl.Lb, wl.k, wl.n, T, soft=soft)
        diff = soft - target
        loss = (diff * diff).mean()
        g = diff * (2.0 / diff.numel())
        ctx.bcjr_backward_adam(g, mW, vW, t + 1, 1e-3, m_c=mc, v_c=vc, lr_c=1e-4)
        e1.record()
        torch.cuda.synchronize()
        if t > 0:
            ms.append(e0.elapsed_time(e1)); losses.append(float(loss))
    nb = W.shape[0]
    return {"workload": wl.name, "blocks": nb, "steps": steps, "T": [temps[0], temps[-1]], "ms_per_step": float(np.mean(ms)),
            "edges_per_s": 2 * nb * wl.steps * wl.S * wl.K / (float(np.mean(ms)) * 1e-3),
            "stand_in_loss_per_step": losses, "note": "T falls from step to step, so the losses of different steps are not comparable",
            "updates": "latent weights and codebook table, Adam, inside bcjr_backward_adam"}


def main():
    ap = argparse.ArgumentParser()
    ap.add_argument("--gpus", type=int, default=1)
    ap.add_argument("--steps", type=int, default=3)
    ap.add_argument("--warmup", type=int, default=3)
    ap.add_argument("--workload", default="layer", choices=sorted(WORKLOADS))
    ap.add_argument("--impl", default="b200", choices=["b200", "reference"])
    ap.add_argument("--blocks", type=int, default=0, help="cap on blocks per matrix (0 = all); for profiling")
    ap.add_argument("--path", type=int, default=0, help="0 auto, 1 generic kernels, 2 cluster kernels")
    ap.add_argument("--fwd-variant", type=int, default=0)
    ap.add_argument("--bwd-variant", type=int, default=0)
    ap.add_argument("--option", action="append", default=[], metavar="NAME=VALUE", help="bcjr_set_option passthrough")
    ap.add_argument("--no-cpu-baseline", action="store_true")
    ap.add_argument("--no-e2e", action="store_true")
    ap.add_argument("--no-viterbi", action="store_true")
    ap.add_argument("--no-legs", action="store_true", help="skip the short legs over the other workloads")
    ap.add_argument("--fixed-table", action="store_true",
                    help="backward calls without grad_codebook (not the headline configuration, which trains the table)")
    args = ap.parse_args()
    if args.fixed_table:
        args.no_e2e = True                                  # the host-buffer call always forms grad_codebook
    wl = WORKLOADS[args.workload]()
    if args.impl == "reference":
        return run_reference(args, wl)

    import torch
    import torch.distributed as dist
    from paper_2605_10655_b200 import Context, binding

    rank = int(os.environ.get("RANK", "0"))
    world = int(os.environ.get("WORLD_SIZE", "1"))
    local = int(os.environ.get("LOCAL_RANK", "0"))
    torch.cuda.set_device(local)
    dev = torch.device("cuda", local)
    if world > 1:
        os.environ.setdefault("MASTER_ADDR", "127.0.0.1")
        dist.init_process_group("nccl", device_id=dev)

    def barrier():
        if world > 1:
            dist.barrier()
        torch.cuda.synchronize()

    # ---- pipe rates of this GPU, measured now (the roofline's denominator)
    peaks = binding.measure_pipe_peaks(local)

    # Every rank processes the whole workload shape on its own seeded data (weak scaling over
    # independent blocks); the only exchange is the all-reduce of grad_codebook.
    ctx = Context(local)
    if args.path:
        ctx.set_option("path", args.path)
    if args.fwd_variant:
        ctx.set_option("fwd_variant", args.fwd_variant)
    if args.bwd_variant:
        ctx.set_option("bwd_variant", args.bwd_variant)
    for kv in args.option:
        name, _, val = kv.partition("=")
        ctx.set_option(name, int(val))
    run = Runner(ctx, wl, dev, args.blocks, rank, world, keep_host=not args.no_e2e, fixed_table=args.fixed_table)
    mats, cb, nblocks, edges_per_step = run.mats, run.cb, run.nblocks, run.edges_per_step
    # the decoder-layer workload anneals T geometrically from 0.3 to 0.01 over the timed steps (warm-up at T_0)
    annealed = wl.name.startswith("llama32_1b_decoder")
    temps_timed = anneal_schedule(0.3, 0.01, args.steps) if annealed else [wl.T] * args.steps
    temps_warm = [temps_timed[0]] * args.warmup
    flush = torch.empty(256 << 20, dtype=torch.uint8, device=dev)      # > L2 (126 MB)

    sampler = ClockSampler(local)
    barrier()
    sampler.start()
    t_wall0 = time.time()
    step_ms, fwd_ms, bwd_ms, diag, launches = run.timed(temps_warm, temps_timed, flush)
    barrier()
    t_wall1 = time.time()
    clocks = sampler.stop(t_wall0, t_wall1)
    total_ms = float(sum(step_ms))
    t = torch.tensor([total_ms], dtype=torch.float64, device=dev)
    if world > 1:
        dist.all_reduce(t, op=dist.ReduceOp.MAX)
    total_ms = float(t.item())
    ms_per_step = total_ms / args.steps
    value = edges_per_step * world / (ms_per_step * 1e-3)

    # ---- Viterbi leg (same workload, same run)
    vit = None
    if not args.no_viterbi:
        def vit_call(Wd):
            if wl.V == 1:
                ctx.viterbi_hard(Wd, cb, wl.Lb, wl.k, wl.n)
            else:
                ctx.viterbi_hard_vec(Wd, cb, wl.Lb, wl.k, wl.V, wl.n)
        vit_call(mats[0]["W"])                                      # warm-up
        torch.cuda.synchronize()
        e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
        flush.zero_()
        e0.record()
        for m in mats:
            vit_call(m["W"])
        e1.record()
        torch.cuda.synchronize()
        vms = e0.elapsed_time(e1)
        vit = {"ms": vms, "edges_per_s": nblocks * wl.steps * wl.S * wl.K / (vms * 1e-3)}

    # ---- the Adam update that follows the backward pass in the QAT loop (HBM-bound: 28 bytes per weight)
    upd = None
    if not args.no_viterbi:
        big = max(mats, key=lambda m: m["W"].numel())
        numel = big["W"].numel()
        mW = torch.zeros_like(big["W"]); vW = torch.zeros_like(big["W"]); Wc = big["W"].clone()
        ctx.bcjr_adam_update(Wc, big["gW"], mW, vW, 1, 1e-4)       # warm-up
        flush.zero_()
        e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
        e0.record()
        ctx.bcjr_adam_update(Wc, big["gW"], mW, vW, 2, 1e-4)
        e1.record()
        torch.cuda.synchronize()
        ums = e0.elapsed_time(e1)
        upd = {"kernel": "adam_kernel", "weights": numel, "ms": ums, "gbs": 28.0 * numel / (ums * 1e-3) / 1e9}
        del mW, vW, Wc
        # the incoherence rotation that precedes the trellis pass (both sides; algorithmic bytes: read + write once)
        rows, cols = dict(wl.matrices)[big["name"]]
        if not args.blocks and rows & (rows - 1) == 0 and cols & (cols - 1) == 0 and cols <= 8192:
            W2 = big["W"].reshape(rows, cols).clone()
            sL = torch.ones(rows, device=dev); sR = torch.ones(cols, device=dev)
            out2 = torch.empty_like(W2)
            ctx.bcjr_rht(W2, sL, sR, out=out2)                         # warm-up
            flush.zero_()
            e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
            e0.record()
            ctx.bcjr_rht(W2, sL, sR, out=out2)
            e1.record()
            torch.cuda.synchronize()
            rms = e0.elapsed_time(e1)
            upd["rht"] = {"shape": [rows, cols], "ms": rms, "gbs": 8.0 * rows * cols / (rms * 1e-3) / 1e9}
            del W2, out2

    # ---- end to end through the host-buffer entry point (pinned host memory both ways), same schedule
    e2e = None
    if not args.no_e2e and wl.V == 1:          # the host-buffer entry point covers the scalar trellis
        host = []
        for m in mats:
            host.append({"W": m["W_host"], "g": m["g"].cpu().pin_memory(),
                         "soft": torch.empty_like(m["W_host"]).pin_memory(),
                         "gW": torch.empty_like(m["W_host"]).pin_memory()})
        cb_h = cb.cpu().pin_memory(); gc_h = torch.empty(wl.S).pin_memory()

        def e2e_step(T_e):
            for h in host:
                ctx.bcjr_step_host(h["W"], cb_h, h["g"], wl.Lb, wl.k, wl.n, T_e, soft=h["soft"], grad_W=h["gW"],
                                   grad_codebook=gc_h)
        e2e_step(temps_timed[0])                                    # warm-up (allocates staging buffers)
        barrier()
        e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
        e0.record()
        for T_e in temps_timed:
            e2e_step(T_e)
        e1.record()
        barrier()
        ems = e0.elapsed_time(e1) / len(temps_timed)
        t = torch.tensor([ems], dtype=torch.float64, device=dev)
        if world > 1:
            dist.all_reduce(t, op=dist.ReduceOp.MAX)
        ems = float(t.item())
        wbytes = sum(h["W"].numel() * 4 for h in host)
        e2e = {"value": edges_per_step * world / (ems * 1e-3), "unit": UNIT, "ms_per_step": ems, "steps": len(temps_timed),
               "h2d_bytes_per_step": 2 * wbytes + len(host) * wl.S * 4,
               "d2h_bytes_per_step": 2 * wbytes + len(host) * wl.S * 4}
        del host

    # ---- roofline of the dominant kernel: special-function pipe, peak measured in this run
    state_steps = run.state_steps
    dom = "bwd" if bwd_ms >= fwd_ms else "fwd"
    dom_ms = (bwd_ms if dom == "bwd" else fwd_ms) / (args.steps * len(mats))      # average launch
    sm_max = clocks.get("sm_max_mhz") or 1965.0
    peak = peaks["ex2_gops"]
    nominal = NUM_SMS * MUFU_PER_CLK_PER_SM * sm_max * 1e6 / 1e9
    fr = mufu_fractions(wl, state_steps, fwd_ms / args.steps, bwd_ms / args.steps, ms_per_step, peak)
    ops = mufu_ops_per_state_step(wl.k, dom, wl.V, "algorithmic") * state_steps / len(mats)
    achieved = ops / (dom_ms * 1e-3) / 1e9
    # DRAM bytes per block of the dominant kernel: dram__bytes_read.sum + dram__bytes_write.sum of one launch of a
    # small case under ncu (summaries under profiles/), divided by its blocks; traffic is proportional to blocks
    per_block = NCU_DRAM_BYTES_PER_BLOCK.get((wl.Lb, wl.k, dom)) if diag.last_path and wl.V == 1 else None
    traffic = per_block * nblocks / len(mats) if per_block else None
    hbm_peak = None
    try:
        hbm_peak = json.loads((ROOT / "MEASURED_PEAKS.json").read_text()).get("hbm_gbs")
    except (OSError, ValueError):
        pass
    hbm = None
    if traffic:
        gbs = traffic / (dom_ms * 1e-3) / 1e9
        hbm = {"achieved_gbs": gbs, "peak_gbs": hbm_peak or 6650.0,
               "peak_source": "MEASURED_PEAKS.json (measured copy bandwidth)" if hbm_peak else "fallback 6.65 TB/s",
               "frac": gbs / (hbm_peak or 6650.0)}
    roofline = {"bound": "alu", "kernel": f"bcjr_{dom}", "achieved": achieved, "peak": peak, "unit": "Gop/s (MUFU)",
                "frac": achieved / peak, "frac_with_rcp": fr[f"{dom}_frac_with_rcp"],
                "count": "frac: algorithmic special-function operations per state-step (2 + 3/K per call: ex2 per state, "
                         "lg2 per group, posterior ex2 per group); frac_with_rcp: operations the backward kernel issues "
                         "(one rcp per group and sweep more)",
                "traffic": traffic,
                "traffic_source": "ncu dram bytes of a small-case launch, per block, scaled by this launch's blocks",
                "peak_source": "measured in this run: ex2.approx chains on all SMs, CUDA events "
                               f"({peaks['ex2_per_clk_sm']:.2f} per clock per SM at {peaks['sm_clock_mhz']:.0f} MHz)",
                "peak_nominal": nominal,
                "peak_nominal_source": f"{NUM_SMS} SMs x {MUFU_PER_CLK_PER_SM} per clock x {sm_max:.0f} MHz",
                "avg_launch_ms": dom_ms, "hbm": hbm,
                "fwd_frac": fr["fwd_frac"], "bwd_frac": fr["bwd_frac"], "whole_step_frac": fr["both_frac"],
                "whole_step_frac_with_rcp": fr["both_frac_with_rcp"],
                "binding_pipe": {"fwd": "special-function unit 76 % busy; FP32 pipe 55 % + integer pipe 24 % of the cycles "
                                        "(ncu sm__pipe_fma_cycles_active, sm__pipe_alu_cycles_active)",
                                 "bwd": "alpha kernel: special-function unit 74 %; beta kernel: FP32 pipe 57 % + integer pipe 21 % of "
                                        "the cycles, special-function unit 53 %.  Integer-pipe instructions do not overlap with "
                                        "packed f32x2 ones (pipe_peaks: packed pairs per clock alone and with an integer "
                                        "instruction beside each), so the two pipes act as one resource 78 % busy"},
                "pipe_peaks": peaks}

    # ---- short legs over the other workloads, so that one line carries every configuration
    legs = None
    if not args.no_legs and world == 1 and not args.blocks and wl.name.startswith("llama32_1b_decoder"):
        del run, mats
        torch.cuda.empty_cache()
        legs = {}
        for name, cap in (("q_proj", 0), ("gate_k3", 32 * NUM_SMS), ("qtip_v2", 16 * NUM_SMS), ("mid", 0)):
            legs[name] = workload_leg(ctx, name, cap, dev, flush, peak)
        legs["q_proj_fixed_table"] = workload_leg(ctx, "q_proj", 32 * NUM_SMS, dev, flush, peak, fixed_table=True)
        legs["qat_loop"] = qat_loop_leg(ctx, dev, flush)

    if rank == 0:
        base = None
        if not args.no_cpu_baseline and world == 1:
            base, _ = cpu_baseline(wl)
        out = {"metric": METRIC, "value": value, "unit": UNIT, "n_gpus": world, "steps": args.steps,
               "warmup": args.warmup, "ms_per_step": ms_per_step, "higher_is_better": True, "scaling": "weak",
               "vs_baseline": None, "dtype": "f32", "data": "synthetic",
               "config": {"workload": wl.name, "matrices": [n for n, _ in wl.matrices], "blocks": nblocks, "n": wl.n,
                          "Lb": wl.Lb, "k": wl.k, "V": wl.V, "T": [temps_timed[0], temps_timed[-1]],
                          "T_schedule": "geometric over the timed steps, warm-up at the first value" if annealed else "constant",
                          "l2": "256 MB flush write between timed steps; per-step working set >> L2",
                          "path": {0: "generic", 1: "cluster", 2: "warp"}[diag.last_path],
                          **({"backward": "grad_W only (--fixed-table)"} if args.fixed_table else {})},
               "clocks": clocks, "e2e": e2e, "gpu_launches": launches, "roofline": roofline, "cpu_baseline": base,
               "breakdown": {"fwd_ms_per_step": fwd_ms / args.steps, "bwd_ms_per_step": bwd_ms / args.steps,
                             "viterbi": vit, "qat_update": upd, "max_posterior_defect": diag.max_posterior_defect,
                             "workloads": legs}}
        print(json.dumps(out))
    if world > 1:
        dist.destroy_process_group()


if __name__ == "__main__":
    main()

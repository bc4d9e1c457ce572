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


def mufu_ops_per_state_step(k: int, kernel: str, V: int = 1) -> float:
    """Algorithmic special-function operations per state per step (one ex2 per state, plus per
    group of K states: one lg2; the beta sweeps add one ex2 per group for the posterior; the
    backward-pass sweeps add one rcp per group for the conditional expectation)."""
    K = 1 << (k * V)
    fwd = (1 + 1 / K) + (1 + 2 / K)
    bwd = (1 + 2 / K) + (1 + 3 / K)
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


def cpu_baseline(wl, seconds_hint: float = 20.0):
    """The float64 oracle, as it stands, on the host cores: forward + backward of a bounded
    sample of blocks of the same workload (one block per core)."""
    import oracle
    cores = oracle.host_cores()
    # ~5 core-seconds per block at S = 2^16, n = 256 (forward + backward); four blocks per core
    # keep the sample near 20 s; smaller trellises take proportionally more blocks
    scale = max(1, int((1 << 16) * 256 / (wl.S * wl.n)))
    nblk = max(1, min(wl.num_blocks(), 4 * cores * min(scale, 64)))
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
    for _ in range(max(1, args.steps)):
        base, dt = cpu_baseline(wl)
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
    ap.add_argument("--no-cpu-baseline", action="store_true")
    ap.add_argument("--no-e2e", action="store_true")
    ap.add_argument("--no-viterbi", action="store_true")
    args = ap.parse_args()
    wl = WORKLOADS[args.workload]()
    if args.impl == "reference":
        return run_reference(args, wl)

    import torch
    import torch.distributed as dist
    from paper_2605_10655_b200 import Context

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

    # Every rank processes the whole workload shape on its own seeded data (weak scaling over
    # independent blocks); the only exchange is the all-reduce of grad_codebook.
    ctx = Context(local)
    if args.path:
        ctx.set_option("path", args.path)
    if args.fwd_variant:
        ctx.set_option("fwd_variant", args.fwd_variant)
    if args.bwd_variant:
        ctx.set_option("bwd_variant", args.bwd_variant)
    cb = torch.from_numpy(wl.codebook()).to(dev)
    mats = []
    for i, (name, _) in enumerate(wl.matrices):
        W = wl.weights(i)
        if args.blocks:
            W = W[:args.blocks]
        W = np.ascontiguousarray(W)
        if world > 1:
            W = np.roll(W, rank, axis=0)
        mats.append({"name": name, "W_host": torch.from_numpy(W).pin_memory(), "W": torch.from_numpy(W).to(dev)})
    total_steps = args.warmup + args.steps
    temps = anneal_schedule(0.3, 0.01, total_steps) if wl.name.startswith("llama32_1b_decoder") else [wl.T] * total_steps
    nblocks = sum(m["W"].shape[0] for m in mats)
    edges_per_step = 2 * nblocks * wl.steps * wl.S * wl.K
    for m in mats:
        m["soft"] = torch.empty_like(m["W"]); m["gW"] = torch.empty_like(m["W"])
        m["g"] = torch.empty_like(m["W"])
    gc = torch.empty(wl.S * wl.V, dtype=torch.float32, device=dev)
    gc_total = torch.zeros(wl.S * wl.V, dtype=torch.float32, device=dev)
    flush = torch.empty(256 << 20, dtype=torch.uint8, device=dev)      # > L2 (126 MB)
    gen = torch.Generator(device=dev)

    def fresh_g(step):
        for i, m in enumerate(mats):
            gen.manual_seed(wl.g_seed + 7919 * step + i + 104729 * rank)
            m["g"].normal_(generator=gen)

    def one_step(step, T, ev=None):
        gc_total.zero_()
        for m in mats:
            if ev is not None:
                ev["f0"].append(torch.cuda.Event(enable_timing=True)); ev["f0"][-1].record()
            if wl.V == 1:
                ctx.bcjr_soft_quantize(m["W"], cb, wl.Lb, wl.k, wl.n, T, soft=m["soft"])
            else:
                ctx.bcjr_soft_quantize_vec(m["W"], cb, wl.Lb, wl.k, wl.V, wl.n, T, soft=m["soft"])
            if ev is not None:
                ev["f1"].append(torch.cuda.Event(enable_timing=True)); ev["f1"][-1].record()
            ctx.bcjr_backward(m["g"], grad_W=m["gW"], grad_codebook=gc)
            if ev is not None:
                ev["b1"].append(torch.cuda.Event(enable_timing=True)); ev["b1"][-1].record()
            gc_total.add_(gc)
        shard.allreduce_grad_codebook(gc_total)          # the one exchange of the data-parallel path

    for s in range(args.warmup):
        fresh_g(s); flush.zero_()
        one_step(s, temps[s])
    d0 = ctx.sync_status()
    launches0 = d0.kernel_launches
    sampler = ClockSampler(local)
    barrier()
    sampler.start()
    t_wall0 = time.time()
    step_ms, fwd_ms, bwd_ms = [], 0.0, 0.0
    evs = []
    for s in range(args.steps):
        fresh_g(args.warmup + s)
        flush.zero_()                                   # evict L2 between timed steps (not timed)
        e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
        ev = {"f0": [], "f1": [], "b1": []}
        e0.record()
        one_step(args.warmup + s, temps[args.warmup + s], ev)
        e1.record()
        evs.append((e0, e1, ev))
    barrier()
    t_wall1 = time.time()
    for e0, e1, ev in evs:
        step_ms.append(e0.elapsed_time(e1))
        fwd_ms += sum(a.elapsed_time(b) for a, b in zip(ev["f0"], ev["f1"]))
        bwd_ms += sum(a.elapsed_time(b) for a, b in zip(ev["f1"], ev["b1"]))
    clocks = sampler.stop(t_wall0, t_wall1)
    diag = ctx.sync_status()
    launches = diag.kernel_launches - launches0
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

    # ---- end to end through the host-buffer entry point (pinned host memory both ways)
    e2e = None
    if not args.no_e2e and wl.V == 1:          # the host-buffer entry point covers the scalar trellis
        host = []
        for m in mats:
            host.append({"W": m["W_host"], "g": m["g"].cpu().pin_memory(),
                         "soft": torch.empty_like(m["W_host"]).pin_memory(),
                         "gW": torch.empty_like(m["W_host"]).pin_memory()})
        cb_h = cb.cpu().pin_memory(); gc_h = torch.empty(wl.S).pin_memory()
        T_e = temps[-1]

        def e2e_step():
            for h in host:
                ctx.bcjr_step_host(h["W"], cb_h, h["g"], wl.Lb, wl.k, wl.n, T_e, soft=h["soft"], grad_W=h["gW"],
                                   grad_codebook=gc_h)
        e2e_step()                                                  # warm-up (allocates staging buffers)
        barrier()
        reps = max(1, min(args.steps, 2))
        e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
        e0.record()
        for _ in range(reps):
            e2e_step()
        e1.record()
        barrier()
        ems = e0.elapsed_time(e1) / reps
        t = torch.tensor([ems], dtype=torch.float64, device=dev)
        if world > 1:
            dist.all_reduce(t, op=dist.ReduceOp.MAX)
        ems = float(t.item())
        wbytes = sum(h["W"].numel() * 4 for h in host)
        e2e = {"value": edges_per_step * world / (ems * 1e-3), "unit": UNIT, "ms_per_step": ems,
               "h2d_bytes_per_step": 2 * wbytes + len(host) * wl.S * 4,
               "d2h_bytes_per_step": 2 * wbytes + len(host) * wl.S * 4}

    # ---- roofline of the dominant kernel (the backward-pass kernel): special-function pipe
    state_steps = nblocks * wl.steps * wl.S
    dom = "bwd" if bwd_ms >= fwd_ms else "fwd"
    dom_ms = (bwd_ms if dom == "bwd" else fwd_ms) / (args.steps * len(mats))
    ops = mufu_ops_per_state_step(wl.k, dom, wl.V) * state_steps / len(mats)
    achieved = ops / (dom_ms * 1e-3) / 1e9
    sm_max = clocks.get("sm_max_mhz") or 1965.0
    peak = NUM_SMS * MUFU_PER_CLK_PER_SM * sm_max * 1e6 / 1e9
    # DRAM bytes per block of the dominant kernel, from the ncu captures summarised under profiles/
    # (dram__bytes_read.sum + dram__bytes_write.sum of one launch / blocks of that launch, small
    # case of the same kernel; traffic grows in proportion to the number of blocks)
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
                "frac": achieved / peak, "traffic": traffic,
                "peak_source": f"{NUM_SMS} SMs x {MUFU_PER_CLK_PER_SM} MUFU/clk x {sm_max:.0f} MHz (derived)",
                "avg_launch_ms": dom_ms, "hbm": hbm,
                "whole_step_frac": mufu_ops_per_state_step(wl.k, "both", wl.V) * state_steps / (ms_per_step * 1e-3) / 1e9 / peak}

    if rank == 0:
        base = None
        if not args.no_cpu_baseline and world == 1:
            base, _ = cpu_baseline(wl)
        out = {"metric": METRIC, "value": value, "unit": UNIT, "n_gpus": world, "steps": args.steps,
               "warmup": args.warmup, "ms_per_step": ms_per_step, "higher_is_better": True, "scaling": "weak",
               "vs_baseline": None, "dtype": "f32", "data": "synthetic",
               "config": {"workload": wl.name, "matrices": [m["name"] for m in mats], "blocks": nblocks, "n": wl.n,
                          "Lb": wl.Lb, "k": wl.k, "V": wl.V, "T": [temps[args.warmup], temps[-1]],
                          "l2": "256 MB flush write between timed steps; per-step working set >> L2",
                          "path": "cluster" if diag.last_path else "generic"},
               "clocks": clocks, "e2e": e2e, "gpu_launches": launches, "roofline": roofline, "cpu_baseline": base,
               "breakdown": {"fwd_ms_per_step": fwd_ms / args.steps, "bwd_ms_per_step": bwd_ms / args.steps,
                             "viterbi": vit, "qat_update": upd, "max_posterior_defect": diag.max_posterior_defect}}
        print(json.dumps(out))
    if world > 1:
        dist.destroy_process_group()


if __name__ == "__main__":
    main()

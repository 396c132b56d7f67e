#!/usr/bin/env python
"""Benchmark of the ParallelSpec hot path: ps_draft_step + ps_verify steps per second.

    python bench.py [--gpus N] [--steps K] [--warmup W] [--workload 13b|7b|33b|13b_sweep|tiny]
                    [--batch B] [--k-masks k]     # a point of the batch / mask-count sweep
    python bench.py --impl reference ...      # the CPU checker timed on the host cores

One "step" = one parallel draft step (all k+1 rows, logits stored) followed by one verify
call on synthetic target logits, for the workload's batch.  N > 1 (under torchrun) runs N
independent replicas, one per GPU, with no data-path collective.  Rank 0 prints ONE JSON line.
"""
from __future__ import annotations

import argparse
import json
import os
import statistics
import sys
import threading
import time

ROOT = os.path.dirname(os.path.abspath(__file__))
if ROOT not in sys.path:
    sys.path.insert(0, ROOT)

METRIC = "draft+verify steps/sec"
NOMINAL_HBM_GBS = 8000.0
FALLBACK_HBM_GBS = 6650.0
L2_BYTES = 126 << 20


def parse_args():
    ap = argparse.ArgumentParser()
    ap.add_argument("--gpus", type=int, default=1)
    ap.add_argument("--steps", type=int, default=1000)
    ap.add_argument("--warmup", type=int, default=20)
    ap.add_argument("--impl", default="ours", choices=["ours", "reference"])
    ap.add_argument("--workload", default="13b",
                    choices=["13b", "7b", "33b", "llama3_8b", "13b_sweep", "tiny", "mini"])
    ap.add_argument("--batch", type=int, default=0, help="sequences per step (default: the workload's)")
    ap.add_argument("--k-masks", type=int, default=-1, help="[MASK] positions per sequence (default: the workload's)")
    ap.add_argument("--temperature", type=float, default=1.0)
    ap.add_argument("--no-cpu-baseline", action="store_true")
    ap.add_argument("--cpu-seconds", type=float, default=15.0)
    return ap.parse_args()


def measured_peak():
    path = os.path.join(ROOT, "MEASURED_PEAKS.json")
    try:
        with open(path) as f:
            return float(json.load(f)["hbm_gbs"]), "measured"
    except Exception:
        return FALLBACK_HBM_GBS, "fallback"


# Kernel that runs each stage of the bf16 small-batch path.
KERNEL_OF_STAGE = {
    "fc_norm": "k_gather_x + k_umma_gemm<STORE>", "qkv_rope": "k_umma_gemm<STORE>",
    "attention": "k_attn_mma", "o_proj": "k_umma_gemm<STORE>", "ffn_gate_up": "k_umma_gemm<SWIGLU>",
    "ffn_down": "k_umma_gemm<STORE>", "lm_head": "k_umma_gemm<LMHEAD>", "verify": "k_verify_cluster",
}


def kernel_of_stage(stage, rows):
    if stage == "lm_head" and rows > 32:   # logits stored by the GEMM, statistics by one block per row
        return "k_umma_gemm<STORE> + k_row_stats"
    return KERNEL_OF_STAGE.get(stage, stage)


# dram__bytes_read.sum + dram__bytes_write.sum per launch from the ncu capture summarised in
# profiles/k_umma_gemm_13b_b1_k4.md, keyed by (workload, batch, k_masks, stage).  Valid for the
# kernels as captured; set an entry to None when its kernel changes.
NCU_DRAM_BYTES = {
    ("13b", 1, 4, "fc_norm"): 106259200 + 4141824,
    ("13b", 1, 4, "qkv_rope"): 158127872 + 3880704,
    ("13b", 1, 4, "o_proj"): 53316352 + 8960,
    ("13b", 1, 4, "ffn_gate_up"): 285139968 + 4767232,
    ("13b", 1, 4, "ffn_down"): 143910144 + 4637184,
    ("13b", 1, 4, "lm_head"): 329474816 + 5147648,
}


def stage_bytes(s, B, lens):
    """Algorithmic bytes each stage must move per step (weights once, KV once, logits written
    once by the LM head and read once by verify together with the target logits)."""
    e = 4 if s.dtype == 0 else 2
    H, F, V = s.hidden, s.ffn, s.vocab
    Hq, Hkv = s.n_heads * s.head_dim, s.n_kv_heads * s.head_dim
    M = B * (s.k_masks + 1)
    return {
        "fc_norm": e * 2 * H * H,
        "qkv_rope": e * (Hq * H + 2 * Hkv * H),
        "attention": e * 2 * Hkv * int(sum(lens)),
        "o_proj": e * H * Hq,
        "ffn_gate_up": e * 2 * H * F,
        "ffn_down": e * H * F,
        "lm_head": e * V * H + 4 * M * V,
        "verify": 8 * M * V,
    }


# A 26-node draft tree of the shape tree drafters use (4 children of the root, depth 6).
TREE26 = [-1, -1, -1, -1, 0, 0, 0, 1, 1, 2, 4, 4, 5, 7, 10, 10, 11, 12, 13, 14, 14, 16, 18, 19, 21, 22]


def tree_verify_leg(g, ps, s, B, T, peak, n_buf=6, reps=60):
    """ps_verify_tree alone on the 26-node tree: synthetic target rows per node, one draft row
    per depth (noisy copies, so that paths of several nodes are accepted), node tokens drawn
    from the draft rows.  Buffers rotate so that rows come from HBM, not from L2."""
    import numpy as np
    import torch

    import synth
    n = len(TREE26)
    depth = []
    for p in TREE26:
        depth.append(0 if p < 0 else depth[p] + 1)
    D, V = max(depth) + 1, s.vocab
    sets = []
    for i in range(n_buf):
        tl = synth.gauss_logits(s.seed, ("tree_t", i), (B, n + 1, V))
        dl = synth.noisy_draft_logits(s.seed, ("tree_d", i), np.repeat(tl[:, :1], D, axis=1), 0.6)
        for j in range(n):
            if depth[j] + 1 < D:
                tl[:, 1 + j] = dl[:, depth[j] + 1] + 0.5 * tl[:, 1 + j]
        toks = synth.sample_from_logits(s.seed, ("tree_x", i), dl[:, depth], temperature=max(T, 0.5))
        sets.append((ps.to_device(toks.astype(np.int32)), ps.to_device(dl), ps.to_device(tl)))
    out = {}
    for i in range(5):
        t_, d_, l_ = sets[i % n_buf]
        g.verify_tree(TREE26, t_, d_, l_, T, 1, i, out=out)
    torch.cuda.synchronize()
    e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
    e0.record()
    for i in range(reps):
        t_, d_, l_ = sets[i % n_buf]
        g.verify_tree(TREE26, t_, d_, l_, T, 1, 100 + i, out=out)
    e1.record()
    torch.cuda.synchronize()
    us = e0.elapsed_time(e1) / reps * 1e3
    rows_with_children = len({p for p in TREE26})            # decision rows that read a draft row
    nbytes = 4 * V * B * ((n + 1) + rows_with_children)
    return {"us": round(us, 2), "nodes": n, "depth": D, "bytes": nbytes,
            "gbs": round(nbytes / (us * 1e-6) / 1e9, 1), "frac_of_peak": round(nbytes / (us * 1e-6) / 1e9 / peak, 4),
            "mean_accepted_nodes": float(out["accept_len"].float().mean().item()),
            "note": "(n+1) target rows and one draft row per row with children, each read once"}


def max_over_ranks(x: float, device="cuda") -> float:
    """Slowest rank's value (every rank gets it).  Replicas exchange nothing else."""
    import torch
    import torch.distributed as dist

    if not (dist.is_available() and dist.is_initialized()) or dist.get_world_size() == 1:
        return float(x)
    t = torch.tensor([float(x)], dtype=torch.float64, device=device)
    dist.all_reduce(t, op=dist.ReduceOp.MAX)
    return float(t.item())


def aggregate_steps_per_s(world: int, steps_per_rank: int, slowest_ms: float) -> float:
    """Whole-job throughput of N independent replicas: all steps over the slowest rank's time."""
    return world * steps_per_rank / (slowest_ms * 1e-3)


class ClockSampler(threading.Thread):
    """Reads SM clock and throttle reasons through NVML while the timed region runs."""

    def __init__(self, device_index: int):
        super().__init__(daemon=True)
        self.samples, self.reasons, self.max_mhz = [], set(), None
        self._stop_evt = threading.Event()
        self.ok = False
        try:
            import pynvml
            import torch

            pynvml.nvmlInit()
            uuid = str(torch.cuda.get_device_properties(device_index).uuid)
            h = None
            for i in range(pynvml.nvmlDeviceGetCount()):
                hi = pynvml.nvmlDeviceGetHandleByIndex(i)
                u = pynvml.nvmlDeviceGetUUID(hi)
                u = u.decode() if isinstance(u, bytes) else u
                if uuid in u or u.replace("GPU-", "") == uuid:
                    h = hi
            self.h = h if h is not None else pynvml.nvmlDeviceGetHandleByIndex(device_index)
            self.nv = pynvml
            self.max_mhz = pynvml.nvmlDeviceGetMaxClockInfo(self.h, pynvml.NVML_CLOCK_SM)
            self.ok = True
        except Exception:
            self.ok = False

    def run(self):
        if not self.ok:
            return
        nv = self.nv
        names = {
            "hw_slowdown": getattr(nv, "nvmlClocksThrottleReasonHwSlowdown", 0x8),
            "hw_thermal_slowdown": getattr(nv, "nvmlClocksThrottleReasonHwThermalSlowdown", 0x40),
            "sw_thermal_slowdown": getattr(nv, "nvmlClocksThrottleReasonSwThermalSlowdown", 0x20),
            "sw_power_cap": getattr(nv, "nvmlClocksThrottleReasonSwPowerCap", 0x4),
        }
        while not self._stop_evt.is_set():
            try:
                self.samples.append(nv.nvmlDeviceGetClockInfo(self.h, nv.NVML_CLOCK_SM))
                r = nv.nvmlDeviceGetCurrentClocksThrottleReasons(self.h)
                for k, bit in names.items():
                    if r & bit:
                        self.reasons.add(k)
            except Exception:
                pass
            time.sleep(0.01)

    def stop(self):
        self._stop_evt.set()
        if self.is_alive():
            self.join(timeout=2)
        med = statistics.median(self.samples) if self.samples else None
        return {"sm_mhz": med, "sm_max_mhz": self.max_mhz, "reasons": sorted(self.reasons),
                "samples": len(self.samples)}


def oracle_setup(s, B, lens):
    import oracle
    import synth
    from synth import bf16_bits_to_f32

    W = synth.weights(s)
    max_ctx = int(max(lens)) + s.rows
    o = oracle.Oracle(oracle.OracleConfig(s.dtype, s.hidden, s.n_heads, s.n_kv_heads, s.head_dim,
                                          s.ffn, s.vocab, s.k_masks, B, max_ctx, s.rope_base,
                                          s.rms_eps), W)
    for b in range(B):
        K, V = synth.kv_rows(s, ("kv", b), int(lens[b]))
        if s.dtype == 1:
            K, V = bf16_bits_to_f32(K), bf16_bits_to_f32(V)
        o.kv_import(b, K.astype("float64"), V.astype("float64"))
    return o


def oracle_time_step(o, s, b, k_use, hidden_last, token_last, target, T):
    """Seconds of one oracle draft step (k_use+1 rows) + verify on those rows, sequence b."""
    import numpy as np

    import oracle

    t0 = time.perf_counter()
    out = o.draft_step(b, hidden_last[b:b + 1], int(token_last[b]), k_use=k_use)
    lg = out["logits"].astype(np.float32)[None]
    toks = lg.argmax(-1).astype(np.int32)
    oracle.verify(toks, lg, target[b:b + 1, :k_use + 1], T, 1, 0)
    return time.perf_counter() - t0


def cpu_baseline(s, B, lens, hidden_last, token_last, target, T, budget_s):
    """The CPU checker, as it stands, on a bounded sample of the same workload."""
    import oracle

    o = oracle_setup(s, B, lens)
    R = s.rows
    # first: one row of sequence 0 to size the sample
    t_row = oracle_time_step(o, s, 0, 0, hidden_last, token_last, target, T)
    full_step = t_row * R * B
    if full_step <= budget_s:
        n_seq, k_use = B, s.k_masks
    elif t_row * R <= budget_s:
        n_seq, k_use = max(1, int(budget_s / (t_row * R))), s.k_masks
    else:
        n_seq, k_use = 1, max(0, int(budget_s / t_row) - 1)
    t, reps = 0.0, 0
    while reps == 0 or (t < 0.7 * budget_s and reps < 200):   # repeat short samples up to the budget
        for b in range(n_seq):
            t += oracle_time_step(o, s, b, k_use, hidden_last, token_last, target, T)
        reps += 1
    rows_done = reps * n_seq * (k_use + 1)
    est_step = t * (B * R) / rows_done
    sample = (f"{reps} x ({n_seq} of {B} sequences x {k_use + 1} of {R} rows of one draft+verify "
              f"step), {t:.1f} s of CPU work, scaled by rows to a full step")
    return {"value": 1.0 / est_step, "unit": "steps/s", "cores": oracle.num_threads(),
            "kind": "oracle", "sample": sample}


def run_reference(args):
    """--impl reference: the CPU checker timed on the host cores (rank 0 only)."""
    if int(os.environ.get("RANK", "0")) != 0:
        return
    import numpy as np

    import oracle
    import synth

    s = workload_shape(args)
    B = s.batch
    lens = synth.ctx_lengths(s, B)
    o = oracle_setup(s, B, lens)
    hl, tl = synth.hidden_states(s, "last", B), synth.token_ids(s, "last", B)
    tgt = (synth.zipf_logits(s.seed, "tgt0", B, s.rows, s.vocab) if s.logits_kind == "zipf"
           else synth.gauss_logits(s.seed, "tgt0", (B, s.rows, s.vocab)))
    R = s.rows
    t_row = oracle_time_step(o, s, 0, 0, hl, tl, tgt, args.temperature)
    total_steps = args.steps + args.warmup
    budget = 150.0 / max(1, total_steps)
    k_use = min(s.k_masks, max(0, int(budget / t_row) - 1))
    n_seq = 1 if t_row * (k_use + 1) * 2 > budget else min(B, max(1, int(budget / (t_row * (k_use + 1)))))
    times = []
    for i in range(total_steps):
        t = sum(oracle_time_step(o, s, b, k_use, hl, tl, tgt, args.temperature) for b in range(n_seq))
        if i >= args.warmup:
            times.append(t)
    per_step = (sum(times) / len(times)) * (B * R) / (n_seq * (k_use + 1))
    value = 1.0 / per_step
    sample = (f"each step: {n_seq} of {B} sequences x {k_use + 1} of {R} rows of the oracle's draft "
              f"step + verify, scaled by rows to a full step")
    line = {
        "impl": "reference", "metric": METRIC, "value": value, "unit": "steps/s",
        "n_gpus": args.gpus, "steps": args.steps, "warmup": args.warmup,
        "ms_per_step": per_step * 1e3, "higher_is_better": True, "scaling": "weak",
        "vs_baseline": None, "dtype": "f64", "data": "synthetic",
        "config": workload_config(s, B, lens),
        "cpu_baseline": {"value": value, "unit": "steps/s", "cores": oracle.num_threads(),
                         "kind": "oracle", "sample": sample},
        "e2e": {"value": value, "unit": "steps/s", "h2d_bytes_per_step": 0, "d2h_bytes_per_step": 0},
        "drafted_tokens_per_s": value * B * R,
    }
    print(json.dumps(line))


def workload_shape(args):
    import synth
    s = synth.CONFIGS[args.workload]
    if args.batch > 0:
        s = s.with_(batch=args.batch)
    if args.k_masks >= 0:
        s = s.with_(k_masks=args.k_masks)
    return s


def workload_config(s, B, lens):
    return {
        "workload": f"{s.name}: H{s.hidden} heads{s.n_heads}x{s.head_dim} F{s.ffn} V{s.vocab} "
                    f"B{B} k{s.k_masks} ctx{int(min(lens))}-{int(max(lens))} "
                    f"{'fp32' if s.dtype == 0 else 'bf16'}",
        "batch": B, "k_masks": s.k_masks, "rows_per_step": B * s.rows,
        "verify": "n_draft=n_target=k+1, draft logits stored, Zipf(1.1)-biased target logits",
    }


def main():
    args = parse_args()
    if args.impl == "reference":
        run_reference(args)
        return

    import numpy as np
    import torch
    import torch.distributed as dist

    import paper_2410_05589_b200 as ps
    import synth

    rank = int(os.environ.get("RANK", "0"))
    world = int(os.environ.get("WORLD_SIZE", "1"))
    local = int(os.environ.get("LOCAL_RANK", "0"))
    if not torch.cuda.is_available():
        raise SystemExit("bench.py needs a CUDA device: the library has no CPU path")
    torch.cuda.set_device(local)
    if world > 1:
        dist.init_process_group("nccl", device_id=torch.device("cuda", local))

    s = workload_shape(args)
    B, R, V, T = s.batch, s.rows, s.vocab, args.temperature
    lens = synth.ctx_lengths(s, B)
    W = synth.weights(s)
    kv_bytes_seq = 2 * s.n_kv_heads * s.head_dim * int(lens.mean()) * (4 if s.dtype == 0 else 2)
    # rotate over enough distinct KV sets that consecutive steps never find their KV in L2
    n_sets = 1 if kv_bytes_seq * B > 2 * L2_BYTES else max(2, min(16, -(-2 * L2_BYTES // max(1, kv_bytes_seq * B))))
    n_sets = min(n_sets, 128 // B)
    max_ctx_bench = int(lens.max()) + R + 64        # + room for the groups of the training-layout leg
    g = ps.drafter_from_shape(s, W, max_batch=B * n_sets, max_ctx=max_ctx_bench)
    del W
    for i in range(n_sets):
        for b in range(B):
            K, Vv = synth.kv_rows(s, ("kv", b), int(lens[b]))
            g.kv_import(i * B + b, ps.to_device(K), ps.to_device(Vv))
    hl_np, tl_np = synth.hidden_states(s, "last", B), synth.token_ids(s, "last", B)
    tgt_np = [(synth.zipf_logits(s.seed, f"tgt{i}", B, R, V) if s.logits_kind == "zipf"
               else synth.gauss_logits(s.seed, f"tgt{i}", (B, R, V))) for i in range(min(n_sets, 4))]
    hl, tl = ps.to_device(hl_np), ps.to_device(tl_np)
    tgt = [ps.to_device(t) for t in tgt_np]
    slots = [[i * B + b for b in range(B)] for i in range(n_sets)]
    d_out, v_out = {}, {}

    def step(i):
        o = g.draft_step(slots[i % n_sets], hl, tl, top_n=1, want_logits=True, out=d_out)
        g.verify(o["top_ids"].view(B, R), o["logits"], tgt[i % len(tgt)], T, 1, i, out=v_out)

    for i in range(max(3, args.warmup)):
        step(i)
    torch.cuda.synchronize()
    if world > 1:
        dist.barrier()
    sampler = ClockSampler(local)
    sampler.start()
    l0 = g.launch_count()
    e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
    torch.cuda.synchronize()
    e0.record()
    for i in range(args.steps):
        step(i)
    e1.record()
    torch.cuda.synchronize()
    launches = g.launch_count() - l0
    clocks = sampler.stop()
    if world > 1:
        dist.barrier()
    ms = max_over_ranks(e0.elapsed_time(e1))
    assert g.poll() == 0, "device status word set during the timed region"
    n_accept = float(v_out["n_out"].float().mean().item())

    # ---- per-stage times (CUDA events recorded by the library between stages) -------------
    g.profile(True)
    n_prof = min(args.steps, 200)
    for i in range(n_prof):
        step(i)
    torch.cuda.synchronize()
    prof = g.profile_read()
    g.profile(False)
    sb = stage_bytes(s, B, lens)
    peak, peak_kind = measured_peak()
    stages = {}
    for name, (tot, cnt) in prof.items():
        if cnt and name in sb:
            # per step, not per launch: a batch beyond 128 rows runs a stage several times a step
            us = tot / n_prof * 1e3
            stages[name] = {"us": round(us, 2), "gbs": round(sb[name] / (us * 1e-6) / 1e9, 1),
                            "launches_per_step": round(cnt / n_prof, 2)}
    dom = max(stages, key=lambda k: stages[k]["us"]) if stages else None
    step_bytes = sum(sb.values())
    roofline = None
    if dom:
        roofline = {
            "bound": "hbm", "kernel": kernel_of_stage(dom, B * R), "stage": dom,
            "achieved": stages[dom]["gbs"], "peak": peak,
            "unit": "GB/s", "frac": round(stages[dom]["gbs"] / peak, 4),
            "traffic": NCU_DRAM_BYTES.get((args.workload, B, s.k_masks, dom)),
            "peak_kind": f"of {peak_kind}", "bytes_per_launch": sb[dom],
        }

    # ---- the same step with the drafts sampled in the LM head (lossless at T > 0) -------------
    sampled = None
    if T > 0:
        s_out = {}

        def step_sampled(i):
            o = g.draft_step_sampled(slots[i % n_sets], hl, tl, T, 1, i, top_n=1, want_logits=True, out=s_out)
            g.verify(o["sampled"], o["logits"], tgt[i % len(tgt)], T, 1, i, out=v_out)

        for i in range(5):
            step_sampled(i)
        torch.cuda.synchronize()
        n_s = min(args.steps, 300)
        f0, f1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
        f0.record()
        for i in range(n_s):
            step_sampled(i)
        f1.record()
        torch.cuda.synchronize()
        sampled = {"ms_per_step": f0.elapsed_time(f1) / n_s, "steps": n_s,
                   "note": "ps_draft_step_sampled (Gumbel-max in the LM-head epilogue) + ps_verify"}

    # ---- group-wise training layout, forward only (Sec. 4.1): groups on the last KV set ---------
    group = None
    if int(lens.max()) + 64 + s.k_masks <= max_ctx_bench:
        n_g = 64
        gh = ps.to_device(synth.hidden_states(s, "grp", n_g))
        gt = ps.to_device(synth.token_ids(s, "grp", n_g))
        for i in range(2):
            g.group_forward(int(slots[0][0]), gh, gt, top_n=1, want_logits=False)
        torch.cuda.synchronize()
        h0, h1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
        h0.record()
        for i in range(5):
            g.group_forward(int(slots[0][0]), gh, gt, top_n=1, want_logits=False)
        h1.record()
        torch.cuda.synchronize()
        group = {"ms_per_call": h0.elapsed_time(h1) / 5, "groups": n_g, "rows": n_g * R,
                 "note": "ps_group_forward; the groups run as draft steps of up to 128 rows per launch"}

    # ---- token-tree verification (Algorithm 1 in full), timed on its own ---------------------
    tree = None
    if V % 4 == 0 and V <= 131072 and s.dtype == 1:
        tree = tree_verify_leg(g, ps, s, B, T, peak)

    # ---- end to end through the host-buffer entry point -----------------------------------
    hl_h = torch.from_numpy(hl_np.view(np.int16) if hl_np.dtype == np.uint16 else hl_np).pin_memory()
    tl_h = torch.from_numpy(tl_np).pin_memory()
    tgt_h = [torch.from_numpy(t).pin_memory() for t in tgt_np]
    r_out = {}
    n_e2e = min(args.steps, 500)
    for i in range(3):
        g.round_host(slots[i % n_sets], hl_h, tl_h, tgt_h[i % len(tgt_h)], T, 1, i, out=r_out)
    torch.cuda.synchronize()
    if world > 1:
        dist.barrier()
    t0 = time.perf_counter()
    for i in range(n_e2e):
        g.round_host(slots[i % n_sets], hl_h, tl_h, tgt_h[i % len(tgt_h)], T, 1, i, out=r_out)
    torch.cuda.synchronize()
    e2e_s = max_over_ranks(time.perf_counter() - t0)
    eb = 4 if s.dtype == 0 else 2
    e2e = {"value": aggregate_steps_per_s(world, n_e2e, e2e_s * 1e3), "unit": "steps/s",
           "h2d_bytes_per_step": B * s.hidden * eb + B * 4 + B * R * V * 4,
           "d2h_bytes_per_step": B * (R + 3) * 4, "steps": n_e2e}

    # ---- ps_kv_append (once per round, off the draft step's path): 4 accepted pairs a sequence ----
    n_new = 4
    ka_h = ps.to_device(synth.hidden_states(s, "app", B * n_new))
    ka_t = ps.to_device(synth.token_ids(s, "app", B * n_new))
    app_slots = slots[0]   # last leg on the device: these slots' contexts are not needed again

    def append_once():
        for x in app_slots:   # host bookkeeping only: the same cache rows are written every time
            g.kv_reset(x)
        g.kv_append(app_slots, [n_new] * B, ka_h, ka_t)

    for i in range(3):
        append_once()
    torch.cuda.synchronize()
    k0, k1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
    k0.record()
    for i in range(50):
        append_once()
    k1.record()
    torch.cuda.synchronize()
    app_us = k0.elapsed_time(k1) / 50 * 1e3
    app_bytes = eb * (2 * s.hidden * s.hidden + 2 * s.n_kv_heads * s.head_dim * s.hidden)
    kv_append = {"us": round(app_us, 2), "rows": B * n_new, "bytes": app_bytes,
                 "gbs": round(app_bytes / (app_us * 1e-6) / 1e9, 1),
                 "note": "fc + k|v weights read once, 4 new real positions per sequence"}

    cpu = None
    if rank == 0 and world == 1 and not args.no_cpu_baseline:
        cpu = cpu_baseline(s, B, lens, hl_np, tl_np, tgt_np[0], T, args.cpu_seconds)

    if rank == 0:
        ms_per_step = ms / args.steps
        value = aggregate_steps_per_s(world, args.steps, ms)
        gbs = step_bytes / (ms_per_step * 1e-3) / 1e9
        line = {
            "metric": METRIC, "value": value, "unit": "steps/s", "n_gpus": world,
            "steps": args.steps, "warmup": max(3, args.warmup), "ms_per_step": ms_per_step,
            "higher_is_better": True, "scaling": "weak", "vs_baseline": None,
            "dtype": "f32" if s.dtype == 0 else "bf16", "data": "synthetic",
            "config": dict(workload_config(s, B, lens),
                           l2="weights exceed L2 and are streamed every step; KV caches rotate over "
                              f"{n_sets} distinct sets, target logits over {len(tgt)} buffers",
                           parallelism="replicas" if world > 1 else "single GPU"),
            "drafted_tokens_per_s": value * B * R,
            "step_bytes": step_bytes, "step_gbs": round(gbs, 1),
            "hbm_frac_of_measured": round(gbs / peak, 4),
            "hbm_frac_of_nominal_8TBs": round(gbs / NOMINAL_HBM_GBS, 4),
            "mean_tokens_per_round": n_accept,
            "clocks": clocks, "e2e": e2e, "gpu_launches": int(launches),
            "roofline": roofline, "stages": stages, "sampled_drafts": sampled, "group_forward": group, "tree_verify": tree, "kv_append": kv_append, "cpu_baseline": cpu,
        }
        print(json.dumps(line))
    if world > 1:
        dist.destroy_process_group()


if __name__ == "__main__":
    main()

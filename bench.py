#!/usr/bin/env python
"""Benchmark of the ParallelSpec hot path: ps_draft_step + ps_verify steps per second.

    python bench.py [--gpus N] [--steps K] [--warmup W] [--workload 13b|7b|33b|13b_sweep|tiny]
                    [--batch B] [--k-masks k]     # a point of the batch / mask-count sweep
                    [--flags F]                   # ps_config.flags (2: plain kernels, 4: mma.sync GEMMs)
                    [--no-configs]                # skip the other workloads' sub-records
    python bench.py --impl reference ...      # the CPU checker timed on the host cores

One "step" = one parallel draft step (all k+1 rows, logits stored) followed by one verify
call on synthetic target logits, for the workload's batch.  At temperature > 0 the drafts are
drawn from the draft distribution inside the LM head (ps_draft_step_sampled), which is what
makes the round lossless (Eq. 1 needs x ~ q); at temperature 0 they are the rows' arg-max
tokens.  N > 1 (under torchrun) runs N independent replicas, one per GPU, with no data-path
collective.  Rank 0 prints ONE JSON line.
"""
from __future__ import annotations

import argparse
import hashlib
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
VERIFY_SIGMA = 0.4     # draft logits = target + N(0, sigma^2): about 3.5 tokens a round at k = 4 (Table 1's regime)


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
    ap.add_argument("--flags", type=int, default=0, help="ps_config.flags of the context")
    ap.add_argument("--no-cpu-baseline", action="store_true")
    ap.add_argument("--no-configs", action="store_true", help="headline workload only")
    ap.add_argument("--cpu-seconds", type=float, default=12.0)
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


# Stages that share a launch when a step has up to 16 rows.
LAUNCH_STAGES = {"chain_fc_qkv": ("fc_norm", "qkv_rope"),
                 "chain_o_ffn_lm": ("o_proj", "ffn_gate_up", "ffn_down", "lm_head")}
KERNEL_OF_STAGE["chain_fc_qkv"] = "k_gather_x + k_umma_chain (fc, q|k|v)"
KERNEL_OF_STAGE["chain_o_ffn_lm"] = "k_umma_chain (o, gate|up, down, LM head)"


def kernel_of_stage(stage, rows):
    if stage == "lm_head" and rows > 32:   # logits stored by the GEMM, statistics by one block per row
        return "k_umma_gemm<STORE> + k_row_stats"
    return KERNEL_OF_STAGE.get(stage, stage)


GEMM_SOURCES = ("fused_kernels.cu", "umma_gemm.cuh", "ws_gemm.cuh", "ps_internal.cuh")


def kernel_sources_digest():
    """sha256 over the sources of the GEMM kernels' translation unit: a counter capture is valid
    for the sources it was taken on."""
    h = hashlib.sha256()
    d = os.path.join(ROOT, "paper_2410_05589_b200", "csrc")
    for name in GEMM_SOURCES:
        with open(os.path.join(d, name), "rb") as f:
            h.update(name.encode())
            h.update(f.read())
    return h.hexdigest()


def captured_dram_bytes(workload, B, k, stage):
    """dram__bytes_read.sum + dram__bytes_write.sum per launch of the stage's kernel, from the
    counter capture recorded under profiles/ -- or None when there is none for this workload or
    the kernel sources have changed since it was taken."""
    try:
        with open(os.path.join(ROOT, "profiles", "dram_bytes_per_launch.json")) as f:
            rec = json.load(f)
        if rec.get("kernel_sources_sha256") != kernel_sources_digest():
            return None
        return rec["bytes"].get(f"{workload}/B{B}/k{k}/{stage}")
    except Exception:
        return None


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


# ---- the CPU checker as a timed baseline ---------------------------------------------------------
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
    """The CPU checker, as it stands, on a bounded sample of the same workload: on all host
    cores, and (a shorter sample) on one."""
    import oracle

    o = oracle_setup(s, B, lens)
    R = s.rows
    cores = oracle.num_threads()
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
    # one thread: rows of sequence 0 for about a third of the budget
    oracle.set_threads(1)
    t1, rows1 = 0.0, 0
    while rows1 == 0 or (t1 < budget_s / 3 and rows1 < 4 * R):
        k1 = min(s.k_masks, 1)
        t1 += oracle_time_step(o, s, 0, k1, hidden_last, token_last, target, T)
        rows1 += k1 + 1
    oracle.set_threads(cores)
    one = {"value": rows1 / (t1 * B * R), "unit": "steps/s", "cores": 1,
           "sample": f"{rows1} rows of sequence 0, {t1:.1f} s, scaled by rows to a full step"}
    return {"value": 1.0 / est_step, "unit": "steps/s", "cores": cores,
            "kind": "oracle", "sample": sample, "one_thread": one}


def run_reference(args):
    """--impl reference: the CPU checker timed on the host cores (rank 0 only)."""
    if int(os.environ.get("RANK", "0")) != 0:
        return
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
        "config": workload_config(s, B, lens, args.temperature),
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


def workload_config(s, B, lens, T):
    drafts = ("drafts drawn from q in the LM head (lossless round)" if T > 0 else "arg-max drafts, greedy verify")
    return {
        "workload": f"{s.name}: H{s.hidden} heads{s.n_heads}x{s.head_dim} F{s.ffn} V{s.vocab} "
                    f"B{B} k{s.k_masks} ctx{int(min(lens))}-{int(max(lens))} "
                    f"{'fp32' if s.dtype == 0 else 'bf16'}",
        "batch": B, "k_masks": s.k_masks, "rows_per_step": B * s.rows,
        "verify": f"n_draft=n_target=k+1, draft logits stored, Zipf(1.1)-biased target logits, T={T:g}, {drafts}",
    }


# ---- one workload resident on the GPU ------------------------------------------------------------
class Workload:
    """A drafter with its KV caches and the step's inputs resident in HBM.  The weights exceed L2
    and are streamed every step; the KV caches rotate over enough distinct sets (and the target
    logits over four buffers) that consecutive steps never find them in L2."""

    def __init__(self, s, flags=0, extra_ctx=0, weights=None):
        import numpy as np  # noqa: F401

        import paper_2410_05589_b200 as ps
        import synth

        self.ps, self.s = ps, s
        B, R, V = s.batch, s.rows, s.vocab
        self.B, self.R = B, R
        self.lens = synth.ctx_lengths(s, B)
        W = weights if weights is not None else synth.weights(s)
        kv_bytes_seq = 2 * s.n_kv_heads * s.head_dim * int(self.lens.mean()) * (4 if s.dtype == 0 else 2)
        n_sets = 1 if kv_bytes_seq * B > 2 * L2_BYTES else max(2, min(16, -(-2 * L2_BYTES // max(1, kv_bytes_seq * B))))
        self.n_sets = n_sets = max(1, min(n_sets, 128 // B))
        self.max_ctx = int(self.lens.max()) + R + extra_ctx
        self.g = ps.drafter_from_shape(s, W, max_batch=B * n_sets, max_ctx=self.max_ctx, flags=flags)
        for b in range(B):
            K, Vv = synth.kv_rows(s, ("kv", b), int(self.lens[b]))
            Kd, Vd = ps.to_device(K), ps.to_device(Vv)
            for i in range(n_sets):
                self.g.kv_import(i * B + b, Kd, Vd)
        self.hl_np, self.tl_np = synth.hidden_states(s, "last", B), synth.token_ids(s, "last", B)
        self.tgt_np = [(synth.zipf_logits(s.seed, f"tgt{i}", B, R, V) if s.logits_kind == "zipf"
                        else synth.gauss_logits(s.seed, f"tgt{i}", (B, R, V))) for i in range(min(max(n_sets, 2), 4))]
        self.hl, self.tl = ps.to_device(self.hl_np), ps.to_device(self.tl_np)
        self.tgt = [ps.to_device(t) for t in self.tgt_np]
        self.slots = [[i * B + b for b in range(B)] for i in range(n_sets)]
        self.d_out, self.v_out = {}, {}

    def step(self, i, T):
        g, B, R = self.g, self.B, self.R
        if T > 0:
            o = g.draft_step_sampled(self.slots[i % self.n_sets], self.hl, self.tl, T, 1, i, top_n=1,
                                     want_logits=True, out=self.d_out)
            g.verify(o["sampled"], o["logits"], self.tgt[i % len(self.tgt)], T, 1, i, out=self.v_out)
        else:
            o = g.draft_step(self.slots[i % self.n_sets], self.hl, self.tl, top_n=1, want_logits=True, out=self.d_out)
            g.verify(o["top_ids"].view(B, R), None, self.tgt[i % len(self.tgt)], 0.0, 1, i, out=self.v_out)

    def timed(self, steps, T, warmup=5):
        """Milliseconds of `steps` back-to-back steps (CUDA events on the launching stream)."""
        import torch
        for i in range(warmup):
            self.step(i, T)
        torch.cuda.synchronize()
        e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
        e0.record()
        for i in range(steps):
            self.step(i, T)
        e1.record()
        torch.cuda.synchronize()
        return e0.elapsed_time(e1)

    def stage_profile(self, n, T, peak, per_launch=False):
        """Per-stage time per step (events recorded by the library between stages: no overlap
        between consecutive kernels, so the stages add up to more than a timed step) and GB/s of
        the stage's algorithmic bytes.  per_launch: an event after every launch instead, so that
        stages that share a launch (up to 16 rows: fc + q|k|v, and o + gate|up + down + LM head)
        are timed as the launch they are."""
        import torch
        self.g.profile(2 if per_launch else 1)
        for i in range(2):   # the kernels of this mode load and warm up outside the record
            self.step(i, T)
        torch.cuda.synchronize()
        self.g.profile_read()
        for i in range(n):
            self.step(i, T)
        torch.cuda.synchronize()
        prof = self.g.profile_read()
        self.g.profile(0)
        sb = stage_bytes(self.s, self.B, self.lens)
        if per_launch:
            sb = dict(sb)
            for name, parts in LAUNCH_STAGES.items():
                sb[name] = sum(sb[p] for p in parts)
        stages = {}
        for name, (tot, cnt) in prof.items():
            if cnt and name in sb:
                us = tot / n * 1e3   # per step: a batch beyond 128 rows runs a stage several times a step
                gbs = sb[name] / (us * 1e-6) / 1e9
                stages[name] = {"us": round(us, 2), "gbs": round(gbs, 1), "frac_of_peak": round(gbs / peak, 4),
                                "launches_per_step": round(cnt / n, 2)}
        return stages, sb

    def summary(self, steps, T, peak, n_prof=40):
        """ms per step, bytes, fractions of the roofline and the stage table of this workload."""
        ms = self.timed(steps, T) / steps
        stages, sb = self.stage_profile(n_prof, T, peak)
        total = sum(sb.values())
        gbs = total / (ms * 1e-3) / 1e9
        return {"ms_per_step": round(ms, 5), "steps": steps, "temperature": T, "step_bytes": total,
                "step_gbs": round(gbs, 1), "hbm_frac_of_measured": round(gbs / peak, 4),
                "hbm_frac_of_nominal_8TBs": round(gbs / NOMINAL_HBM_GBS, 4),
                "drafted_tokens_per_s": round(self.B * self.R / (ms * 1e-3), 1), "stages": stages}

    def close(self):
        import torch
        self.g = None
        self.tgt = self.hl = self.tl = None
        self.d_out, self.v_out = {}, {}
        torch.cuda.empty_cache()


# A 26-node draft tree of the shape tree drafters use (4 children of the root, depth 6).
TREE26 = [-1, -1, -1, -1, 0, 0, 0, 1, 1, 2, 4, 4, 5, 7, 10, 10, 11, 12, 13, 14, 14, 16, 18, 19, 21, 22]


def tree_legs(w, T, peak, n_buf=6, reps=60):
    """Token-tree round (Algorithm 1 in full).  (1) ps_verify_tree alone on the 26-node tree:
    synthetic target rows per node, one draft row per depth (noisy copies, so that paths of several
    nodes are accepted), node tokens drawn from the draft rows; buffers rotate so that rows come
    from HBM.  (2) the whole round on the device: ps_draft_step (top-4) -> ps_build_tree ->
    ps_verify_tree."""
    import numpy as np
    import torch

    import synth
    g, ps, s, B = w.g, w.ps, w.s, w.B
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
    alone = {"us": round(us, 2), "nodes": n, "depth": D, "bytes": nbytes,
             "gbs": round(nbytes / (us * 1e-6) / 1e9, 1), "frac_of_peak": round(nbytes / (us * 1e-6) / 1e9 / peak, 4),
             "mean_accepted_nodes": float(out["accept_len"].float().mean().item()),
             "note": "(n+1) target rows and one draft row per row with children, each read once"}
    # the whole round on the device: the tree cut to the depths a draft step of k+1 rows gives
    keep = [i for i in range(n) if depth[i] < s.rows]
    renum = {old: new for new, old in enumerate(keep)}
    tree = [renum.get(TREE26[i], -1) for i in keep]
    rank = [sum(1 for j in range(i) if tree[j] == tree[i]) for i in range(len(tree))]
    Dt, nt = min(D, s.rows), len(tree)
    tgt_sets = [t[2][:, :nt + 1].contiguous() for t in sets]
    d_out, tok_out, t_out = {}, torch.empty((B, nt), dtype=torch.int32, device="cuda"), {}

    def tree_round(i):
        o = g.draft_step(w.slots[i % w.n_sets], w.hl, w.tl, top_n=4, want_logits=True, out=d_out)
        g.build_tree(tree, rank, o["top_ids"], out=tok_out)
        dl = o["logits"] if Dt == s.rows else o["logits"][:, :Dt].contiguous()
        g.verify_tree(tree, tok_out, dl, tgt_sets[i % n_buf], T, 1, i, out=t_out)

    for i in range(5):
        tree_round(i)
    torch.cuda.synchronize()
    f0, f1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
    f0.record()
    for i in range(reps):
        tree_round(i)
    f1.record()
    torch.cuda.synchronize()
    whole = {"ms_per_round": round(f0.elapsed_time(f1) / reps, 5), "rounds": reps, "nodes": nt, "depth": Dt,
             "note": "ps_draft_step (top-4) -> ps_build_tree -> ps_verify_tree, nothing on the host"}
    return alone, whole


def verify_alone_leg(w, T, peak, n_host=12, n_dev=144, reps=288):
    """ps_verify on its own in the acceptance regime of the paper's tables: draft logits = target
    + N(0, sigma^2) with sigma chosen for about 3.5 tokens a round at k = 4, drafts drawn from q on
    the host.  The logits rotate over `n_dev` device buffers (more than L2 holds), so every call
    reads its rows from HBM."""
    import numpy as np
    import torch

    import synth
    g, ps, s, B, R, V = w.g, w.ps, w.s, w.B, w.R, w.s.vocab
    per_set = 2 * B * R * V * 4
    n_dev = max(4, min(n_dev, int(1.5 * L2_BYTES // per_set) + 1, (2 << 30) // per_set))
    host = []
    for i in range(min(n_host, n_dev)):
        tl = (synth.zipf_logits(s.seed, ("va_t", i), B, R, V) if s.logits_kind == "zipf"
              else synth.gauss_logits(s.seed, ("va_t", i), (B, R, V)))
        dl = synth.noisy_draft_logits(s.seed, ("va_d", i), tl, VERIFY_SIGMA)
        tk = synth.sample_from_logits(s.seed, ("va_x", i), dl, temperature=T if T > 0 else 1.0)
        if T == 0:
            tk = dl.argmax(-1).astype(np.int32)
        host.append((ps.to_device(tk.astype(np.int32)), ps.to_device(dl), ps.to_device(tl)))
    dev = [(host[i % len(host)][0], host[i % len(host)][1].clone(), host[i % len(host)][2].clone())
           for i in range(n_dev)]
    out = {}
    for i in range(8):
        tk, dl, tl = dev[i % n_dev]
        g.verify(tk, dl if T > 0 else None, tl, T, 1, i, out=out)
    torch.cuda.synchronize()
    n_out = 0.0
    e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
    acc = torch.zeros((), dtype=torch.float32, device="cuda")
    e0.record()
    for i in range(reps):
        tk, dl, tl = dev[i % n_dev]
        g.verify(tk, dl if T > 0 else None, tl, T, 1, 1000 + i, out=out)
    e1.record()
    torch.cuda.synchronize()
    us = e0.elapsed_time(e1) / reps * 1e3
    for i in range(min(reps, 4 * len(host))):     # acceptance statistics (untimed)
        tk, dl, tl = dev[i % n_dev]
        g.verify(tk, dl if T > 0 else None, tl, T, 1, 5000 + i, out=out)
        acc += out["n_out"].float().mean()
        n_out += 1
    torch.cuda.synchronize()
    nbytes = (8 if T > 0 else 4) * B * R * V
    return {"us": round(us, 2), "bytes": nbytes, "gbs": round(nbytes / (us * 1e-6) / 1e9, 1),
            "frac_of_peak": round(nbytes / (us * 1e-6) / 1e9 / peak, 4),
            "mean_tokens_per_round": round(float(acc.item()) / n_out, 3), "sigma": VERIFY_SIGMA,
            "buffers": n_dev, "buffer_bytes_total": n_dev * per_set, "temperature": T,
            "note": "ps_verify alone, n_draft = n_target = k+1, logits read from HBM (buffers rotate over more than L2)"}


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
    peak, peak_kind = measured_peak()

    s = workload_shape(args)
    T = args.temperature
    w = Workload(s, flags=args.flags, extra_ctx=64)   # + room for the groups of the training-layout leg
    g, B, R, V = w.g, w.B, w.R, s.vocab
    lens = w.lens

    # ---- headline: K timed steps after W warm-up steps, barrier + synchronize on both sides -----
    for i in range(max(3, args.warmup)):
        w.step(i, T)
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
        w.step(i, T)
    e1.record()
    torch.cuda.synchronize()
    launches = g.launch_count() - l0
    clocks = sampler.stop()
    if world > 1:
        dist.barrier()
    ms = max_over_ranks(e0.elapsed_time(e1))
    assert g.poll() == 0, "device status word set during the timed region"
    n_accept = float(w.v_out["n_out"].float().mean().item())

    # ---- steady state: the same step for at least a second, clocks sampled meanwhile ------------
    per = ms / args.steps
    n_steady = int(min(20000, max(args.steps, 1100.0 / max(per, 1e-3))))
    sampler2 = ClockSampler(local)
    sampler2.start()
    ms_steady = w.timed(n_steady, T, warmup=3)
    steady = {"ms_per_step": round(ms_steady / n_steady, 5), "steps": n_steady, "seconds": round(ms_steady * 1e-3, 3),
              "clocks": sampler2.stop()}

    # ---- per-stage times and the roofline of the slowest stage's kernel -------------------------
    n_prof = min(max(args.steps, 20), 200)
    stages, sb = w.stage_profile(n_prof, T, peak)
    step_bytes = sum(sb.values())
    # the launches as the timed steps make them (stages that share a launch timed together)
    by_launch, lb = w.stage_profile(n_prof, T, peak, per_launch=True)
    dom = max(by_launch, key=lambda k: by_launch[k]["us"]) if by_launch else None
    roofline = None
    if dom:
        per_launch_us = by_launch[dom]["us"] / max(by_launch[dom]["launches_per_step"], 1.0)
        roofline = {
            "bound": "hbm", "kernel": kernel_of_stage(dom, B * R), "stage": dom,
            "achieved": by_launch[dom]["gbs"], "peak": peak, "unit": "GB/s",
            "frac": round(by_launch[dom]["gbs"] / peak, 4),
            "traffic": captured_dram_bytes(args.workload, B, s.k_masks, dom),
            "peak_kind": f"of {peak_kind}", "bytes_per_launch": lb[dom], "us_per_launch": round(per_launch_us, 2),
            "note": "the step's longest launch, events between launches (no overlap with its neighbours); "
                    "the step-level fractions are hbm_frac_of_*",
        }

    # ---- the other temperature of the headline workload (Table 1 has T = 0 and T = 1) -----------
    T_other = 0.0 if T > 0 else 1.0
    n_o = min(args.steps, 300)
    ms_o = w.timed(n_o, T_other) / n_o
    other_T = {"temperature": T_other, "ms_per_step": round(ms_o, 5), "steps": n_o,
               "step_gbs": round(step_bytes / (ms_o * 1e-3) / 1e9, 1),
               "hbm_frac_of_measured": round(step_bytes / (ms_o * 1e-3) / 1e9 / peak, 4),
               "note": "arg-max drafts + greedy verify" if T_other == 0 else "drafts drawn from q + stochastic verify"}
    # arg-max drafts verified against the full q at T > 0: the faster but biased variant, for comparison
    argmax_T = None
    if T > 0:
        a_out = {}

        def step_argmax(i):
            o = g.draft_step(w.slots[i % w.n_sets], w.hl, w.tl, top_n=1, want_logits=True, out=a_out)
            g.verify(o["top_ids"].view(B, R), o["logits"], w.tgt[i % len(w.tgt)], T, 1, i, out=w.v_out)

        for i in range(5):
            step_argmax(i)
        torch.cuda.synchronize()
        f0, f1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
        f0.record()
        for i in range(n_o):
            step_argmax(i)
        f1.record()
        torch.cuda.synchronize()
        argmax_T = {"ms_per_step": round(f0.elapsed_time(f1) / n_o, 5), "steps": n_o,
                    "note": "ps_draft_step (arg-max drafts) + ps_verify with the full draft distribution: not lossless at T > 0"}

    # ---- verify alone in the paper's acceptance regime ------------------------------------------
    verify_alone = verify_alone_leg(w, T, peak) if s.vocab >= 1000 else None

    # ---- group-wise training layout, forward only (Sec. 4.1): groups on the first KV set --------
    group = None
    if int(lens.max()) + 64 + s.k_masks <= w.max_ctx:
        n_g = 64
        gh = ps.to_device(synth.hidden_states(s, "grp", n_g))
        gt = ps.to_device(synth.token_ids(s, "grp", n_g))
        for i in range(2):
            g.group_forward(int(w.slots[0][0]), gh, gt, top_n=1, want_logits=False)
        torch.cuda.synchronize()
        h0, h1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
        h0.record()
        for i in range(5):
            g.group_forward(int(w.slots[0][0]), gh, gt, top_n=1, want_logits=False)
        h1.record()
        torch.cuda.synchronize()
        group = {"ms_per_call": h0.elapsed_time(h1) / 5, "groups": n_g, "rows": n_g * R,
                 "note": "ps_group_forward; the groups run as draft steps of up to 128 rows per launch"}

    # ---- token-tree verification (Algorithm 1 in full) and the whole tree round -----------------
    tree, tree_round = (None, None)
    if V % 4 == 0 and V <= 131072 and s.dtype == 1 and s.k_masks >= 1:
        tree, tree_round = tree_legs(w, T, peak)

    # ---- end to end through the host-buffer entry point -----------------------------------------
    hl_h = torch.from_numpy(w.hl_np.view(np.int16) if w.hl_np.dtype == np.uint16 else w.hl_np).pin_memory()
    tl_h = torch.from_numpy(w.tl_np).pin_memory()
    tgt_h = [torch.from_numpy(t).pin_memory() for t in w.tgt_np]
    r_out = {}
    n_e2e = min(args.steps, 500)
    for i in range(3):
        g.round_host(w.slots[i % w.n_sets], hl_h, tl_h, tgt_h[i % len(tgt_h)], T, 1, i, out=r_out)
    torch.cuda.synchronize()
    if world > 1:
        dist.barrier()
    t0 = time.perf_counter()
    for i in range(n_e2e):
        g.round_host(w.slots[i % w.n_sets], hl_h, tl_h, tgt_h[i % len(tgt_h)], T, 1, i, out=r_out)
    torch.cuda.synchronize()
    e2e_s = max_over_ranks(time.perf_counter() - t0)
    eb = 4 if s.dtype == 0 else 2
    e2e = {"value": aggregate_steps_per_s(world, n_e2e, e2e_s * 1e3), "unit": "steps/s",
           "h2d_bytes_per_step": B * s.hidden * eb + B * 4 + B * R * V * 4,
           "d2h_bytes_per_step": B * (R + 3) * 4, "steps": n_e2e,
           "note": "ps_round_host: pinned host inputs up, results down and a stream wait, every step"}

    # ---- ps_kv_append (once per round, off the draft step's path): 4 accepted pairs a sequence ----
    n_new = 4
    ka_h = ps.to_device(synth.hidden_states(s, "app", B * n_new))
    ka_t = ps.to_device(synth.token_ids(s, "app", B * n_new))
    app_slots = w.slots[0]   # last leg on this context: these slots' contexts are not needed again

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
    hl_np, tl_np, tgt0 = w.hl_np, w.tl_np, w.tgt_np[0]
    w.close()

    # ---- the other workloads: step time, roofline fractions and the stage table of each --------
    configs = None
    if rank == 0 and world == 1 and not args.no_configs and args.workload == "13b" and args.batch == 0 \
            and args.k_masks < 0 and args.flags == 0:
        configs = {}
        n_c = min(max(args.steps, 20), 200)
        for name in ("7b", "33b"):
            wc = Workload(synth.CONFIGS[name])
            configs[wc.s.name] = dict(wc.summary(n_c, T, peak), config=workload_config(wc.s, wc.B, wc.lens, T)["workload"])
            wc.close()
        W13 = synth.weights(synth.CONFIGS["13b_sweep"])
        for Bc, kc in ((1, 2), (16, 4), (64, 8)):
            sc = synth.CONFIGS["13b_sweep"].with_(batch=Bc, k_masks=kc)
            Wc = dict(W13, mask_embed=W13["mask_embed"][:kc], mask_feat=W13["mask_feat"][:kc])
            wc = Workload(sc, weights=Wc)
            configs[f"13b_sweep_B{Bc}_k{kc}"] = dict(wc.summary(max(20, n_c // (1 + Bc // 8)), T, peak),
                                                   config=workload_config(sc, Bc, wc.lens, T)["workload"])
            wc.close()
        del W13

    cpu = None
    if rank == 0 and world == 1 and not args.no_cpu_baseline:
        cpu = cpu_baseline(s, B, lens, hl_np, tl_np, tgt0, T, args.cpu_seconds)

    if rank == 0:
        ms_per_step = ms / args.steps
        value = aggregate_steps_per_s(world, args.steps, ms)
        gbs = step_bytes / (ms_per_step * 1e-3) / 1e9
        line = {
            "metric": METRIC, "value": value, "unit": "steps/s", "n_gpus": world,
            "steps": args.steps, "warmup": max(3, args.warmup), "ms_per_step": ms_per_step,
            "higher_is_better": True, "scaling": "weak", "vs_baseline": None,
            "dtype": "f32" if s.dtype == 0 else "bf16", "data": "synthetic",
            "config": dict(workload_config(s, B, lens, T),
                           l2="weights exceed L2 and are streamed every step; KV caches rotate over "
                              f"{w.n_sets} distinct sets, target logits over {len(w.tgt_np)} buffers",
                           parallelism="replicas" if world > 1 else "single GPU", flags=args.flags),
            "drafted_tokens_per_s": value * B * R,
            "step_bytes": step_bytes, "step_gbs": round(gbs, 1),
            "hbm_frac_of_measured": round(gbs / peak, 4),
            "hbm_frac_of_nominal_8TBs": round(gbs / NOMINAL_HBM_GBS, 4),
            "mean_tokens_per_round": n_accept,
            "clocks": clocks, "e2e": e2e, "gpu_launches": int(launches),
            "roofline": roofline, "stages": stages, "launches": by_launch, "steady": steady, "other_temperature": other_T,
            "argmax_drafts": argmax_T, "verify_alone": verify_alone, "group_forward": group,
            "tree_verify": tree, "tree_round": tree_round, "kv_append": kv_append, "configs": configs,
            "cpu_baseline": cpu,
        }
        print(json.dumps(line))
    if world > 1:
        dist.destroy_process_group()


if __name__ == "__main__":
    main()

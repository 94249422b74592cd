"""Bench of the hybrid-batch attention hot path (plan once, run K steps) on synthetic batches.

    python bench.py [--gpus N] [--steps K] [--warmup W] [--workload NAME] [--impl reference]

One step = one pass of the whole hot path (attention kernel + split-KV merge) over one
synthetic hybrid batch.  Prints ONE JSON line.  `value` is useful TFLOP/s (masked-out work
excluded) with inputs resident in HBM; `kv_gbs` is K+V GB/s of the same runs; `e2e` repeats
the measurement through the public API with the step's inputs (the fused QKV of the new
tokens, block table, request table) coming from pinned host memory, the new K/V appended to
the paged cache, and O / LSE read back, host-side planning included.  The cached history is
device-resident state, as in serving.

`--impl reference` times the fp64 CPU oracle (as it stands) on a bounded sample of the same
workload on the host cores.
"""
from __future__ import annotations

import argparse
import json
import math
import os
import subprocess
import sys
import threading
import time

import numpy as np

ROOT = os.path.dirname(os.path.abspath(__file__))
if ROOT not in sys.path:
    sys.path.insert(0, ROOT)

SCALE = 1.0 / math.sqrt(128.0)
NOMINAL_TFLOPS = 2250.0
NOMINAL_GBS = 8000.0
FALLBACK_TFLOPS = 1590.0
FALLBACK_TFLOPS_SUSTAINED = 1400.0
FALLBACK_GBS = 6650.0


def measured_peaks():
    p = os.path.join(ROOT, "MEASURED_PEAKS.json")
    if os.path.exists(p):
        d = json.load(open(p))
        return {"hbm_gbs": float(d["hbm_gbs"]), "bf16_tflops": float(d["bf16_tflops"]),
                "bf16_tflops_sustained": float(d.get("bf16_tflops_sustained", d["bf16_tflops"])),
                "source": "measured"}
    return {"hbm_gbs": FALLBACK_GBS, "bf16_tflops": FALLBACK_TFLOPS,
            "bf16_tflops_sustained": FALLBACK_TFLOPS_SUSTAINED, "source": "fallback"}


class ClockSampler:
    """Samples SM clocks and throttle reasons with nvidia-smi while the timed region runs."""

    FIELDS = ("clocks.sm,clocks.max.sm,power.draw,clocks_event_reasons.hw_slowdown,"
              "clocks_event_reasons.hw_thermal_slowdown,clocks_event_reasons.sw_thermal_slowdown,"
              "clocks_event_reasons.sw_power_cap")

    def __init__(self, index: int):
        self.index = index
        self.proc = None
        self.lines = []

    def start(self):
        try:
            self.proc = subprocess.Popen(
                ["nvidia-smi", "-i", str(self.index), "--query-gpu=" + self.FIELDS,
                 "--format=csv,noheader,nounits", "-lms", "100"],
                stdout=subprocess.PIPE, stderr=subprocess.DEVNULL, text=True)
            self.thread = threading.Thread(target=self._read, daemon=True)
            self.thread.start()
        except OSError:
            self.proc = None

    def _read(self):
        for line in self.proc.stdout:
            self.lines.append(line.strip())

    def stop(self):
        if self.proc is None:
            return {"sm_mhz": None, "sm_max_mhz": None, "reasons": ["nvidia-smi unavailable"]}
        self.proc.terminate()
        try:
            self.proc.wait(timeout=5)
        except subprocess.TimeoutExpired:
            self.proc.kill()
        sm, mx, pw, reasons = [], [], [], set()
        names = ["hw_slowdown", "hw_thermal_slowdown", "sw_thermal_slowdown", "sw_power_cap"]
        for line in self.lines:
            parts = [x.strip() for x in line.split(",")]
            if len(parts) < 7:
                continue
            try:
                sm.append(float(parts[0]))
                mx.append(float(parts[1]))
                pw.append(float(parts[2]))
            except ValueError:
                continue
            for n, v in zip(names, parts[3:7]):
                if v.lower().startswith("active"):
                    reasons.add(n)
        if not sm:
            return {"sm_mhz": None, "sm_max_mhz": None, "reasons": ["no samples"]}
        return {"sm_mhz": float(np.median(sm)), "sm_max_mhz": float(max(mx)),
                "power_w_max": float(max(pw)), "samples": len(sm), "reasons": sorted(reasons)}


def dist_env():
    return int(os.environ.get("RANK", "0")), int(os.environ.get("LOCAL_RANK", "0")), int(os.environ.get("WORLD_SIZE", "1"))


def row_pairs(batch):
    """Allowed keys of every new-token row (pure counting): kv_len + i + 1 under the causal
    mask, kv_len + depth(i) under a tree mask (depth counts the node itself)."""
    out = []
    for r in range(batch.num_requests):
        n, h = int(batch.q_len[r]), int(batch.kv_len[r])
        par = batch.tree_parents(r)
        if par is None:
            out.append(h + 1 + np.arange(n, dtype=np.int64))
        else:
            depth = np.zeros(n, dtype=np.int64)
            for i in range(n):
                depth[i] = 1 if par[i] < 0 else depth[par[i]] + 1
            out.append(h + depth)
    return np.concatenate(out) if out else np.zeros(0, np.int64)


def pick_sample(batch, rng, target_pairs):
    """Rows (request, head, row) drawn uniformly over all (token, head) rows until their allowed
    (row, key) pairs reach `target_pairs`; returns the exact pair count of the sample."""
    T, Hq = batch.total_q, batch.num_q_heads
    q_start = batch.q_start
    req_of_tok = np.repeat(np.arange(batch.num_requests), batch.q_len)
    per_row = row_pairs(batch)
    order = rng.permutation(T * Hq)
    req, head, row, pairs = [], [], [], 0
    for x in order:
        t, a = divmod(int(x), Hq)
        r = int(req_of_tok[t])
        req.append(r)
        head.append(a)
        row.append(t - int(q_start[r]))
        pairs += int(per_row[t])
        if pairs >= target_pairs:
            break
    return np.array(req, np.int32), np.array(head, np.int32), np.array(row, np.int32), pairs


def host_cpu():
    """Core count and model string of the host the oracle is timed on."""
    model = "unknown"
    try:
        for line in open("/proc/cpuinfo"):
            if line.lower().startswith("model name"):
                model = line.split(":", 1)[1].strip()
                break
    except OSError:
        pass
    return {"nproc": os.cpu_count(), "model": model}


def time_oracle_full(batch, tensors):
    """The oracle over the whole workload, once (minutes on the large configurations)."""
    import oracle
    t0 = time.perf_counter()
    oracle.attention(batch, tensors, SCALE)
    dt = time.perf_counter() - t0
    pairs = int(row_pairs(batch).sum()) * batch.num_q_heads
    return {"tflops": 4.0 * batch.head_dim * pairs / dt / 1e12, "seconds": dt, "rows": batch.total_q * batch.num_q_heads,
            "pairs": pairs, "cores": oracle.num_threads()}


def time_oracle_sample(batch, tensors, seconds_target=12.0):
    """Times the oracle on a bounded random sample of output rows of the workload."""
    import oracle
    rng = np.random.default_rng(1234)
    # calibrate on a small sample, then size the real one for about `seconds_target`
    req, head, row, pairs = pick_sample(batch, rng, 2_000_000)
    t0 = time.perf_counter()
    oracle.attention_rows(batch, tensors, SCALE, req, head, row)
    dt = max(time.perf_counter() - t0, 1e-4)
    rate = pairs / dt
    req, head, row, pairs = pick_sample(batch, rng, int(rate * seconds_target))
    t0 = time.perf_counter()
    oracle.attention_rows(batch, tensors, SCALE, req, head, row)
    dt = time.perf_counter() - t0
    flops = 4.0 * batch.head_dim * pairs
    return {"tflops": flops / dt / 1e12, "seconds": dt, "rows": int(len(req)), "pairs": int(pairs),
            "cores": oracle.num_threads()}


def tree_pairs_note():
    return "pairs counted exactly per sampled row (kv_len + row + 1 causal, kv_len + depth for tree rows)"


def run_reference(args):
    rank, local_rank, world = dist_env()
    if rank != 0:
        return 0
    from paper_2412_18106_b200 import workloads as W
    batch = W.CONFIGS[args.workload](seed=0)
    tensors = W.make_tensors(batch)
    # each "step" is one bounded sample; warm-up steps are shorter
    per_step = max(2.0, min(12.0, 150.0 / max(1, args.steps + args.warmup)))
    for _ in range(args.warmup):
        time_oracle_sample(batch, tensors, per_step / 4)
    vals, secs, rows = [], 0.0, 0
    for _ in range(args.steps):
        r = time_oracle_sample(batch, tensors, per_step)
        vals.append(r["tflops"])
        secs += r["seconds"]
        rows = r["rows"]
        cores = r["cores"]
    v = float(np.mean(vals))
    line = {
        "impl": "reference", "metric": "hybrid_attention_useful_tflops", "value": v, "unit": "TFLOP/s",
        "n_gpus": args.gpus, "steps": args.steps, "warmup": args.warmup,
        "ms_per_step": 1e3 * secs / max(1, args.steps), "higher_is_better": True, "scaling": "weak",
        "vs_baseline": None, "dtype": "f64", "data": "synthetic",
        "config": workload_config(args.workload, batch),
        "cpu_baseline": {"value": v, "unit": "TFLOP/s", "cores": cores, "kind": "oracle", "host": host_cpu(),
                         "sample": "%d random output rows (request, head, token) of the workload per step; %s"
                                   % (rows, tree_pairs_note())},
        "e2e": {"value": v, "unit": "TFLOP/s", "h2d_bytes_per_step": 0, "d2h_bytes_per_step": 0},
    }
    print(json.dumps(line))
    return 0


# DRAM bytes (read + write) of one launch of the attention meta-kernel, from the ncu captures
# summarised under profiles/ (same workload, seed 0), each stamped with the commit of the kernel
# that was captured and the date; a kernel change that may move traffic needs a new capture.
NCU_TRAFFIC = {
    # full_mix: the 5 GB pool is beyond what a multi-pass capture should hold; the dense path and the
    # queue order that decide its traffic have not changed since this capture
    "full_mix": {"bytes": 6.00e9, "commit": "29136c8", "date": "2026-11-24", "summary": "profiles/launch_list_full_mix.md"},
    "splitfuse_mix": {"bytes": 1.666e9, "commit": "e5bad30", "date": "2026-11-25",
                      "summary": "profiles/meta_attention_splitfuse_mix.md"},
    "verify_trees": {"bytes": 2.503e9, "commit": "e5bad30", "date": "2026-11-25",
                     "summary": "profiles/meta_attention_verify_trees.md"},
    "decode_only": {"bytes": 0.593e9, "commit": "e5bad30", "date": "2026-11-25",
                    "summary": "profiles/meta_attention_decode_only.md"},
    "long_context_decode": {"bytes": 3.202e9, "commit": "29136c8", "date": "2026-11-24",
                            "summary": "profiles/meta_attention_long_context_decode.md"},
}


def ncu_traffic(name):
    e = NCU_TRAFFIC.get(name)
    return (e["bytes"], "ncu, commit %s, %s (%s)" % (e["commit"], e["date"], e["summary"])) if e else (None, None)


def workload_config(name, batch):
    """The `config` object both arms print for a workload (same keys, so the two lines compare)."""
    return {"workload": name, "num_requests": batch.num_requests, "total_q_tokens": batch.total_q,
            "q_heads": batch.num_q_heads, "kv_heads": batch.num_kv_heads, "page_size": batch.page_size,
            "kv_tokens": int((batch.q_len + batch.kv_len).sum())}


def roofline_entry(flops, alg_bytes, kernel_ms, merge_ms, peaks, clocks):
    """Everything needed to recompute a configuration's roofline fraction: the algorithmic work,
    the measured kernel time and the fraction against every candidate peak.  The headline `frac`
    uses the measured peak that matches the clocks seen during the timed region: the burst bf16
    figure when the median SM clock stayed within 10 % of the maximum, else the sustained one (HBM
    bound: the measured copy bandwidth either way)."""
    t = kernel_ms * 1e-3
    sm, mx = (clocks or {}).get("sm_mhz"), (clocks or {}).get("sm_max_mhz")
    at_max = bool(sm and mx and sm >= 0.9 * mx)
    tf_peak = peaks["bf16_tflops"] if at_max else peaks["bf16_tflops_sustained"]
    t_flop, t_byte = flops / (tf_peak * 1e12), alg_bytes / (peaks["hbm_gbs"] * 1e9)
    tensor = t_flop >= t_byte
    e = {"bound": "tensor" if tensor else "hbm",
         "achieved": flops / t / 1e12 if tensor else alg_bytes / t / 1e9,
         "peak": tf_peak if tensor else peaks["hbm_gbs"], "unit": "TFLOP/s" if tensor else "GB/s"}
    e["frac"] = e["achieved"] / e["peak"]
    e["peak_source"] = "%s (%s)" % (peaks["source"], ("burst bf16: median SM clock within 10% of max" if at_max else
                                                     "sustained bf16: SM clock below 0.9 max") if tensor else "copy")
    e["kernel_ms"], e["merge_ms"] = kernel_ms, merge_ms
    e["kernel_mcycles"] = kernel_ms * 1e-3 * sm if sm else None   # duration x median SM MHz
    e["algorithmic_flops"], e["algorithmic_bytes"] = flops, alg_bytes
    roof = lambda tf, gb: max(flops / (tf * 1e12), alg_bytes / (gb * 1e9))
    e["frac_burst"] = roof(peaks["bf16_tflops"], peaks["hbm_gbs"]) / t
    e["frac_sustained"] = roof(peaks["bf16_tflops_sustained"], peaks["hbm_gbs"]) / t
    e["frac_nominal"] = roof(NOMINAL_TFLOPS, NOMINAL_GBS) / t
    return e


def measure_other(name, kernel, dev, peaks, steps=20, warmup=3):
    """Short device-timed measurement of another benchmark configuration (same method as the
    primary one: inputs resident, CUDA events, KV pool far larger than L2)."""
    import torch

    from paper_2412_18106_b200 import binding as xb
    from paper_2412_18106_b200 import workloads as W
    batch = W.CONFIGS[name](seed=0)
    tensors = W.make_tensors(batch)
    ctx = xb.XYAttn(batch.num_q_heads, batch.num_kv_heads, batch.page_size, device=dev.index, kernel=kernel,
                    max_requests=max(256, batch.num_requests), max_q_tokens=max(1 << 15, batch.total_q),
                    max_pages_per_req=max(1024, batch.block_table.shape[1]),
                    max_tree_nodes=max(64, int(batch.q_len.max())))
    info = ctx.plan_batch(batch)
    q, k_pool, v_pool = tensors.q.to(dev), tensors.k_pool.to(dev), tensors.v_pool.to(dev)
    bt = torch.from_numpy(np.where(batch.block_table < 0, 0, batch.block_table).astype(np.int32)).to(dev)
    o = torch.empty((batch.total_q, batch.num_q_heads, batch.head_dim), dtype=torch.bfloat16, device=dev)
    lse = torch.empty((batch.total_q, batch.num_q_heads), dtype=torch.float32, device=dev)
    e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
    e0.record()
    for _ in range(warmup):
        ctx.run(q, k_pool, v_pool, bt, SCALE, o, lse)
    e1.record()
    torch.cuda.synchronize()
    # enough steps for the clock sampler to see the timed region (about 0.4 s), at most 4000
    steps = int(min(4000, max(steps, 400.0 / max(e0.elapsed_time(e1) / warmup, 1e-3))))
    sampler = ClockSampler(dev.index)
    sampler.start()
    time.sleep(0.25)
    ctx.set_timing(True)
    e0.record()
    for _ in range(steps):
        ctx.run(q, k_pool, v_pool, bt, SCALE, o, lse)
    e1.record()
    torch.cuda.synchronize()
    clocks = sampler.stop()
    ms = e0.elapsed_time(e1) / steps
    attn_ms, merge_ms, runs = ctx.get_timing()
    assert ctx.device_status() == 0
    ctx.close()
    flops, alg = float(info.useful_flops), float(W.algorithmic_bytes(batch))
    e = roofline_entry(flops, alg, attn_ms / max(1, runs), merge_ms / max(1, runs), peaks, clocks)
    e.update({"ms_per_step": ms, "tflops": flops / (ms * 1e-3) / 1e12, "kv_gbs": float(info.kv_bytes) / (ms * 1e-3) / 1e9,
              "steps": steps, "tasks": info.num_tasks, "merge_units": info.num_merge_units,
              "clocks": {k: clocks.get(k) for k in ("sm_mhz", "sm_max_mhz", "reasons")}})
    e["traffic"], e["traffic_source"] = ncu_traffic(name)
    return e


def measure_stream(kernel, dev, peaks, chunks=48, budget=4096, reserved=512, sessions=96, seed=0):
    """A serving-like request stream through the scheduling front (Section 3.1): sessions arrive
    with prompts (prefix-cache hits included), then decode one token per step, a fifth of them
    verify a token tree instead; the chunk former cuts fixed-budget chunks, every chunk is planned
    (Task-Table cache on) and run.  K/V pool and Q are random and resident; the block table maps
    every session onto random pages of one pool (contents do not matter for timing).  Reports the
    host time of chunk forming and planning (the C calls, chunk handed from one to the other as
    the request array) and the device time of attention per chunk."""
    import torch

    from paper_2412_18106_b200 import binding as xb
    from paper_2412_18106_b200 import sched as xs
    from paper_2412_18106_b200 import workloads as W
    rng = np.random.default_rng(seed)
    Hq, Hkv, B, D = 32, 8, 128, 128
    max_kv = 12288
    pages_per_req = max_kv // B + 1
    num_pages = 6144  # 2 x 1.6 GB of K/V: far beyond L2
    g = torch.Generator(device=dev).manual_seed(seed)
    k_pool = torch.randn((num_pages, Hkv, B, D), device=dev, generator=g).to(torch.bfloat16)
    v_pool = torch.randn((num_pages, Hkv, B, D), device=dev, generator=g).to(torch.bfloat16)
    q = torch.randn((budget, Hq, D), device=dev, generator=g).to(torch.bfloat16)
    o = torch.empty((budget, Hq, D), dtype=torch.bfloat16, device=dev)
    lse = torch.empty((budget, Hq), dtype=torch.float32, device=dev)
    cap = 256
    ctx = xb.XYAttn(Hq, Hkv, B, device=dev.index, kernel=kernel, max_requests=cap, max_q_tokens=budget,
                    max_pages_per_req=pages_per_req, max_tree_nodes=64)
    sch = xs.XYSched(budget, reserved, cap)
    bt_all = torch.from_numpy(rng.integers(0, num_pages, size=(sessions, pages_per_req)).astype(np.int32))
    bt_dev = torch.zeros((cap, pages_per_req), dtype=torch.int32, device=dev)
    kv_of = {}
    for sid in range(sessions):
        prompt = int(round(math.exp(rng.uniform(math.log(256), math.log(4096)))))
        hit = int(prompt * rng.uniform(0.0, 0.9)) if rng.random() < 0.5 else 0
        sch.add_prefill(sid, prompt, min(hit, prompt - 1))
        kv_of[sid] = prompt
    t_sched = t_plan = 0.0
    flops = kvb = 0.0
    tokens = 0
    ctx.set_timing(True)
    e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
    done = 0
    e0.record()
    while done < chunks and sch.pending() != (0, 0):
        t0 = time.perf_counter()
        n, reqs_raw, ents_raw, par_raw, npar = sch.next_chunk_raw()
        t1 = time.perf_counter()
        info = ctx.plan_raw(reqs_raw, n, par_raw, npar)
        t3 = time.perf_counter()
        t2 = t1
        chunk = [dict(id=int(ents_raw[k].id), kind=int(ents_raw[k].kind), last=bool(ents_raw[k].last),
                      q_len=int(reqs_raw[k].q_len), kv_len=int(reqs_raw[k].kv_len)) for k in range(n)]
        ql = [e["q_len"] for e in chunk]
        rows = torch.tensor([e["id"] for e in chunk], dtype=torch.long)
        bt_dev[: len(chunk)].copy_(bt_all[rows], non_blocking=False)
        T = int(sum(ql))
        ctx.run(q[:T], k_pool, v_pool, bt_dev, SCALE, o[:T], lse[:T])
        t_sched += t1 - t0
        t_plan += t3 - t2
        flops += float(info.useful_flops)
        kvb += float(info.kv_bytes)
        tokens += T
        done += 1
        # the serving loop: finished prompts and decoded / verified sessions come back
        for e in chunk:
            if not e["last"]:
                continue
            sid = e["id"]
            if e["kind"] != xs.XY_SCHED_PREFILL:
                kv_of[sid] = e["kv_len"] + (1 if e["kind"] == xs.XY_SCHED_DECODE else 3)
            if kv_of[sid] + 64 >= max_kv:
                continue
            if sid % 5 == 0:
                sch.add_verify(sid, kv_of[sid], W.random_tree(rng, int(rng.integers(4, 33)), 6))
            else:
                sch.add_decode(sid, kv_of[sid])
    e1.record()
    torch.cuda.synchronize()
    wall_ms = e0.elapsed_time(e1)
    attn_ms, merge_ms, runs = ctx.get_timing()
    assert ctx.device_status() == 0
    hits, misses = ctx.plan_cache()
    ctx.close()
    sch.close()
    # Where the Task-Table cache does earn hits: 64 steps of a pure decode phase (every request one
    # token further each step; a step misses only when some request enters a new 128-key tile).
    # Host-only context: the planner alone is timed.
    hctx = xb.XYAttn(64, 8, 128, device=-1, num_workers=148, max_requests=256)
    hctx.plan_cache(64)
    kv0 = np.random.default_rng(1).integers(512, 8192, size=64)
    t_hit, t_miss = [], []
    for step in range(64):
        h_before = hctx.plan_cache()[0]
        t0 = time.perf_counter()
        hctx.plan([1] * 64, list(kv0 + step), [0] * 64, [-1] * 64)
        dt = time.perf_counter() - t0
        (t_hit if hctx.plan_cache()[0] > h_before else t_miss).append(dt)
    dh, dm = hctx.plan_cache()
    hctx.close()
    decode_phase = {"requests": 64, "steps": 64, "hits": dh, "misses": dm,
                    "plan_us_hit": 1e6 * float(np.median(t_hit)) if t_hit else None,
                    "plan_us_miss": 1e6 * float(np.median(t_miss)) if t_miss else None}
    n = max(1, done)
    return {"chunks": done, "budget_tokens": budget, "reserved_dv_tokens": reserved, "sessions": sessions,
            "tokens": tokens, "sched_us_per_chunk": 1e6 * t_sched / n, "plan_us_per_chunk": 1e6 * t_plan / n,
            "attn_ms_per_chunk": (attn_ms + merge_ms) / n, "wall_ms_per_chunk": wall_ms / n,
            "tflops_attention": flops / ((attn_ms + merge_ms) * 1e-3) / 1e12,
            "kv_gbs_attention": kvb / ((attn_ms + merge_ms) * 1e-3) / 1e9,
            "task_table_cache": {"hits": hits, "misses": misses, "decode_phase": decode_phase}}


def measure_gemm(dev, peaks, steps=20):
    """SmoothGEMM (Section 5) on the Linear shapes of the benchmark model (hidden 4096, 32 + 2 x 8
    heads of 128, MLP 14336) for token counts from a decode batch to a full chunk.  Device-timed
    back-to-back launches (the smallest cases are bound by launch latency, not by the kernel).
    `frac`: the roofline time (flops at the measured burst bf16 peak, each kernel being timed alone, or
    the bytes of A + W + C once at the measured copy bandwidth, whichever is longer) over the
    measured time.  `lib_us`: the library GEMM (torch.matmul) timed beside it, for context."""
    import torch

    from paper_2412_18106_b200 import gemm as xg
    out = {}
    ws = xg.xy_gemm_workspace(dev)  # scratch for the split of a thin last wave (long K only)
    for name, N, K in (("qkv", 6144, 4096), ("oproj", 4096, 4096), ("gate_up", 28672, 4096), ("down", 4096, 14336)):
        g = torch.Generator(device=dev).manual_seed(N + K)
        w = torch.randn((N, K), device=dev, generator=g).to(torch.bfloat16)
        for M in (16, 256, 4096):
            a = torch.randn((M, K), device=dev, generator=g).to(torch.bfloat16)
            c = torch.empty((M, N), dtype=torch.bfloat16, device=dev)

            def timed(fn):
                for _ in range(3):
                    fn()
                torch.cuda.synchronize()
                e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
                e0.record()
                for _ in range(steps):
                    fn()
                e1.record()
                torch.cuda.synchronize()
                return e0.elapsed_time(e1) / steps
            ms = timed(lambda: xg.xy_gemm_run(a, w, c, workspace=ws))
            ms_lib = timed(lambda: torch.matmul(a, w.T, out=c))
            flops, byts = 2.0 * M * N * K, 2.0 * (M * K + N * K + M * N)
            t_roof = max(flops / (peaks["bf16_tflops"] * 1e12), byts / (peaks["hbm_gbs"] * 1e9))
            out["%s_M%d" % (name, M)] = {"us": round(ms * 1e3, 1), "tflops": round(flops / ms / 1e9, 1),
                                         "frac": round(t_roof / (ms * 1e-3), 3), "lib_us": round(ms_lib * 1e3, 1)}
    assert xg.xy_gemm_device_status() == 0
    return out


def measure_shared_prefix(kernel, dev, peaks, steps=20):
    """Shared-prefix ("cascade") decode: 4 groups of 32 decode requests, each group sharing an
    8192-token cached prefix (same pages), 0..1024 own tokens per request, 32/8 heads.  Times the
    plain plan (every request reads its whole history) and the grouped plan (the shared keys are
    read once per group by dense tiles).  The roofline fraction of the grouped plan counts the
    bytes that must be read at least once: the shared prefixes once per group plus every
    member's own keys."""
    import torch

    from paper_2412_18106_b200 import binding as xb
    from paper_2412_18106_b200 import workloads as W
    batch, groups = W.shared_prefix_decode(seed=0)
    tensors = W.make_tensors(batch)
    q, k_pool, v_pool = tensors.q.to(dev), tensors.k_pool.to(dev), tensors.v_pool.to(dev)
    bt = torch.from_numpy(np.where(batch.block_table < 0, 0, batch.block_table).astype(np.int32)).to(dev)
    o = torch.empty((batch.total_q, batch.num_q_heads, batch.head_dim), dtype=torch.bfloat16, device=dev)
    lse = torch.empty((batch.total_q, batch.num_q_heads), dtype=torch.float32, device=dev)
    per_token = 2 * batch.num_kv_heads * batch.head_dim * 2
    unique = sum(g[2] for g in groups) * per_token
    in_group = np.zeros(batch.num_requests, bool)
    for first, n, prefix in groups:
        in_group[first: first + n] = True
        unique += int((batch.kv_len[first: first + n] + 1 - prefix).sum()) * per_token
    unique += int((batch.kv_len[~in_group] + 1).sum()) * per_token
    out = {"requests": batch.num_requests, "groups": len(groups), "prefix_tokens": groups[0][2],
           "unique_kv_bytes": unique}
    for name, gs in (("plain", None), ("grouped", groups)):
        ctx = xb.XYAttn(batch.num_q_heads, batch.num_kv_heads, batch.page_size, device=dev.index, kernel=kernel,
                        max_requests=512, max_q_tokens=1 << 15, max_pages_per_req=max(1024, batch.block_table.shape[1]))
        info = ctx.plan_batch(batch, groups=gs)
        for _ in range(3):
            ctx.run(q, k_pool, v_pool, bt, SCALE, o, lse)
        torch.cuda.synchronize()
        ctx.set_timing(True)
        for _ in range(steps):
            ctx.run(q, k_pool, v_pool, bt, SCALE, o, lse)
        attn_ms, merge_ms, runs = ctx.get_timing()
        assert ctx.device_status() == 0
        ctx.close()
        k_ms, m_ms = attn_ms / runs, merge_ms / runs
        out[name] = {"kernel_ms": k_ms, "merge_ms": m_ms, "tasks": info.num_tasks, "merge_units": info.num_merge_units,
                     "kv_bytes_read_per_request": int(info.kv_bytes)}
    out["speedup"] = (out["plain"]["kernel_ms"] + out["plain"]["merge_ms"]) / (out["grouped"]["kernel_ms"] + out["grouped"]["merge_ms"])
    out["grouped"]["roofline_frac_measured"] = unique / (peaks["hbm_gbs"] * 1e9) / (out["grouped"]["kernel_ms"] * 1e-3)
    return out


def measure_fp8_decode(dev, peaks, steps=200):
    """decode_only with an fp8 (e4m3) KV cache: the same requests, K and V stored as bytes with one
    fp32 scale per page and kv head.  The HBM roofline counts the fp8 bytes (half of bf16) plus
    scales, Q, O, LSE and block-table entries."""
    import torch

    from paper_2412_18106_b200 import binding as xb
    from paper_2412_18106_b200 import workloads as W
    batch = W.CONFIGS["decode_only"](seed=0)
    t8 = W.to_fp8_kv(W.make_tensors(batch))
    q, k8, v8 = t8.q.to(dev), t8.k_pool.to(dev), t8.v_pool.to(dev)
    ks, vs = t8.k_scale.to(dev), t8.v_scale.to(dev)
    bt = torch.from_numpy(np.where(batch.block_table < 0, 0, batch.block_table).astype(np.int32)).to(dev)
    o = torch.empty((batch.total_q, batch.num_q_heads, batch.head_dim), dtype=torch.bfloat16, device=dev)
    lse = torch.empty((batch.total_q, batch.num_q_heads), dtype=torch.float32, device=dev)
    ctx = xb.XYAttn(batch.num_q_heads, batch.num_kv_heads, batch.page_size, device=dev.index,
                    max_pages_per_req=max(1024, batch.block_table.shape[1]), kv_dtype=xb.XY_KV_FP8_E4M3)
    info = ctx.plan_batch(batch)
    for _ in range(5):
        ctx.run_fp8kv(q, k8, v8, ks, vs, bt, SCALE, o, lse)
    torch.cuda.synchronize()
    ctx.set_timing(True)
    for _ in range(steps):
        ctx.run_fp8kv(q, k8, v8, ks, vs, bt, SCALE, o, lse)
    attn_ms, merge_ms, runs = ctx.get_timing()
    assert ctx.device_status() == 0
    ctx.close()
    pages = int(((batch.q_len + batch.kv_len + batch.page_size - 1) // batch.page_size).sum())
    alg = float(info.kv_bytes) + 2.0 * pages * batch.num_kv_heads * 4 + (W.algorithmic_bytes(batch) - W.kv_bytes(batch))
    k_ms = attn_ms / runs
    return {"kernel_ms": k_ms, "merge_ms": merge_ms / runs, "kv_bytes_fp8": int(info.kv_bytes), "algorithmic_bytes": alg,
            "gbs": alg / (k_ms * 1e-3) / 1e9, "bound": "hbm", "roofline_frac_measured": alg / (peaks["hbm_gbs"] * 1e9) / (k_ms * 1e-3),
            "note": "bound by the e4m3 -> f16 conversion unit (16 results / clk / SM), not by HBM"}


def measure_long_decode(kernel, dev, peaks, steps=20):
    """Long-context decode: 4 requests with 128k - 512k cached tokens, 32/8 heads, page 128.  Every
    (request, kv head) row is cut into up to 32 key ranges handled by different workers and the
    partials are merged by the second kernel.  The pools are random and generated on the device
    (contents do not matter for timing); the roofline counts every cached K/V byte once."""
    import torch

    from paper_2412_18106_b200 import binding as xb
    from paper_2412_18106_b200 import workloads as W
    batch = W.long_context_decode(seed=0)
    g = torch.Generator(device=dev).manual_seed(0)
    shape = (batch.num_pages, batch.num_kv_heads, batch.page_size, batch.head_dim)
    k_pool = torch.empty(shape, dtype=torch.bfloat16, device=dev)
    v_pool = torch.empty(shape, dtype=torch.bfloat16, device=dev)
    step_pages = 2048
    for pool in (k_pool, v_pool):
        for p0 in range(0, batch.num_pages, step_pages):
            n = min(step_pages, batch.num_pages - p0)
            pool[p0: p0 + n] = torch.randn((n,) + shape[1:], device=dev, generator=g).to(torch.bfloat16)
    q = torch.randn((batch.total_q, batch.num_q_heads, batch.head_dim), device=dev, generator=g).to(torch.bfloat16)
    bt = torch.from_numpy(np.where(batch.block_table < 0, 0, batch.block_table).astype(np.int32)).to(dev)
    o = torch.empty((batch.total_q, batch.num_q_heads, batch.head_dim), dtype=torch.bfloat16, device=dev)
    lse = torch.empty((batch.total_q, batch.num_q_heads), dtype=torch.float32, device=dev)
    ctx = xb.XYAttn(batch.num_q_heads, batch.num_kv_heads, batch.page_size, device=dev.index, kernel=kernel,
                    max_requests=256, max_q_tokens=1 << 15, max_pages_per_req=batch.block_table.shape[1])
    info = ctx.plan_batch(batch)
    for _ in range(3):
        ctx.run(q, k_pool, v_pool, bt, SCALE, o, lse)
    torch.cuda.synchronize()
    ctx.set_timing(True)
    for _ in range(steps):
        ctx.run(q, k_pool, v_pool, bt, SCALE, o, lse)
    attn_ms, merge_ms, runs = ctx.get_timing()
    assert ctx.device_status() == 0
    ctx.close()
    # Every output row against the plain SIMT kernel (independent device code, same inputs), with
    # bounds that scale with the signal: two bf16 roundings of O apart, fp32 LSE.
    ref = xb.XYAttn(batch.num_q_heads, batch.num_kv_heads, batch.page_size, device=dev.index,
                    kernel=xb.XY_KERNEL_REFERENCE, max_requests=256, max_q_tokens=1 << 15,
                    max_pages_per_req=batch.block_table.shape[1])
    ref.plan_batch(batch)
    o_r, lse_r = torch.empty_like(o), torch.empty_like(lse)
    ref.run(q, k_pool, v_pool, bt, SCALE, o_r, lse_r)
    torch.cuda.synchronize()
    ref.close()
    err = (o.float() - o_r.float()).norm(dim=-1)
    row_rel = float((err / (o_r.float().norm(dim=-1) + 1e-4 * 2 ** 6)).max())
    lse_rel = float(((lse - lse_r).abs() / lse_r.abs().clamp(min=1.0)).max())
    assert row_rel <= 2.0 ** -6 and lse_rel <= 4e-5, ("long-context decode disagrees with the SIMT kernel", row_rel, lse_rel)
    alg = float(W.algorithmic_bytes(batch))
    k_ms, m_ms = attn_ms / runs, merge_ms / runs
    return {"requests": batch.num_requests, "kv_tokens": [int(x) for x in batch.kv_len], "tasks": info.num_tasks,
            "merge_units": info.num_merge_units, "kernel_ms": k_ms, "merge_ms": m_ms,
            "kv_gbs": float(info.kv_bytes) / (k_ms * 1e-3) / 1e9, "bound": "hbm",
            "roofline_frac_measured": alg / (peaks["hbm_gbs"] * 1e9) / (k_ms * 1e-3), "steps": steps,
            "check": {"against": "SIMT kernel, every row", "o_row_rel_max": row_rel, "lse_rel_max": lse_rel}}


def self_launch(n):
    """`--gpus N` without a launcher: start N ranks of this script, one process per GPU, with the
    rendezvous variables torch.distributed reads; rank 0 prints the line.  NCCL's communicator log
    (which transport and algorithms it picked) goes to stderr."""
    import socket
    with socket.socket() as sk:
        sk.bind(("127.0.0.1", 0))
        port = sk.getsockname()[1]
    procs = []
    for r in range(n):
        env = dict(os.environ, RANK=str(r), LOCAL_RANK=str(r), WORLD_SIZE=str(n), MASTER_ADDR="127.0.0.1",
                   MASTER_PORT=str(port))
        env.setdefault("NCCL_DEBUG", "INFO")
        env.setdefault("NCCL_DEBUG_SUBSYS", "INIT")
        procs.append(subprocess.Popen([sys.executable, os.path.abspath(__file__)] + sys.argv[1:], env=env,
                                      stdout=None if r == 0 else subprocess.DEVNULL))
    return max(p.wait() for p in procs)


def main():
    ap = argparse.ArgumentParser()
    ap.add_argument("--gpus", type=int, default=1)
    ap.add_argument("--steps", type=int, default=50)
    ap.add_argument("--warmup", type=int, default=5)
    ap.add_argument("--impl", default="ours", choices=["ours", "reference"])
    ap.add_argument("--workload", default="full_mix",
                    choices=["decode_only", "splitfuse_mix", "verify_trees", "full_mix", "tiny_hybrid",
                             "prefill_prefix", "long_context_decode"])
    ap.add_argument("--kernel", default="auto", choices=["auto", "reference", "mma"])
    ap.add_argument("--no-cpu-baseline", action="store_true")
    ap.add_argument("--cpu-full", action="store_true",
                    help="time the oracle on the whole workload once instead of a bounded sample (minutes)")
    ap.add_argument("--no-e2e", action="store_true")
    ap.add_argument("--no-others", action="store_true",
                    help="skip the short extra measurements of the other benchmark configurations")
    args = ap.parse_args()
    if args.impl == "reference":
        return run_reference(args)
    if args.gpus > 1 and "WORLD_SIZE" not in os.environ:
        return self_launch(args.gpus)

    import torch
    import torch.distributed as dist

    from paper_2412_18106_b200 import binding as xb
    from paper_2412_18106_b200 import workloads as W

    rank, local_rank, world = dist_env()
    assert torch.cuda.is_available(), "bench.py needs a CUDA device (there is no CPU path)"
    torch.cuda.set_device(local_rank)
    dev = torch.device("cuda", local_rank)
    if world > 1:
        dist.init_process_group("nccl", device_id=dev)

    warmup = max(3, args.warmup)
    # weak scaling: every rank serves its own batch of the same recipe (independent requests,
    # no exchange on the data path)
    batch = W.CONFIGS[args.workload](seed=rank)
    tensors = W.make_tensors(batch, fused_qkv=True)  # Q is read with a stride from [T, Hq + 2 Hkv, D]
    kernel = {"auto": xb.XY_KERNEL_AUTO, "reference": xb.XY_KERNEL_REFERENCE, "mma": xb.XY_KERNEL_MMA}[args.kernel]
    ctx = xb.XYAttn(batch.num_q_heads, batch.num_kv_heads, batch.page_size, device=local_rank,
                    kernel=kernel, max_requests=max(256, batch.num_requests),
                    max_q_tokens=max(1 << 15, batch.total_q),
                    max_pages_per_req=max(1024, batch.block_table.shape[1]),
                    max_tree_nodes=max(64, int(batch.q_len.max())))
    t0 = time.perf_counter()
    info = ctx.plan_batch(batch)
    plan_us = (time.perf_counter() - t0) * 1e6

    bt_host = torch.from_numpy(np.where(batch.block_table < 0, 0, batch.block_table).astype(np.int32))
    qkv_host = tensors.qkv.contiguous().pin_memory()
    bt_pin = bt_host.pin_memory()
    qkv = qkv_host.to(dev)
    q = qkv[:, : batch.num_q_heads, :]
    k_pool = tensors.k_pool.to(dev)
    v_pool = tensors.v_pool.to(dev)
    bt = bt_host.to(dev)
    T, Hq, D = batch.total_q, batch.num_q_heads, batch.head_dim
    o = torch.empty((T, Hq, D), dtype=torch.bfloat16, device=dev)
    lse = torch.empty((T, Hq), dtype=torch.float32, device=dev)
    o_host = torch.empty((T, Hq, D), dtype=torch.bfloat16).pin_memory()
    lse_host = torch.empty((T, Hq), dtype=torch.float32).pin_memory()

    flops = float(info.useful_flops)
    kvb = float(info.kv_bytes)
    alg_bytes = float(W.algorithmic_bytes(batch))

    def barrier():
        if world > 1:
            dist.barrier()
        torch.cuda.synchronize()

    def step():
        ctx.run(q, k_pool, v_pool, bt, SCALE, o, lse)

    for _ in range(warmup):
        step()
    barrier()
    assert ctx.device_status() == 0

    # ---- timed region: K steps, inputs resident in HBM; KV pools are far larger than L2
    sampler = ClockSampler(local_rank)
    if rank == 0:
        sampler.start()
        time.sleep(0.3)
    ctx.set_timing(True)
    ev0, ev1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
    barrier()
    ev0.record()
    for _ in range(args.steps):
        step()
    ev1.record()
    barrier()
    total_ms = ev0.elapsed_time(ev1)
    attn_ms, merge_ms, runs = ctx.get_timing()
    ctx.set_timing(False)
    launches = ctx.last_launches() * args.steps
    clocks = sampler.stop() if rank == 0 else None
    tms = torch.tensor([total_ms], dtype=torch.float64, device=dev)
    if world > 1:
        dist.all_reduce(tms, op=dist.ReduceOp.MAX)
    ms_per_step = float(tms.item()) / args.steps
    # every rank processes the same recipe; whole-job units = sum over ranks
    tot = torch.tensor([flops, kvb], dtype=torch.float64, device=dev)
    if world > 1:
        dist.all_reduce(tot, op=dist.ReduceOp.SUM)
    job_flops, job_kvb = float(tot[0].item()), float(tot[1].item())
    value = job_flops / (ms_per_step * 1e-3) / 1e12
    kv_gbs = job_kvb / (ms_per_step * 1e-3) / 1e9

    # ---- end to end: host planning + H2D of the step's inputs + run + D2H of O and LSE
    e2e = None
    if not args.no_e2e:
        # Steps are independent, so they are software-pipelined over three streams with two sets of
        # buffers: the H2D copy of step i+1 and the D2H copy of step i-1 run beside the kernels of
        # step i.  Every step still does all of its own work inside the timed region: host plan,
        # H2D of its fused QKV + block table + task tables, KV-cache append, attention, D2H of O, LSE.
        s_in, s_run, s_out = torch.cuda.Stream(dev), torch.cuda.Stream(dev), torch.cuda.Stream(dev)
        qkv_d = [qkv, torch.empty_like(qkv)]
        bt_d = [bt, torch.empty_like(bt)]
        o_d = [o, torch.empty_like(o)]
        lse_d = [lse, torch.empty_like(lse)]
        o_h = [o_host, torch.empty_like(o_host).pin_memory()]
        lse_h = [lse_host, torch.empty_like(lse_host).pin_memory()]

        def e2e_run(n):
            ev_in = [None, None]
            ev_run = [None, None]
            ev_out = [None, None]

            def copy_in(i):
                b = i & 1
                with torch.cuda.stream(s_in):
                    if ev_run[b] is not None:
                        s_in.wait_event(ev_run[b])  # step i-2 has read this input buffer
                    qkv_d[b].copy_(qkv_host, non_blocking=True)
                    bt_d[b].copy_(bt_pin, non_blocking=True)
                    ev_in[b] = torch.cuda.Event()
                    ev_in[b].record(s_in)

            copy_in(0)
            for i in range(n):
                b = i & 1
                if i + 1 < n:
                    copy_in(i + 1)
                with torch.cuda.stream(s_run):
                    s_run.wait_event(ev_in[b])
                    if ev_out[b] is not None:
                        s_run.wait_event(ev_out[b])  # step i-2's results have left this output buffer
                    ctx.plan_batch(batch, stream=s_run)
                    ctx.append_kv(qkv_d[b], k_pool, v_pool, bt_d[b], stream=s_run)
                    ctx.run(qkv_d[b][:, : batch.num_q_heads, :], k_pool, v_pool, bt_d[b], SCALE, o_d[b], lse_d[b],
                            stream=s_run)
                    ev_run[b] = torch.cuda.Event()
                    ev_run[b].record(s_run)
                with torch.cuda.stream(s_out):
                    s_out.wait_event(ev_run[b])
                    o_h[b].copy_(o_d[b], non_blocking=True)
                    lse_h[b].copy_(lse_d[b], non_blocking=True)
                    ev_out[b] = torch.cuda.Event()
                    ev_out[b].record(s_out)
            torch.cuda.synchronize()

        e2e_run(3)
        barrier()
        n_e2e = max(3, min(args.steps, 20))
        e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
        cur = torch.cuda.current_stream()
        e0.record(cur)
        for st in (s_in, s_run, s_out):
            st.wait_stream(cur)  # nothing of the pipeline starts before e0
        t_host0 = time.perf_counter()
        e2e_run(n_e2e)  # ends with a device synchronize
        t_host1 = time.perf_counter()
        e1.record(cur)
        barrier()
        assert ctx.device_status() == 0
        # Both buffer sets must carry the same bits as one more device-resident run on the cache as
        # the appends left it (reported, not asserted).
        o_check = torch.empty_like(o)
        ctx.run(q, k_pool, v_pool, bt, SCALE, o_check, lse)
        torch.cuda.synchronize()
        o_res_host = o_check.cpu()
        e2e_same = bool(torch.equal(o_h[0], o_res_host) and torch.equal(o_h[1], o_res_host))
        del o_check, o_res_host
        e2e_host_ms = (t_host1 - t_host0) * 1e3 / n_e2e
        ems = torch.tensor([e0.elapsed_time(e1) / n_e2e], dtype=torch.float64, device=dev)
        if world > 1:
            dist.all_reduce(ems, op=dist.ReduceOp.MAX)
        e2e_ms = float(ems.item())
        h2d = qkv_host.numel() * 2 + bt_pin.numel() * 4 + info.num_tasks * 32 + batch.num_requests * 32
        d2h = o_host.numel() * 2 + lse_host.numel() * 4
        e2e = {"value": job_flops / (e2e_ms * 1e-3) / 1e12, "unit": "TFLOP/s", "ms_per_step": e2e_ms,
               "h2d_bytes_per_step": int(h2d), "d2h_bytes_per_step": int(d2h), "steps": n_e2e,
               "host_clock_ms_per_step": e2e_host_ms, "bit_identical_to_resident_run": e2e_same,
               "includes": "per step: host plan, H2D (fused QKV of the new tokens, block table, task tables), "
                           "KV append, run, D2H (O, LSE); steps pipelined over three streams; cached history "
                           "device-resident; CUDA events around all steps"}

    if world > 1:  # every collective is behind us: all ranks leave the group together
        dist.barrier()
        dist.destroy_process_group()
    if rank != 0:
        return 0

    peaks = measured_peaks()
    attn_ms_avg = attn_ms / max(1, runs)
    roof = roofline_entry(flops, alg_bytes, attn_ms_avg, merge_ms / max(1, runs), peaks, clocks)
    roof["traffic"], roof["traffic_source"] = ncu_traffic(args.workload)
    roof["kernel"] = "attention meta-kernel"
    roof["workload"] = args.workload

    cpu = None
    if not args.no_cpu_baseline and world == 1:  # the oracle is timed at N = 1 only
        if args.cpu_full:
            r = time_oracle_full(batch, tensors)
            what = "the whole workload once (%d output rows), %.1f s" % (r["rows"], r["seconds"])
        else:
            r = time_oracle_sample(batch, tensors, 12.0)
            what = "%d random output rows (request, head, token) of the workload, %.1f s" % (r["rows"], r["seconds"])
        cpu = {"value": r["tflops"], "unit": "TFLOP/s", "cores": r["cores"], "kind": "oracle", "host": host_cpu(),
               "sample": "%s; %s" % (what, tree_pairs_note())}

    pool_gb = 2 * k_pool.numel() * 2 / 1e9
    others = None
    if not args.no_others and world == 1:
        others = {}
        del q, qkv, k_pool, v_pool, o, lse, tensors
        torch.cuda.empty_cache()
        per_config = {}
        for name in ("decode_only", "splitfuse_mix", "verify_trees", "full_mix"):
            if name == args.workload:
                per_config[name] = "this line's primary workload: see the keys of `roofline` itself"
                continue
            try:
                per_config[name] = measure_other(name, kernel, dev, peaks)
            except Exception as e:  # report, never hide the primary line
                per_config[name] = {"error": repr(e)}
        roof["per_config"] = per_config
        try:
            torch.cuda.empty_cache()
            others["serving_stream"] = measure_stream(kernel, dev, peaks)
        except Exception as e:
            others["serving_stream"] = {"error": repr(e)}
        try:
            torch.cuda.empty_cache()
            others["decode_shared_prefix"] = measure_shared_prefix(kernel, dev, peaks)
        except Exception as e:
            others["decode_shared_prefix"] = {"error": repr(e)}
        try:
            torch.cuda.empty_cache()
            others["long_context_decode"] = measure_long_decode(kernel, dev, peaks)
        except Exception as e:
            others["long_context_decode"] = {"error": repr(e)}
        try:
            torch.cuda.empty_cache()
            others["decode_only_fp8kv"] = measure_fp8_decode(dev, peaks)
        except Exception as e:
            others["decode_only_fp8kv"] = {"error": repr(e)}
        try:
            torch.cuda.empty_cache()
            others["smoothgemm"] = measure_gemm(dev, peaks)
        except Exception as e:
            others["smoothgemm"] = {"error": repr(e)}

    line = {
        "metric": "hybrid_attention_useful_tflops", "value": value, "unit": "TFLOP/s",
        "kv_gbs": kv_gbs, "n_gpus": world, "steps": args.steps, "warmup": warmup,
        "ms_per_step": ms_per_step, "higher_is_better": True, "scaling": "weak", "vs_baseline": None,
        "dtype": "bf16", "data": "synthetic",
        "config": dict(workload_config(args.workload, batch), kernel=args.kernel, tasks=info.num_tasks,
                       merge_units=info.num_merge_units, plan_us=plan_us,
                       l2="KV pool (%.2f GB) exceeds L2; no flush" % pool_gb,
                       parallelism="replicas x%d (requests sharded, no collective)" % world),
        "other_workloads": others, "cpu_baseline": cpu, "e2e": e2e, "gpu_launches": launches, "clocks": clocks,
        "roofline": roof,
    }
    print(json.dumps(compact(line)))
    return 0


def compact(x):
    """Floats to five significant digits: the line stays short enough that its tail still holds
    every configuration."""
    if isinstance(x, float):
        return float("%.5g" % x) if math.isfinite(x) else None
    if isinstance(x, dict):
        return {k: compact(v) for k, v in x.items()}
    if isinstance(x, (list, tuple)):
        return [compact(v) for v in x]
    return x


if __name__ == "__main__":
    sys.exit(main())

"""Benchmark of the MixAttention decode path (and a prompt-pass figure beside it).

  python bench.py [--gpus N] [--steps K] [--warmup W] [--impl reference] [--workload NAME]

A step is one decode step of the whole model: for each of the 24 layers, append
the new token's K/V if the layer owns a cache, then attend (split pass +
combine).  Workload: the mid-decode configuration (batch 32, context 32768,
window 1024, 32/8 heads of 128, bf16) with seeded synthetic inputs.

Prints ONE JSON line (rank 0).  `value` is decode-attention GB/s: KV bytes each
layer reads (a shared cache counted once per reading layer) / device time, with
all inputs resident in HBM.  `e2e` is the same metric with each step's inputs
copied from pinned host memory and the step's outputs read back, inside the
timed region.  With --gpus N > 1 every rank runs an independent replica (the
path has no exchange step); the value is the sum over ranks / max time.

--impl reference times the CPU checker (oracle/) on the host cores on a
bounded sample of the same workload.
"""
from __future__ import annotations

import argparse
import json
import os
import subprocess
import sys
import threading
import time

ROOT = os.path.dirname(os.path.abspath(__file__))
if ROOT not in sys.path:
    sys.path.insert(0, ROOT)

import numpy as np
import torch

from synth import configs as cf
from synth import inputs as si

METRIC = "decode attention HBM GB/s (% of peak) & tokens/s; prefill TFLOP/s (% bf16 peak)"
NOMINAL_BF16_TFLOPS = 2250.0     # dense bf16 datasheet figure of a B200 (context; fractions of it are reported too)
BURST_IDLE_S = 0.5   # idle time before each short tensor-core measurement (see prefill_figures)
FALLBACK_PEAKS = {"hbm_gbs": 6650.0, "bf16_tflops": 1590.0, "bf16_tflops_sustained": 1400.0}

# (dram__bytes_read.sum + dram__bytes_write.sum) / algorithmic KV bytes of the dominant kernel, from an
# ncu capture of one standard-layer launch at batch 4 (540.62 MB moved for 536.94 MB of keys and values;
# the full-size launch holds too much device memory for a multi-pass capture).  DRAM traffic grows in
# proportion to the keys read, so the full-size figure is this ratio times the launch's algorithmic
# bytes.  Set to None when the kernel changes until the counters are taken again.
DECODE_FULL_TRAFFIC_RATIO = 540.617984 / 536.936448


def load_peaks():
    path = os.path.join(ROOT, "MEASURED_PEAKS.json")
    if os.path.exists(path):
        with open(path) as f:
            d = json.load(f)
        d["_source"] = "measured"
        d.setdefault("bf16_tflops_sustained", FALLBACK_PEAKS["bf16_tflops_sustained"])
        return d
    d = dict(FALLBACK_PEAKS)
    d["_source"] = "fallback"
    return d


def get_workload(name: str) -> cf.Workload:
    if name == "long_decode_pairs":
        return cf.long_decode(pairs=True)
    return cf.ALL[name]()


# ---------------------------------------------------------------------------
# clocks
# ---------------------------------------------------------------------------
class ClockSampler:
    FIELDS = ("clocks.sm,clocks.max.sm,clocks_event_reasons.hw_slowdown,"
              "clocks_event_reasons.hw_thermal_slowdown,clocks_event_reasons.sw_thermal_slowdown,"
              "clocks_event_reasons.sw_power_cap")

    def __init__(self, index: int):
        self.index = index
        self.proc = None
        self.lines = []          # (host time, csv line)
        self.t_lo = self.t_hi = None

    def start(self):
        try:
            self.proc = subprocess.Popen(
                ["nvidia-smi", f"--query-gpu={self.FIELDS}", "--format=csv,noheader,nounits",
                 "-i", str(self.index), "-lms", "20"],
                stdout=subprocess.PIPE, stderr=subprocess.DEVNULL, text=True)
            self.thread = threading.Thread(target=self._read, daemon=True)
            self.thread.start()
        except Exception:
            self.proc = None

    def _read(self):
        for line in self.proc.stdout:
            self.lines.append((time.perf_counter(), line.strip()))

    def mark_begin(self):
        self.t_lo = time.perf_counter()

    def mark_end(self):
        self.t_hi = time.perf_counter()

    def stop(self):
        if self.proc is None:
            return {"sm_mhz": None, "sm_max_mhz": None, "reasons": ["unavailable"]}
        self.proc.terminate()
        try:
            self.proc.wait(timeout=5)
        except Exception:
            self.proc.kill()
        sm, sm_all, mx, reasons = [], [], None, set()
        names = ["hw_slowdown", "hw_thermal_slowdown", "sw_thermal_slowdown", "sw_power_cap"]
        for t, ln in self.lines:
            parts = [p.strip() for p in ln.split(",")]
            if len(parts) < 6:
                continue
            try:
                mhz = float(parts[0])
                mx = float(parts[1])
            except ValueError:
                continue
            sm_all.append(mhz)
            # a sample belongs to the timed part when it was read between the two marks (the
            # query itself takes a few milliseconds, hence the small allowance at the end)
            if self.t_lo is not None and self.t_hi is not None and not (self.t_lo <= t <= self.t_hi + 0.03):
                continue
            sm.append(mhz)
            for nm, val in zip(names, parts[2:6]):
                if val.lower().startswith("active"):
                    reasons.add(nm)
        return {"sm_mhz": float(np.median(sm)) if sm else None, "sm_max_mhz": mx,
                "reasons": sorted(reasons), "samples": len(sm), "samples_whole_run": len(sm_all),
                "sm_mhz_whole_run": float(np.median(sm_all)) if sm_all else None}


# ---------------------------------------------------------------------------
# CPU checker timing (cpu_baseline leg and --impl reference)
# ---------------------------------------------------------------------------
def oracle_sample_prepare(wl: cf.Workload, n_seqs: int, heads_per_layer: int):
    """Inputs of the CPU checker's timed sample: layer 0 (standard) and layer 1
    (sliding window), the first `n_seqs` sequences, `heads_per_layer` query heads."""
    dt = torch.bfloat16 if wl.dtype == cf.BF16 else torch.float32
    e = 2 if wl.dtype == cf.BF16 else 4
    G = wl.n_q_heads // wl.n_kv_heads
    n = wl.context + 1
    heads = list(range(heads_per_layer))
    jobs = []
    for layer in (0, 1):
        kind, W, owner = wl.layout[layer]
        lo = 0 if kind == cf.FULL else max(0, n - W)
        for b in range(n_seqs):
            q = si.q_tokens(wl.seed, layer, b, n - 1, 1, wl.n_q_heads, wl.head_dim, dt)[0].double().numpy()
            kv = {}
            for g in sorted({h // G for h in heads}):
                K, V = si.kv_tokens_head(wl.seed, owner, b, lo, n - lo, wl.n_kv_heads, wl.head_dim, g, dt)
                kv[g] = (K.double().numpy(), V.double().numpy())
            # bytes the job stands for: the KV heads touched, counted once per group of heads
            jobs.append((q, kv, heads, G, (n - lo) * 2 * wl.head_dim * e * (len(heads) / G)))
    return jobs, 1.0 / np.sqrt(wl.head_dim)


def oracle_sample_run(jobs, scale):
    """One pass of the CPU checker over the prepared sample: (seconds, KV bytes)."""
    from oracle import mixattn_oracle as mo
    t0 = time.perf_counter()
    nbytes = 0.0
    for q, kv, heads, G, b in jobs:
        for h in heads:
            K, V = kv[h // G]
            mo.softmax_attend(q[h], K, V, scale)
        nbytes += b
    return time.perf_counter() - t0, nbytes


def blas_threads() -> int:
    try:
        from threadpoolctl import threadpool_info
        return max([p.get("num_threads", 1) for p in threadpool_info()] + [1])
    except Exception:
        return 1


def run_reference_arm(args, wl):
    """The CPU checker as the reference arm: K steps, each one pass over a bounded sample."""
    rank = int(os.environ.get("RANK", "0"))
    if rank != 0:
        return
    n_seqs, heads = 2, wl.n_q_heads
    jobs, scale = oracle_sample_prepare(wl, n_seqs, heads)
    for _ in range(args.warmup):
        oracle_sample_run(jobs, scale)
    secs, nbytes = 0.0, 0.0
    for _ in range(args.steps):
        s, b = oracle_sample_run(jobs, scale)
        secs += s
        nbytes += b
    threads = blas_threads()
    value = nbytes / secs / 1e9
    sample = (f"layers 0 (standard) and 1 (sliding window) of sequences 0..{n_seqs - 1}, all {heads} query "
              f"heads, context {wl.context}+1, per step")
    line = {
        "impl": "reference", "metric": METRIC, "value": value, "unit": "GB/s", "n_gpus": args.gpus,
        "steps": args.steps, "warmup": args.warmup, "ms_per_step": secs / args.steps * 1e3,
        "higher_is_better": True, "scaling": "weak", "vs_baseline": None, "dtype": "f64",
        "data": "synthetic",
        "config": {"workload": wl.name, "batch": wl.batch, "context": wl.context or list(wl.context_range),
                   "window": 1024, "layers": len(wl.layout), "heads": f"{wl.n_q_heads}/{wl.n_kv_heads}x{wl.head_dim}",
                   "l2": "host run: no device cache involved", "parallelism": "replicas only", "sample": sample},
        "cpu_baseline": {"value": value, "unit": "GB/s", "cores": threads, "kind": "oracle", "sample": sample},
        "e2e": {"value": value, "unit": "GB/s", "h2d_bytes_per_step": 0, "d2h_bytes_per_step": 0},
    }
    print(json.dumps(line), flush=True)


# ---------------------------------------------------------------------------
# GPU arm
# ---------------------------------------------------------------------------
def prefill_figures(mx, runner, peaks, device):
    """Prompt pass on the prefill configuration: one standard and one sliding layer."""
    wl = cf.prefill_chunk()
    sess = runner.Session(wl, [0] * wl.batch, device=device)
    res = {}
    try:
        S, W, D, Hq, B = wl.seq_len, 1024, wl.head_dim, wl.n_q_heads, wl.batch
        pairs_full = S * (S + 1) // 2
        pairs_slide = sum(min(i + 1, W) for i in range(S))
        for name, layer, pairs, cls in (("full", 12, pairs_full, mx.K_PREFILL_FULL),
                                        ("sliding", 2, pairs_slide, mx.K_PREFILL_SLIDING)):
            q, k, v = sess.prefill_inputs(layer)      # readers: no cache writes, repeatable
            out = torch.empty_like(q)
            reps = 20
            # a burst figure, read against a burst peak that was measured on an otherwise idle GPU:
            # let the board's power average fall back before each one
            torch.cuda.synchronize()
            time.sleep(BURST_IDLE_S)
            for _ in range(3):
                sess.prefill_layer(layer, q, k, v, out)
            torch.cuda.synchronize()
            sess.ctx.profile_enable(True)
            for _ in range(reps):
                sess.prefill_layer(layer, q, k, v, out)
            n, ms = sess.ctx.profile_read(cls)
            sess.ctx.profile_enable(False)
            flops = 4.0 * D * pairs * Hq * B
            tf = flops / (ms / n * 1e-3) / 1e12
            res[name] = {"ms_per_layer": ms / n, "tflops": tf, "frac_of_bf16_peak": tf / peaks["bf16_tflops"],
                         "frac_of_nominal_2250": tf / NOMINAL_BF16_TFLOPS, "useful_flop": flops, "launches_timed": n}
        res["config"] = {"workload": wl.name, "batch": B, "seq_len": S, "window": W}
        # the stated target (sliding-window layer at half the bf16 dense peak) read both ways
        res["target_half_of_nominal_met"] = res["sliding"]["frac_of_nominal_2250"] >= 0.5
        res["target_half_of_measured_met"] = res["sliding"]["frac_of_bf16_peak"] >= 0.5
        res["peak_tflops"] = peaks["bf16_tflops"]
        res["nominal_tflops"] = NOMINAL_BF16_TFLOPS
        res["peak_source"] = peaks["_source"]
    finally:
        sess.close()
    return res


def prefill_sustained(mx, runner, peaks, device, res):
    """The launches of prefill_figures last 12-40 ms each way: bursts, read against the burst
    peak.  Here the same launch is repeated for about 1.5 s, which settles at the clock the power
    limit allows; the last two thirds of the loop are read against the sustained peak.  Runs after
    every burst measurement, so that none of them starts on a GPU a long loop has just driven to
    its power limit."""
    wl = cf.prefill_chunk()
    sess = runner.Session(wl, [0] * wl.batch, device=device)
    try:
        for name, layer, cls in (("full", 12, mx.K_PREFILL_FULL), ("sliding", 2, mx.K_PREFILL_SLIDING)):
            q, k, v = sess.prefill_inputs(layer)
            out = torch.empty_like(q)
            n_loop = max(30, int(1500.0 / res[name]["ms_per_layer"]))
            for _ in range(n_loop // 3):
                sess.prefill_layer(layer, q, k, v, out)
            sess.ctx.profile_enable(True)
            for _ in range(n_loop - n_loop // 3):
                sess.prefill_layer(layer, q, k, v, out)
            n_s, ms_s = sess.ctx.profile_read(cls)
            sess.ctx.profile_enable(False)
            tf_s = res[name]["useful_flop"] / (ms_s / n_s * 1e-3) / 1e12
            res[name]["sustained"] = {"tflops": tf_s, "ms_per_layer": ms_s / n_s, "launches_timed": n_s,
                                      "frac_of_bf16_peak_sustained": tf_s / peaks["bf16_tflops_sustained"]}
        res["target_half_of_measured_sustained_met"] = res["sliding"]["sustained"]["frac_of_bf16_peak_sustained"] >= 0.5
        res["peak_tflops_sustained"] = peaks["bf16_tflops_sustained"]
    finally:
        sess.close()


def chunk_figures(mx, runner, peaks, device, prefix=6144, chunk=2048):
    """The last chunk of the prefill configuration's prompts served in chunks: `chunk` new
    tokens per sequence behind `prefix` cached ones (gather of the cached keys + attention)."""
    wl = cf.prefill_chunk().scaled(seq_len=0)
    B, D, Hq, W = wl.batch, wl.head_dim, wl.n_q_heads, 1024
    sess = runner.Session(wl, [prefix] * B, device=device, headroom_tokens=chunk,
                          chunk_scratch_tokens=B * (prefix + chunk))
    res = {}
    try:
        sess.fill(2048)
        ids, lens = list(range(B)), [chunk] * B
        pairs_full = sum(prefix + r + 1 for r in range(chunk))
        pairs_slide = sum(min(prefix + r + 1, W) for r in range(chunk))
        # "sliding": the ring read in place by the attention kernel (the default); "sliding_copied":
        # the same call with the cached keys copied out of the ring first
        for name, layer, pairs, cls, in_place in (("full", 12, pairs_full, mx.K_PREFILL_FULL, True),
                                                  ("sliding", 2, pairs_slide, mx.K_PREFILL_SLIDING, True),
                                                  ("sliding_copied", 2, pairs_slide, mx.K_PREFILL_SLIDING, False)):
            sess.ctx.set_chunk_ring_direct(in_place)
            owner = wl.layout[layer][2]
            q = si.q_tokens_multi(wl.seed, layer, ids, [prefix] * B, chunk, Hq, D, sess.dt,
                                  sess.dev).reshape(-1, Hq, D)
            K, V = si.kv_tokens_multi(wl.seed, owner, ids, [prefix] * B, chunk, wl.n_kv_heads, D, sess.dt, sess.dev)
            K, V = K.reshape(-1, wl.n_kv_heads, D), V.reshape(-1, wl.n_kv_heads, D)
            out = torch.empty_like(q)
            reps = 10
            torch.cuda.synchronize()
            time.sleep(BURST_IDLE_S)
            for _ in range(2):
                sess.ctx.attend_chunk(layer, ids, lens, q, K, V, out)
            torch.cuda.synchronize()
            sess.ctx.profile_enable(True)
            for _ in range(reps):
                sess.ctx.attend_chunk(layer, ids, lens, q, K, V, out)
            n, ms = sess.ctx.profile_read(cls)
            ng, msg = sess.ctx.profile_read(mx.K_GATHER)
            sess.ctx.profile_enable(False)
            flops = 4.0 * D * pairs * Hq * B
            ms_gather = msg / ng if ng else 0.0
            t = (ms / n + ms_gather) * 1e-3
            res[name] = {"ms_attention": ms / n, "ms_gather": ms_gather, "tflops": flops / t / 1e12,
                         "frac_of_bf16_peak": flops / t / 1e12 / peaks["bf16_tflops"],
                         "frac_of_nominal_2250": flops / t / 1e12 / NOMINAL_BF16_TFLOPS, "useful_flop": flops}
        # the same chunk through all 24 layers, each reader handed its owner's K/V; the rings are
        # read in place, and the copy of the standard cache's keys serves both layers that read it
        sess.ctx.set_chunk_ring_direct(True)
        sess.ctx.set_chunk_gather_reuse(True)
        kv = {}
        for o in sess.owners:
            K, V = si.kv_tokens_multi(wl.seed, o, ids, [prefix] * B, chunk, wl.n_kv_heads, D, sess.dt, sess.dev)
            kv[o] = (K.reshape(-1, wl.n_kv_heads, D), V.reshape(-1, wl.n_kv_heads, D))
        q = si.q_tokens_multi(wl.seed, 0, ids, [prefix] * B, chunk, Hq, D, sess.dt, sess.dev).reshape(-1, Hq, D)
        out = torch.empty_like(q)
        flops_pass = 0.0
        for timed in (False, True):
            sess.ctx.set_chunk_gather_reuse(True)   # forgets the previous pass: a chunk's first reader copies
            sess.ctx.profile_enable(timed)
            for layer, (kind, _, owner) in enumerate(wl.layout):
                sess.ctx.attend_chunk(layer, ids, lens, q, kv[owner][0], kv[owner][1], out)
                if timed:
                    flops_pass += 4.0 * D * (pairs_full if kind == cf.FULL else pairs_slide) * Hq * B
            torch.cuda.synchronize()
        ms_pass = sum(sess.ctx.profile_read(c)[1] for c in (mx.K_PREFILL_FULL, mx.K_PREFILL_SLIDING, mx.K_GATHER))
        n_gather = sess.ctx.profile_read(mx.K_GATHER)[0]
        sess.ctx.profile_enable(False)
        sess.ctx.set_chunk_gather_reuse(False)
        res["layout_pass"] = {"layers": len(wl.layout), "gathers": n_gather, "ms": ms_pass,
                              "tflops": flops_pass / (ms_pass * 1e-3) / 1e12,
                              "frac_of_bf16_peak": flops_pass / (ms_pass * 1e-3) / 1e12 / peaks["bf16_tflops"]}
        res["config"] = {"workload": wl.name, "batch": B, "cached_prefix": prefix, "chunk": chunk, "window": W}
    finally:
        sess.close()
    return res


def reduce_over_ranks(dist, times, work, device):
    """Replicas-only aggregation: times -> max over ranks, work -> sum over ranks.
    (No data-path collective exists; this is the only communication of a run.)"""
    t = torch.tensor([float(x) for x in times], device=device, dtype=torch.float64)
    dist.all_reduce(t, op=dist.ReduceOp.MAX)
    w = torch.tensor([float(x) for x in work], device=device, dtype=torch.float64)
    dist.all_reduce(w, op=dist.ReduceOp.SUM)
    return t.tolist(), w.tolist()


MIN_TIMED_S = 0.4        # the K-step region is repeated until this much device time has been timed
MAX_EXTRA_STEPS = 600    # at most this many steps beyond the first region


def n_regions_for(region_ms: float, K: int) -> int:
    """How many K-step regions to time so that the timed part spans at least MIN_TIMED_S (a
    region of a few tens of milliseconds is shorter than two ticks of the clock sampler)."""
    if region_ms <= 0:
        return 1
    want = int(np.ceil(MIN_TIMED_S * 1e3 / region_ms))
    return max(1, min(want, 1 + MAX_EXTRA_STEPS // max(K, 1)))


def make_session(runner, wl, device, total_steps, kv_format=0):
    """Session with the workload's lengths drawn, its page order permuted if asked, caches filled."""
    if wl.context_range != (0, 0):
        lengths = si.draw_lengths(wl.seed, wl.batch, *wl.context_range).tolist()
    else:
        lengths = [wl.context] * wl.batch
    free_order = None
    if wl.permute_pages:
        n_pages = sum(-(-(n + total_steps) // wl.page_size) for n in lengths)
        free_order = si.page_permutation(wl.seed, n_pages)
    sess = runner.Session(wl, lengths, device=device, headroom_tokens=total_steps, free_order=free_order,
                          kv_format=kv_format)
    sess.fill(1024)
    return sess, lengths


def step_input_ring(sess, n):
    """n distinct seeded steps' inputs, reused cyclically (the values do not change the work;
    positions, appends and lengths advance every step as in serving)."""
    ring = []
    pos_save = sess.pos.copy()
    for _ in range(n):
        ring.append(sess.step_inputs())
        sess.pos += 1
    sess.pos[:] = pos_save
    return ring


def device_pass(sess, runner, wl, ring, outs, stream, K, Wm, barrier, sampler=None):
    """Wm warm-up steps, then regions of exactly K decode steps between CUDA events on the
    launching stream, inputs resident in HBM.  The first region decides how many more follow
    (n_regions_for).  Returns (mean ms per region, mean KV bytes per region, regions, launches
    per region)."""
    tables = [sess.step_tables(inp, outs) for inp in ring]    # pointer tables, built once per ring entry
    step = 0
    for _ in range(Wm):
        sess.decode_step(ring[step % len(ring)], outs, stream, tables=tables[step % len(ring)])
        step += 1
    launches0 = sess.ctx.get_launch_count()
    barrier()
    if sampler is not None:
        sampler.mark_begin()
    events, nbytes = [], []

    def region():
        nonlocal step
        e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
        # bytes of the region's K steps, counted ahead of the timed calls (every step adds one token per sequence)
        b = sum(runner.kv_bytes_per_step(wl, sess.pos + 1 + k, sess.kv_format) for k in range(K))
        e0.record(stream)
        for _ in range(K):
            sess.decode_step(ring[step % len(ring)], outs, stream, tables=tables[step % len(ring)])
            step += 1
        e1.record(stream)
        events.append((e0, e1))
        nbytes.append(b)

    region()
    torch.cuda.synchronize()
    more = n_regions_for(events[0][0].elapsed_time(events[0][1]), K) - 1
    for _ in range(more):
        region()
    barrier()
    if sampler is not None:
        sampler.mark_end()
    ms = [a.elapsed_time(b) for a, b in events]
    launches = (sess.ctx.get_launch_count() - launches0) / len(events)
    assert sess.ctx.get_device_status() == 0, "a kernel reported a wait time-out"
    return float(np.mean(ms)), float(np.mean(nbytes)), len(events), launches


def other_workload_figures(runner, peaks, device, K, Wm):
    """The other decode configurations, device-resident, in compact form: long-context decode,
    its variant with rings shared in pairs, the mixed serving batch, and the mid-decode
    configuration on a quantised cache (FP8 E4M3 elements: bytes = what that cache holds)."""
    from paper_2409_15012_b200 import binding as mx
    res = {}
    for name, kvf in (("long_decode", 0), ("long_decode_pairs", 0), ("mixed_serving", 0),
                      ("mid_decode", mx.KV_FP8_E4M3)):
        wl = get_workload(name)
        if kvf:
            wl = wl.scaled(name=wl.name + "_fp8_kv")
        total = Wm + K + MAX_EXTRA_STEPS + 2
        sess, lengths = make_session(runner, wl, device, total, kvf)
        try:
            ring = step_input_ring(sess, min(4, Wm + K))
            outs = sess.alloc_outputs()
            stream = torch.cuda.current_stream()
            ms, nbytes, regions, launches = device_pass(sess, runner, wl, ring, outs, stream, K, Wm,
                                                        torch.cuda.synchronize)
            gbs = nbytes / (ms * 1e-3) / 1e9
            res[wl.name] = {"gbs": gbs, "ms_per_step": ms / K, "frac_of_measured_hbm": gbs / peaks["hbm_gbs"],
                            "frac_of_nominal_8TBs": gbs / 8000.0, "tokens_per_s": wl.batch / (ms / K * 1e-3),
                            "launches_per_step": launches / K, "steps": K, "regions": regions,
                            "batch": wl.batch, "context": wl.context or list(wl.context_range),
                            "kv_gb_per_step": nbytes / K / 1e9}
        finally:
            sess.close()
    return res


def run_gpu_arm(args, wl):
    from paper_2409_15012_b200 import build as mbuild
    rank = int(os.environ.get("RANK", "0"))
    world = int(os.environ.get("WORLD_SIZE", "1"))
    local = int(os.environ.get("LOCAL_RANK", "0"))
    if not torch.cuda.is_available():
        raise SystemExit("bench.py needs a CUDA device: there is no CPU path")
    if rank == 0:
        mbuild.build()
    torch.cuda.set_device(local)
    dist = None
    if world > 1:
        import torch.distributed as dist
        dist.init_process_group("nccl", device_id=torch.device(f"cuda:{local}"))
        dist.barrier()
    from paper_2409_15012_b200 import binding as mx, runner
    peaks = load_peaks()
    K, Wm = args.steps, args.warmup
    # device-timed pass, e2e pass (each up to MAX_EXTRA_STEPS more), profiled pass
    total_steps = 2 * (K + Wm + MAX_EXTRA_STEPS) + min(K, 20) + 2
    sampler = ClockSampler(local)
    if rank == 0:
        sampler.start()          # before the fill and the warm-up: the GPU is under load when timing starts
    kvf = mx.KV_FP8_E4M3 if args.kv_format == "fp8" else mx.KV_NATIVE
    sess, lengths = make_session(runner, wl, local, total_steps, kvf)
    stream = torch.cuda.current_stream()
    outs = sess.alloc_outputs()

    def barrier():
        if dist is not None:
            dist.barrier()
        torch.cuda.synchronize()

    # ---- device-resident pass: `value` ----
    kRing = min(8, Wm + K)
    step_inputs = step_input_ring(sess, kRing)
    ms, kv_bytes, regions, launches = device_pass(sess, runner, wl, step_inputs, outs, stream, K, Wm, barrier,
                                                  sampler if rank == 0 else None)
    clocks = sampler.stop() if rank == 0 else None

    # ---- end-to-end pass: host inputs, host outputs ----
    # Each step's inputs sit in one pinned host buffer and travel in two pieces on a copy
    # stream (the first layers' inputs, then the rest, while the first layers already run);
    # the outputs go back in pieces on a third stream while later layers run (only the last
    # layer's output is copied after the step's last kernel).  Every step ends with a host wait for its complete result.
    pos_save = sess.pos.copy()
    n_layers = len(wl.layout)
    order = [(l, k) for l in range(n_layers) for k in ("q", "k", "v") if k in step_inputs[0][l]]
    offs, total = {}, 0
    for l, k in order:
        t = step_inputs[0][l][k]
        offs[(l, k)] = total
        total += -(-t.numel() * t.element_size() // 256) * 256
    cut_layer = 2                                          # layers before this one travel first
    cut = offs[(cut_layer, "q")]
    host_flat = [torch.empty(total, dtype=torch.uint8).pin_memory() for _ in range(kRing)]
    dev_flat = torch.empty(total, dtype=torch.uint8, device=sess.dev)

    def views(flat):
        out = {}
        for l, k in order:
            t = step_inputs[0][l][k]
            n = t.numel() * t.element_size()
            out.setdefault(l, {})[k] = flat[offs[(l, k)]:offs[(l, k)] + n].view(t.dtype).view(t.shape)
        return out

    for s in range(kRing):
        hv = views(host_flat[s])
        for l, k in order:
            hv[l][k].copy_(step_inputs[s][l][k])
    dev_buf = views(dev_flat)
    host_out = torch.empty(outs.shape, dtype=outs.dtype).pin_memory()
    h2d = sum(t.numel() * t.element_size() for d in step_inputs[0].values() for t in d.values())
    d2h = outs.numel() * outs.element_size()
    h2d_stream, d2h_stream = torch.cuda.Stream(device=sess.dev), torch.cuda.Stream(device=sess.dev)
    ev_in = [torch.cuda.Event() for _ in range(2)]
    d2h_cuts = sorted({n_layers // 2, (5 * n_layers) // 6, n_layers - 1} - {0, n_layers})   # outputs leave in pieces
    ev_out = [torch.cuda.Event() for _ in d2h_cuts]
    ids_all = list(range(wl.batch))
    # the step is issued in a few mixattn_decode_layers calls, cut where a copy has to be awaited
    # (second piece of the inputs) or started (a piece of the outputs)
    dev_tables = sess.step_tables(dev_buf, outs)
    bounds = sorted({0, cut_layer, n_layers} | set(d2h_cuts))

    def e2e_step(s):
        src = host_flat[s % kRing]
        with torch.cuda.stream(h2d_stream):
            dev_flat[:cut].copy_(src[:cut], non_blocking=True)
            ev_in[0].record(h2d_stream)
            dev_flat[cut:].copy_(src[cut:], non_blocking=True)
            ev_in[1].record(h2d_stream)
        for lo_l, hi_l in zip(bounds[:-1], bounds[1:]):
            if lo_l == 0 or lo_l == cut_layer:
                stream.wait_event(ev_in[0 if lo_l == 0 else 1])
            sess.ctx.decode_layers(lo_l, hi_l, ids_all, *dev_tables, stream)
            if hi_l in d2h_cuts:
                i = d2h_cuts.index(hi_l)
                lo = d2h_cuts[i - 1] if i > 0 else 0
                ev_out[i].record(stream)
                d2h_stream.wait_event(ev_out[i])
                with torch.cuda.stream(d2h_stream):
                    host_out[lo:hi_l].copy_(outs[lo:hi_l], non_blocking=True)
        sess.pos += 1
        with torch.cuda.stream(stream):
            host_out[d2h_cuts[-1]:].copy_(outs[d2h_cuts[-1]:], non_blocking=True)
        stream.synchronize()
        d2h_stream.synchronize()

    for s in range(Wm):
        e2e_step(s)
    barrier()
    # as many K-step regions as the device-resident pass timed; each region's time is the larger of
    # the device time between its events and the host's wall clock around it (every step ends with
    # a host wait, so the two agree)
    e2e_ms_all, e2e_bytes_all = [], []
    ev0, ev1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
    step = Wm
    for _ in range(regions):
        b = sum(runner.kv_bytes_per_step(wl, sess.pos + 1 + k, kvf) for k in range(K))   # counted ahead of the timed steps
        t0 = time.perf_counter()
        ev0.record(stream)
        for _ in range(K):
            e2e_step(step)
            step += 1
        ev1.record(stream)
        torch.cuda.synchronize()
        e2e_ms_all.append(max(ev0.elapsed_time(ev1), (time.perf_counter() - t0) * 1e3))
        e2e_bytes_all.append(b)
    barrier()
    e2e_ms, e2e_bytes = float(np.mean(e2e_ms_all)), float(np.mean(e2e_bytes_all))

    # ---- per-kernel pass: roofline of the dominant kernel (split pass of a standard layer) ----
    full_layers = [l for l, (kind, _, _) in enumerate(wl.layout) if kind == cf.FULL]
    slide_layers = [l for l, (kind, _, _) in enumerate(wl.layout) if kind == cf.SLIDING]
    e = 2 if wl.dtype == cf.BF16 else 4
    per_tok = 2 * wl.n_kv_heads * (wl.head_dim + 1 if kvf else wl.head_dim * e)
    sess.ctx.profile_enable(True)
    full_bytes = 0
    Kp = min(K, 20)
    prof_tables = [sess.step_tables(inp, outs) for inp in step_inputs]
    for s in range(Kp):
        full_bytes += sum(int(p) + 1 for p in sess.pos) * per_tok
        sess.decode_step(step_inputs[s % kRing], outs, stream, tables=prof_tables[s % kRing])
    n_full, ms_full = sess.ctx.profile_read(mx.K_DECODE_FULL)
    n_slide, ms_slide = sess.ctx.profile_read(mx.K_DECODE_SLIDING)
    n_comb, ms_comb = sess.ctx.profile_read(mx.K_COMBINE)
    n_app, ms_app = sess.ctx.profile_read(mx.K_APPEND)
    sess.ctx.profile_enable(False)

    # ---- max over ranks, sum of work ----
    if dist is not None:
        (ms, e2e_ms), (kv_bytes, e2e_bytes, launches) = reduce_over_ranks(
            dist, [ms, e2e_ms], [kv_bytes, e2e_bytes, launches], sess.dev)
    if rank != 0:
        sess.close()
        dist.destroy_process_group()
        return

    value = kv_bytes / (ms * 1e-3) / 1e9
    # achieved = bytes per launch / seconds per launch
    bytes_per_launch = full_bytes / Kp if Kp else 0
    sec_per_launch = ms_full / max(n_full, 1) * 1e-3
    achieved = bytes_per_launch / sec_per_launch / 1e9
    roofline = {
        "kernel": "decode_split_bf16_kernel (standard layer)" if wl.dtype == cf.BF16 else "decode_split_f32_kernel",
        "bound": "hbm", "achieved": achieved, "peak": peaks["hbm_gbs"], "unit": "GB/s",
        "frac": achieved / peaks["hbm_gbs"],
        "traffic": None if DECODE_FULL_TRAFFIC_RATIO is None or kvf else DECODE_FULL_TRAFFIC_RATIO * bytes_per_launch,
        "peak_source": f"of {peaks['_source']}", "bytes_per_launch": bytes_per_launch,
        "us_per_launch": sec_per_launch * 1e6, "frac_of_nominal_8TBs": achieved / 8000.0,
    }

    # ---- CPU checker beside it (bounded sample) ----
    cpu = None
    if not args.no_cpu_baseline:
        jobs, scale = oracle_sample_prepare(wl.scaled(context=int(lengths[0])), 2, wl.n_q_heads)
        secs, nbytes, reps = 0.0, 0.0, 0
        while secs < 10.0:
            s_, b_ = oracle_sample_run(jobs, scale)
            secs += s_
            nbytes += b_
            reps += 1
        cpu = {"value": nbytes / secs / 1e9, "unit": "GB/s", "cores": blas_threads(), "kind": "oracle",
               "sample": f"layers 0 (standard) and 1 (sliding window), sequences 0-1, all {wl.n_q_heads} query "
                         f"heads, context {int(lengths[0])}+1; {reps} passes, {secs:.1f} s",
               "host_cores": os.cpu_count()}

    prefill, others = None, None
    closed = False
    if not args.no_prefill:
        sess.close()
        closed = True
        prefill = prefill_figures(mx, runner, peaks, local)
        prefill["chunked"] = chunk_figures(mx, runner, peaks, local)
    if not args.no_other_workloads and world == 1 and args.workload == "mid_decode" and args.batch == 0 and not kvf:
        if not closed:
            sess.close()
            closed = True
        others = other_workload_figures(runner, peaks, local, min(K, 20), Wm)
    if prefill is not None:
        prefill_sustained(mx, runner, peaks, local, prefill)   # last: it leaves the GPU at its power limit

    line = {
        "metric": METRIC, "value": value, "unit": "GB/s", "n_gpus": world, "steps": K, "warmup": Wm,
        "ms_per_step": ms / K, "higher_is_better": True, "scaling": "weak", "vs_baseline": None,
        "dtype": "bf16" if wl.dtype == cf.BF16 else "f32", "data": "synthetic",
        "config": {"workload": wl.name + ("_fp8_kv" if kvf else ""), "batch": wl.batch, "context": wl.context or list(wl.context_range),
                   "window": 1024, "layers": len(wl.layout), "heads": f"{wl.n_q_heads}/{wl.n_kv_heads}x{wl.head_dim}",
                   "l2": "inputs larger than L2 (KV read per step >> 126 MB)", "parallelism": "replicas only"},
        "tokens_per_s": wl.batch * world / (ms / K * 1e-3),
        "frac_of_measured_hbm": value / world / peaks["hbm_gbs"],
        "frac_of_nominal_8TBs": value / world / 8000.0,
        "us_per_layer": {"full_split": ms_full / max(n_full, 1) * 1e3, "sliding_split": ms_slide / max(n_slide, 1) * 1e3,
                         "combine": ms_comb / max(n_comb, 1) * 1e3, "append": ms_app / max(n_app, 1) * 1e3},
        "e2e": {"value": e2e_bytes / (e2e_ms * 1e-3) / 1e9, "unit": "GB/s", "h2d_bytes_per_step": h2d,
                "d2h_bytes_per_step": d2h, "ms_per_step": e2e_ms / K},
        "gpu_launches": int(round(launches)),
        "timed_regions": regions,
        "clocks": clocks,
        "roofline": roofline,
        "cpu_baseline": cpu,
        "prefill": prefill,
        "other_workloads": others,
    }
    print(json.dumps(line), flush=True)
    if not closed:
        sess.close()
    if dist is not None:
        dist.destroy_process_group()


def run_trace_arm(args):
    """Attention-only serving of requests shaped like the paper's benchmark (Section 5.4: prompts of
    31000 tokens, then generated tokens; 12 query / 3 KV heads), one wave of concurrent requests, for
    the standard layout (every layer its own full cache), MixAttention and its pairs variant."""
    from paper_2409_15012_b200 import build as mbuild
    if not torch.cuda.is_available():
        raise SystemExit("bench.py needs a CUDA device: there is no CPU path")
    mbuild.build()
    from paper_2409_15012_b200 import runner
    torch.cuda.set_device(0)
    layouts = {"standard": cf.layout_all_full(24), "sliding_window": cf.layout_all_sliding(24, 1024),
               "mid-decode layout (1 full cache + 2 shared rings)": cf.layout_mid(1024)}
    for name in ("MA", "MA-EndSlide", "MA-Offset", "MA-Pairs", "MA-Offset-SlideShare", "MA-Pairs-SlideShare"):
        layouts[name] = cf.PAPER_VARIANTS[name]()     # the paper's named variants (layer indices: see synth/configs.py)
    if args.trace_layouts:
        keep = [s.strip() for s in args.trace_layouts.split(",")]
        layouts = {k: v for k, v in layouts.items() if k in keep or k == "standard"}
    from paper_2409_15012_b200 import binding as mx
    kvf = mx.KV_FP8_E4M3 if args.kv_format == "fp8" else mx.KV_NATIVE
    res = {}
    for name, lay in layouts.items():
        res[name] = runner.serve_trace(lay, 12, 3, 128, args.trace_requests, args.trace_prompt, args.trace_gen, 2048,
                                       concurrency=args.trace_concurrency, kv_format=kvf)
        res[name]["speedup_over_standard"] = res[name]["tokens_per_s"] / res["standard"]["tokens_per_s"]
        res[name]["cache_bytes_vs_standard"] = res[name]["cache_bytes"] / res["standard"]["cache_bytes"]
    ma = res["MA-Offset"]
    line = {"metric": "attention-only serving throughput on a paper-shaped trace", "value": ma["tokens_per_s"],
            "unit": "tokens/s", "n_gpus": 1, "higher_is_better": True, "dtype": "bf16", "data": "synthetic",
            "vs_baseline": None,
            "config": {"workload": "serving_trace", "layout": "MA-Offset", "requests": args.trace_requests,
                       "concurrency": args.trace_concurrency or args.trace_requests, "kv_format": args.kv_format,
                       "prompt_len": args.trace_prompt, "gen_len": args.trace_gen, "chunk": 2048, "heads": "12/3x128",
                       "layers": 24, "window": 1024,
                       "timing": "sum of the library's kernel times (CUDA events around every launch)"},
            "layouts": res}
    print(json.dumps(line), flush=True)


def replica_envs(n: int, port: int, base_env=None):
    """Environment of each of the n replica processes `--gpus n` starts when it was not launched
    by torchrun: one rank per GPU of this node, rendezvous on the loopback address."""
    envs = []
    for r in range(n):
        e = dict(os.environ if base_env is None else base_env)
        e.update({"RANK": str(r), "LOCAL_RANK": str(r), "WORLD_SIZE": str(n), "LOCAL_WORLD_SIZE": str(n),
                  "MASTER_ADDR": "127.0.0.1", "MASTER_PORT": str(port)})
        envs.append(e)
    return envs


def spawn_replicas(n: int, argv) -> int:
    """Runs this script once per GPU (independent replicas; NCCL carries only the barrier and the
    two scalar reductions of the timing).  Rank 0 prints the JSON line.  Returns the worst exit code."""
    import socket
    with socket.socket() as sk:
        sk.bind(("127.0.0.1", 0))
        port = sk.getsockname()[1]
    procs = [subprocess.Popen([sys.executable, os.path.abspath(__file__)] + list(argv), env=e)
             for e in replica_envs(n, port)]
    rc = 0
    for p in procs:
        p.wait()
        rc = rc or p.returncode
    return rc


def main():
    ap = argparse.ArgumentParser()
    ap.add_argument("--gpus", type=int, default=1)
    ap.add_argument("--steps", type=int, default=200)
    ap.add_argument("--warmup", type=int, default=3)
    ap.add_argument("--impl", default="ours", choices=["ours", "reference"])
    ap.add_argument("--workload", default="mid_decode",
                    choices=["mid_decode", "long_decode", "long_decode_pairs", "mixed_serving", "tiny_decode"])
    ap.add_argument("--batch", type=int, default=0,
                    help="override the batch size (smaller cases for profiler captures; not a bench value)")
    ap.add_argument("--no-cpu-baseline", action="store_true")
    ap.add_argument("--no-prefill", action="store_true")
    ap.add_argument("--no-other-workloads", action="store_true",
                    help="skip the compact figures of the other decode configurations")
    ap.add_argument("--kv-format", default="native", choices=["native", "fp8"],
                    help="fp8: quantised KV storage (FP8 E4M3 elements); bytes counted are the quantised cache's")
    ap.add_argument("--trace", action="store_true", help="paper-shaped serving trace instead of the decode step")
    ap.add_argument("--trace-requests", type=int, default=8)
    ap.add_argument("--trace-prompt", type=int, default=31000)
    ap.add_argument("--trace-gen", type=int, default=100)
    ap.add_argument("--trace-concurrency", type=int, default=0,
                    help="requests served at a time (0 = all at once); every layout gets the same number, so the "
                         "standard layout's cache has to fit")
    ap.add_argument("--trace-layouts", default="", help="comma-separated subset of the layouts (standard always runs)")
    args = ap.parse_args()
    if args.warmup < 3:
        args.warmup = 3
    wl = get_workload(args.workload)
    if args.batch > 0:
        wl = wl.scaled(batch=args.batch, name=f"{wl.name}_batch{args.batch}")
    if args.impl == "ours" and not args.trace and args.gpus > 1 and "WORLD_SIZE" not in os.environ:
        if torch.cuda.device_count() < args.gpus:
            raise SystemExit(f"--gpus {args.gpus}: this node shows {torch.cuda.device_count()} CUDA devices")
        raise SystemExit(spawn_replicas(args.gpus, sys.argv[1:]))
    if args.impl == "reference":
        run_reference_arm(args, wl)
    elif args.trace:
        run_trace_arm(args)
    else:
        run_gpu_arm(args, wl)


if __name__ == "__main__":
    main()

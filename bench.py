"""Benchmark of the R-KV compression step on B200: one "step" = one firing of rkv_compress (prep, scores,
select, gather) over one batch of synthetic caches.

    python bench.py [--gpus N] [--steps K] [--warmup W] [--workload NAME] [--impl reference]

Prints ONE JSON line (rank 0).  The headline workload is the largest configuration (the Qwen-14B cache shape:
12 288 head-problems of 4224 cached tokens, 26.6 GB of K+V; one compressing firing per step).  value = cached
tokens scored per second over all ranks with the inputs already in HBM; e2e = the same through the host-buffer
entry point with the copies inside the timed region; roofline = the slower of the two tensor-core scoring passes
against the measured dense bf16 peak, roofline_hbm = the HBM-bound kernels against the measured copy bandwidth;
cpu_baseline = the CPU oracle timed on this machine's host cores; configs = the other configurations (and the
default one under settings that defeat the two-pass shortcut), each with its own per-kernel table.
"""
from __future__ import annotations

import argparse
import json
import os
import statistics
import subprocess
import sys
import threading
import time

ROOT = os.path.dirname(os.path.abspath(__file__))
if ROOT not in sys.path:
    sys.path.insert(0, ROOT)

import torch  # noqa: E402

import rkv_inputs as ri  # noqa: E402

METRIC = "cached tokens scored/s (KV compressions/s alongside)"
UNIT = "tokens/s"
# DRAM traffic (dram__bytes_read.sum + dram__bytes_write.sum) per head-problem of one launch, from the ncu capture
# of a 256-head-problem slice at n = 4216 summarised in profiles/all_kernels_llama8b_b16_batch1.md.  Every kernel
# works head by head, so a full launch's traffic is this figure times the launch's head-problems (only taken for
# workloads of that cache size; the capture has G = 4, other group sizes differ only in the few KB of queries per head).
# None = the kernel has changed since the counters were taken.
NCU_TRAFFIC_PER_HEAD_N4216 = {
    "prep": 317.48e6 / 256,                   # prep kernel + the per-head key sums
    "scores_pass1": 359.29e6 / 256, "scores_list": 4.34e6 / 256,
    "scores_pass2": 375.66e6 / 256,           # both scans, the second listing and the symmetric route's two launches, as bench.py's interval has them
    "row_stats": 34.61e6 / 256, "importance": 34.63e6 / 256, "select": 8.69e6 / 256, "gather": 1001.05e6 / 256,
}
DEFAULT_WORKLOAD = "qwen14b_b32"


def parse_args():
    ap = argparse.ArgumentParser()
    ap.add_argument("--gpus", type=int, default=1)
    ap.add_argument("--steps", type=int, default=10)
    ap.add_argument("--warmup", type=int, default=5)
    ap.add_argument("--workload", default=DEFAULT_WORKLOAD, choices=[c for c in ri.SPECS if c != "tiny"])
    ap.add_argument("--no-configs", action="store_true",
                    help="only the named workload, without the other configurations under `configs`")
    ap.add_argument("--impl", default="b200", choices=["b200", "reference"])
    ap.add_argument("--beta", type=int, default=None)
    ap.add_argument("--threshold", type=float, default=None)
    ap.add_argument("--pool-w", type=int, default=None)
    ap.add_argument("--mean-then-pool", action="store_true", help="importance in Algorithm 1's order (a variant)")
    ap.add_argument("--gqa-mean-pool", action="store_true",
                    help="mean instead of max over a group's query heads in Eq. 3 (a variant)")
    ap.add_argument("--head-mean", action="store_true",
                    help="Algorithm 1's aggregated selection: one kept set per sequence from the head-averaged score")
    ap.add_argument("--no-cpu-baseline", action="store_true")
    ap.add_argument("--no-e2e", action="store_true")
    ap.add_argument("--batch", type=int, default=None, help="fewer sequences than the workload names (ncu captures)")
    ap.add_argument("--layers", type=int, default=None, help="fewer layers than the workload names (ncu captures)")
    ap.add_argument("--stream", action="store_true",
                    help="generation stream: append buffer-sized blocks of seeded K/V and fire the step after each; "
                         "reports the total compression time (the last benchmark configuration)")
    ap.add_argument("--stream-tokens", type=int, default=32768, help="tokens generated per sequence in --stream")
    ap.add_argument("--mem-gb", type=float, default=60.0, help="device memory the input replicas may take")
    return ap.parse_args()


# ------------------------------------------------------------------------------------------------- helpers
def measured_peaks():
    path = os.path.join(ROOT, "MEASURED_PEAKS.json")
    if os.path.exists(path):
        with open(path) as f:
            d = json.load(f)
        return dict(hbm_gbs=d["hbm_gbs"], bf16_tflops=d["bf16_tflops"],
                    bf16_tflops_sustained=d.get("bf16_tflops_sustained"), source="measured")
    return dict(hbm_gbs=6650.0, bf16_tflops=1590.0, bf16_tflops_sustained=1400.0, source="fallback")


class ClockSampler:
    """nvidia-smi clocks and throttle reasons of one GPU while the timed region runs."""
    FIELDS = ("clocks.sm,clocks.max.sm,power.draw,clocks_event_reasons.hw_slowdown,"
              "clocks_event_reasons.hw_thermal_slowdown,clocks_event_reasons.sw_thermal_slowdown,"
              "clocks_event_reasons.sw_power_cap")

    def __init__(self, index: int):
        self.index, self.proc, self.lines = index, None, []

    def start(self):
        try:
            self.proc = subprocess.Popen(["nvidia-smi", "-i", str(self.index), f"--query-gpu={self.FIELDS}",
                                          "--format=csv,noheader,nounits", "-lms", "100"],
                                         stdout=subprocess.PIPE, stderr=subprocess.DEVNULL, text=True)
            self.thread = threading.Thread(target=self._pump, daemon=True)
            self.thread.start()
        except OSError:
            self.proc = None

    def _pump(self):
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
        sm, mx, reasons = [], [], set()
        names = ["hw_slowdown", "hw_thermal_slowdown", "sw_thermal_slowdown", "sw_power_cap"]
        for ln in self.lines:
            parts = [x.strip() for x in ln.split(",")]
            if len(parts) < 7:
                continue
            try:
                sm.append(float(parts[0]))
                mx.append(float(parts[1]))
            except ValueError:
                continue
            for nm, val in zip(names, parts[3:7]):
                if val.lower().startswith("active"):
                    reasons.add(nm)
        return {"sm_mhz": statistics.median(sm) if sm else None, "sm_max_mhz": max(mx) if mx else None,
                "samples": len(sm), "reasons": sorted(reasons)}


def tokens_per_step(spec: ri.CacheSpec) -> int:
    return spec.head_problems * (spec.cap - spec.alpha)       # every cache is full: n = L - alpha per head


def sim_flops_per_step(spec: ri.CacheSpec) -> float:
    n = spec.cap - spec.alpha
    return 2.0 * n * n * spec.head_dim * spec.head_problems    # Eq. 5: the full n x n x d product per head


# ------------------------------------------------------------------------------------------------- reference arm
def run_reference(args, rank: int):
    """The CPU oracle as it stands, on the host cores; each step is a bounded sample of the workload."""
    if rank != 0:
        return
    import oracle
    spec = ri.SPECS[args.workload]
    n = spec.cap - spec.alpha
    cores = os.cpu_count() or 1
    # size one step to roughly a second or two: the similarity matrix costs n^2 d multiply-adds per head
    heads = max(cores, min(spec.head_problems, int(cores * 2.5e8 / (n * n * spec.head_dim)) or 1))
    seqs = max(1, heads // spec.n_kv_heads)
    small = ri.scaled(spec, layers=1, batch=seqs)
    wl = ri.make_workload(small, device="cpu", seed=ri.BASE_SEED + 77)
    K, Q = wl.k_cache.float().numpy(), wl.q_window.float().numpy()
    seq = wl.seq_lens.numpy()
    kw = dict(budget=spec.budget, alpha=spec.alpha, lam=spec.lam, W=4 if args.pool_w is None else args.pool_w,
              beta=1 if args.beta is None else args.beta, T=0.5 if args.threshold is None else args.threshold,
              mean_then_pool=args.mean_then_pool, head_mean=args.head_mean, gqa_mean_pool=args.gqa_mean_pool)
    oracle.build()
    steps, warm = max(1, min(args.steps, 5)), max(1, min(args.warmup, 1))
    for _ in range(warm):
        res = oracle.oracle_batch(K, Q, seq, want_scores=False, **kw)
    t0 = time.perf_counter()
    for _ in range(steps):
        res = oracle.oracle_batch(K, Q, seq, want_scores=False, **kw)
    dt = (time.perf_counter() - t0) / steps
    toks = small.head_problems * n
    value = toks / dt
    line = {
        "impl": "reference", "metric": METRIC, "value": value, "unit": UNIT, "n_gpus": args.gpus, "steps": steps,
        "warmup": warm, "ms_per_step": dt * 1e3, "higher_is_better": True, "scaling": "weak", "vs_baseline": None,
        "dtype": "f64", "data": "synthetic",
        "config": {"workload": args.workload, "sample": f"{small.head_problems} of {spec.head_problems} head-problems per step"},
        "compressions_per_s": small.folded_batch / dt,
        "cpu_baseline": {"value": value, "unit": UNIT, "cores": res.threads, "kind": "oracle",
                         "sample": f"{small.head_problems} head-problems x n={n} per step, {steps} steps"},
        "e2e": {"value": value, "unit": UNIT, "h2d_bytes_per_step": 0, "d2h_bytes_per_step": 0},
        "gpu_launches": 0,
    }
    print(json.dumps(line))


# ------------------------------------------------------------------------------------------------- stream mode
def stream_measure(rkv, rd, dev, rank, spec, stream_tokens):
    """A generation stream: every `buffer` tokens the caches of all sequences and layers fill up and the step fires.
    Appending the seeded blocks is not timed; each firing is bracketed by CUDA events on the call's stream."""
    k, v, seq, gen, scale = ri.stream_state(spec, device=dev, seed=ri.BASE_SEED + 5 + 1000 * rank)
    comp = rkv.Compressor(spec.folded_batch, spec.n_kv_heads, spec.n_q_heads, spec.budget, spec.buffer, spec.alpha,
                          spec.lam, dtype=spec.torch_dtype, head_dim=spec.head_dim, device=dev)
    stream = torch.cuda.current_stream()
    firings = stream_tokens // spec.buffer
    rd.barrier()
    torch.cuda.synchronize()
    total_ms, real, scored, real_ms = 0.0, 0, 0, 0.0
    for f in range(firings):
        q = ri.make_stream_block(spec, k, v, seq, gen, scale)
        live = bool((seq > spec.budget).any().item())
        e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
        e0.record(stream)
        comp.compress(k, v, q, seq, stream=stream)
        e1.record(stream)
        torch.cuda.synchronize()
        ms = e0.elapsed_time(e1)
        total_ms += ms
        if live:
            real += 1
            real_ms += ms
            scored += spec.head_problems * (spec.cap - spec.alpha)
    comp.check_status()
    rd.barrier()
    value, ms_slowest = rd.whole_job_rate(scored, total_ms, dev)
    launches = firings * rkv.rkv_launch_count_for(comp.desc, spec.budget, spec.buffer, spec.alpha, rkv.RKV_STAGE_ALL)
    cache_gib = 2 * k.numel() * k.element_size() / 2 ** 30
    del comp, k, v
    torch.cuda.empty_cache()
    return {"tokens_per_s": value, "tokens_generated_per_sequence": stream_tokens, "firings": firings,
            "compressing_firings": real, "total_compression_ms": ms_slowest,
            "ms_per_compressing_firing": real_ms / max(real, 1), "compressions": real * spec.folded_batch,
            "gpu_launches": launches, "cache_gib": cache_gib}


def run_stream(args, rkv, rd, dev, rank, world, spec):
    peaks = measured_peaks()
    sampler = ClockSampler(dev.index or 0)
    sampler.start()
    st = stream_measure(rkv, rd, dev, rank, spec, args.stream_tokens)
    clocks = sampler.stop()
    if rank == 0:
        print(json.dumps({
            "metric": METRIC, "value": st["tokens_per_s"], "unit": UNIT, "n_gpus": world, "steps": st["firings"], "warmup": 0,
            "ms_per_step": st["total_compression_ms"] / max(st["firings"], 1), "higher_is_better": True, "scaling": "weak",
            "vs_baseline": None, "dtype": "bf16", "data": "synthetic",
            "config": {"workload": spec.name + " stream", "tokens_generated_per_sequence": args.stream_tokens,
                       "head_problems_per_gpu": spec.head_problems, "budget": spec.budget, "buffer": spec.buffer,
                       "l2": f"caches of {st['cache_gib']:.1f} GiB, far beyond L2",
                       "parallelism": f"{world} independent replicas, no collective"},
            "stream": {k2: st[k2] for k2 in ("firings", "compressing_firings", "total_compression_ms",
                                             "ms_per_compressing_firing", "compressions")},
            "gpu_launches": st["gpu_launches"],
            "clocks": clocks, "peaks": peaks["source"]}))
    if torch.distributed.is_initialized():
        torch.distributed.destroy_process_group()


# ------------------------------------------------------------------------------------------------- main arm
def variant_kwargs(args, rkv):
    kw = {}
    if args.beta is not None:
        kw["beta"] = args.beta
    if args.threshold is not None:
        kw["sim_threshold"] = args.threshold
    if args.pool_w is not None:
        kw["pool_w"] = args.pool_w
    if args.mean_then_pool or args.head_mean or args.gqa_mean_pool:
        kw["flags"] = (rkv.RKV_FLAG_MEAN_THEN_POOL if args.mean_then_pool else 0) | \
                      (rkv.RKV_FLAG_HEAD_MEAN if args.head_mean else 0) | \
                      (rkv.RKV_FLAG_GQA_MEAN_POOL if args.gqa_mean_pool else 0)
    return kw


class Timed:
    """One workload resident in HBM with its pristine copy; steps restore the caches outside the timed events (or
    cycle through replicas when they fit), so that every step compresses full caches that are not in L2."""

    def __init__(self, rkv, rd, dev, wl, mem_gb, steps_needed):
        self.rkv, self.rd, self.dev, self.wl, self.spec = rkv, rd, dev, wl, wl.spec
        self.bytes_per_replica = 2 * wl.k_cache.numel() * wl.k_cache.element_size()
        n_rep = max(1, min(steps_needed, int(mem_gb * 2 ** 30) // self.bytes_per_replica))
        self.contiguous = n_rep >= steps_needed
        self.reps = [(wl.k_cache.clone(), wl.v_cache.clone(), wl.seq_lens.clone()) for _ in range(n_rep)]
        self.flush = torch.empty(256 * 2 ** 20, dtype=torch.uint8, device=dev)     # > L2 (126 MB)
        self.stream = torch.cuda.current_stream()

    def restore(self, i):
        k, v, s = self.reps[i % len(self.reps)]
        k.copy_(self.wl.k_cache)
        v.copy_(self.wl.v_cache)
        s.copy_(self.wl.seq_lens)

    def step(self, comp, i):
        k, v, s = self.reps[i % len(self.reps)]
        comp.compress(k, v, self.wl.q_window, s, stream=self.stream)

    def l2_note(self):
        return (f"{len(self.reps)} input replicas of {self.bytes_per_replica / 2**20:.0f} MiB cycled, each used once"
                if self.contiguous else "inputs restored and a 256 MiB buffer written between timed steps")

    def run_timed(self, comp, K, W, sampler=None):
        """W warm-up steps, then K steps timed with CUDA events on the launching stream; returns this rank's ms."""
        rd = self.rd
        for i in range(W):
            if not self.contiguous:
                self.restore(i)
            self.step(comp, i)
        torch.cuda.synchronize()
        comp.check_status()
        if sampler is not None:
            sampler.start()
            time.sleep(0.3)
        rd.barrier()
        torch.cuda.synchronize()
        if self.contiguous:
            e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
            e0.record(self.stream)
            for i in range(K):
                self.step(comp, W + i)
            e1.record(self.stream)
            torch.cuda.synchronize()
            ms_total = e0.elapsed_time(e1)
        else:
            ms_total = 0.0
            for i in range(K):
                self.restore(i)
                self.flush.fill_(i & 255)                   # evicts the restored caches from L2
                e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
                e0.record(self.stream)
                self.step(comp, i)
                e1.record(self.stream)
                torch.cuda.synchronize()
                ms_total += e0.elapsed_time(e1)
        rd.barrier()
        torch.cuda.synchronize()
        comp.check_status()
        return ms_total

    def close(self):
        self.reps = None
        self.flush = None
        torch.cuda.empty_cache()


def kernel_table(rkv, timed: Timed, kw, KB, peaks):
    """The same steps with an event after every kernel: per-kernel times, the work each launch had to do, and the
    rate against the roofline that bounds it."""
    spec, wl, dev = timed.spec, timed.wl, timed.dev
    comp_ev = rkv.Compressor(spec.folded_batch, spec.n_kv_heads, spec.n_q_heads, spec.budget, spec.buffer, spec.alpha,
                             spec.lam, dtype=spec.torch_dtype, head_dim=spec.head_dim, device=dev, stage_events=True, **kw)
    names = list(comp_ev.KERNEL_NAMES)
    kernel_ms = [0.0] * len(names)
    tiles_executed = pairs2 = moved_rows = 0
    for i in range(KB):
        timed.restore(i)
        timed.flush.fill_(i & 255)
        timed.step(comp_ev, i)
        torch.cuda.synchronize()
        for s_i, t in enumerate(comp_ev.kernel_ms()):
            kernel_ms[s_i] += t / KB
        if i == 0:
            tiles_executed = int(comp_ev.counters[0].item())
            pairs2 = int(comp_ev.counters[5].item())
            idx = comp_ev.out_idx
            moved_rows = int((idx != torch.arange(spec.budget, device=dev, dtype=idx.dtype)).sum().item())
    comp_ev.check_status()
    n = spec.cap - spec.alpha
    esz = wl.k_cache.element_size()
    row = spec.head_dim * esz
    wide_row = max(spec.head_dim, 128 if spec.head_dim == 64 else 0) * 2       # a row of the bf16 scoring copy (8-bit caches, d = 64)
    P = spec.head_problems
    T = (n + 127) // 128
    q_cols = -(-(spec.n_q_heads // spec.n_kv_heads) * spec.alpha // 16) * 16 + 16
    # one tile product = 128 x 128 outputs over K = 128 + 16: the head dimension plus the one extra K = 16 step that
    # folds the threshold test into the accumulator (both scoring passes issue it for every key tile)
    # (head dimension 64 runs on keys padded to 128: the padding's products are not counted as work)
    tile_flops = 2.0 * 128 * 128 * (spec.head_dim + 16)
    rule_on = comp_ev.desc.beta > 0 and comp_ev.desc.sim_threshold < 1.0
    pass1_tiles = P * T if rule_on else 0              # every row tile meets the last key tile once
    pass1_flops = pass1_tiles * tile_flops + P * T * 2.0 * 128 * q_cols * spec.head_dim
    pass2_flops = max(tiles_executed - pass1_tiles, 0) * tile_flops
    pass2_useful = pairs2 * 2.0 * 128 * (128 + 16)     # listed tokens x keys of the streamed tiles x 2 (d + 16)
    # algorithmic work per launch: bytes a kernel has to move / flops it has to execute, nothing it merely could
    work = {
        # K once; r_i, Kbar_i.Kbar_i and the 32-byte slice out.  8-bit caches and d = 64: the stored keys in and their bf16 /
        # padded copy out (written by the prep kernel itself when a stored row is 128 bytes and the capacity a whole
        # number of tiles; else by a pass of its own, and read back)
        "prep": ("hbm", P * (n * row + spec.cap * (8 + 32)) if (esz > 1 and spec.head_dim != 64) else
                 (P * (n * row + n * wide_row + spec.cap * (8 + 32)) if (row == 128 and spec.cap % 128 == 0) else
                  P * (spec.cap * row + spec.cap * wide_row + n * wide_row + spec.cap * (8 + 32)))),
        "scores_pass1": ("tensor", pass1_flops),
        "scores_list": ("hbm", P * n * 8),
        "scores_pass2": ("tensor", pass2_flops),
        "row_stats": ("hbm", P * spec.alpha * n * 4),
        "importance": ("hbm", P * (spec.alpha + 1) * n * 4),
        "select": ("hbm", P * (2 * n * 4 + spec.budget * 4)),
        "gather": ("hbm", moved_rows * row * 2 * 2 + P * spec.budget * 4),      # K and V rows that move: read + write
    }
    kernels = {}
    for nm, ms in zip(names, kernel_ms):
        bound, amount = work[nm]
        rate = amount / (ms * 1e-3) if ms > 0 else 0.0
        if bound == "tensor":
            kernels[nm] = {"ms": ms, "tflops": rate / 1e12, "frac_of_bf16_peak": rate / 1e12 / peaks["bf16_tflops"],
                           "flops_per_launch": amount}
        else:
            kernels[nm] = {"ms": ms, "gbs": rate / 1e9, "frac_of_hbm_peak": rate / 1e9 / peaks["hbm_gbs"],
                           "bytes_per_launch": amount}
    if kernel_ms[3] > 0:
        kernels["scores_pass2"]["useful_tflops"] = pass2_useful / (kernel_ms[3] * 1e-3) / 1e12
    scoring_ms = kernel_ms[1] + kernel_ms[2] + kernel_ms[3]
    scoring = {"tiles_executed": tiles_executed, "tiles_full_matrix": P * T * T,
               "pass2_token_tile_pairs": pairs2,
               "executed_tflops": (pass1_flops + pass2_flops) / (scoring_ms * 1e-3) / 1e12,
               "full_matrix_equivalent_tflops": sim_flops_per_step(spec) / (scoring_ms * 1e-3) / 1e12}
    del comp_ev
    return kernels, scoring


def rooflines(spec, kernels, scoring, peaks):
    """roofline: the slower (lower fraction of its peak) of the two tcgen05 scoring passes on the tile products it
    executed.  roofline_hbm: the HBM-bound kernels that move the bulk of the bytes."""
    cands = [nm for nm in ("scores_pass1", "scores_pass2") if kernels[nm]["ms"] > 0 and kernels[nm]["flops_per_launch"] > 0]
    n = spec.cap - spec.alpha
    per_head = NCU_TRAFFIC_PER_HEAD_N4216 if n == 4216 else {}

    def traffic(nm):
        t = per_head.get(nm)
        return None if t is None else t * spec.head_problems

    roofline = None
    if cands:
        nm = min(cands, key=lambda c: kernels[c]["frac_of_bf16_peak"])
        k = kernels[nm]
        roofline = {"kernel": nm, "bound": "tensor", "achieved": k["tflops"], "peak": peaks["bf16_tflops"],
                    "unit": "TFLOP/s", "frac": k["frac_of_bf16_peak"],
                    "peak_source": f"{peaks['source']} burst cuBLAS bf16",
                    "traffic": traffic(nm), "flops_per_launch": k["flops_per_launch"],
                    "counts": "128x128x(128+16) tile products the kernel executed (counted by the kernel) + its query products",
                    "full_matrix_equivalent_tflops": scoring["full_matrix_equivalent_tflops"],
                    "other_pass": {c: kernels[c]["frac_of_bf16_peak"] for c in cands if c != nm}}
    hbm = {}
    for nm in ("gather", "prep"):
        k = kernels[nm]
        hbm[nm] = {"bound": "hbm", "achieved": k["gbs"], "peak": peaks["hbm_gbs"], "unit": "GB/s",
                   "frac": k["frac_of_hbm_peak"], "peak_source": f"{peaks['source']} copy",
                   "traffic": traffic(nm), "bytes_per_launch": k["bytes_per_launch"]}
    return roofline, hbm


def measure_e2e(rkv, rd, dev, wl, kw, KE, toks):
    """The host-buffer entry point, copies inside the timed region (wall clock around call + synchronise)."""
    spec = wl.spec
    esz = wl.k_cache.element_size()
    row = spec.head_dim * esz
    ch = rkv.Compressor(spec.folded_batch, spec.n_kv_heads, spec.n_q_heads, spec.budget, spec.buffer, spec.alpha,
                        spec.lam, dtype=spec.torch_dtype, head_dim=spec.head_dim, device=dev, host_staging=True, **kw)
    hk = torch.empty(wl.k_cache.shape, dtype=wl.k_cache.dtype, pin_memory=True)
    hv = torch.empty(wl.v_cache.shape, dtype=wl.v_cache.dtype, pin_memory=True)
    hq = wl.q_window.cpu().pin_memory()
    hs = wl.seq_lens.cpu().pin_memory()
    hi = torch.empty(spec.folded_batch, spec.n_kv_heads, spec.budget, dtype=torch.int32).pin_memory()
    stream = torch.cuda.current_stream()
    ms_e2e = 0.0
    for i in range(KE + 1):                       # the first step warms up
        hk.copy_(wl.k_cache)
        hv.copy_(wl.v_cache)
        hs.copy_(wl.seq_lens)
        rd.barrier()
        torch.cuda.synchronize()
        t0 = time.perf_counter()
        ch.compress_host(hk, hv, hq, hs, hi, stream=stream)
        torch.cuda.synchronize()                  # the step's results are on the host from here
        if i > 0:
            ms_e2e += (time.perf_counter() - t0) * 1e3
    ch.check_status()
    e2e_value, _ = rd.whole_job_rate(toks * KE, ms_e2e, dev)
    h2d = 2 * wl.k_cache.numel() * esz + wl.q_window.numel() * esz + wl.seq_lens.numel() * 4
    d2h = 2 * spec.head_problems * spec.budget * row + spec.head_problems * spec.budget * 4 + wl.seq_lens.numel() * 4
    del ch, hk, hv
    torch.cuda.empty_cache()
    return {"value": e2e_value, "unit": UNIT, "h2d_bytes_per_step": h2d, "d2h_bytes_per_step": d2h,
            "steps": KE, "ms_per_step": ms_e2e / KE,
            "how": "rkv_compress_host from pinned host buffers; wall clock around the call and a synchronise"}


def measure_cpu(wl, desc, args):
    """The oracle as it stands on this machine's cores: a bounded sample (about 12 s) of the same workload."""
    import oracle
    spec = wl.spec
    n = spec.cap - spec.alpha
    cores = os.cpu_count() or 1
    heads = max(spec.n_kv_heads, min(spec.head_problems, int(cores * 2.5e9 / (n * n * spec.head_dim))))
    seqs = max(1, heads // spec.n_kv_heads)
    Kh = wl.k_cache[:seqs].float().cpu().numpy()
    Qh = wl.q_window[:seqs].float().cpu().numpy()
    oracle.build()
    seq_h = wl.seq_lens[:seqs].cpu().numpy()
    passes, t0 = 0, time.perf_counter()
    while passes < 1 or (time.perf_counter() - t0 < 12.0 and passes < 200):
        res = oracle.oracle_batch(Kh, Qh, seq_h, budget=spec.budget, alpha=spec.alpha, lam=spec.lam, W=desc.pool_w,
                                  beta=desc.beta, T=desc.sim_threshold, eps=desc.eps, want_scores=False,
                                  mean_then_pool=args.mean_then_pool, head_mean=args.head_mean,
                                  gqa_mean_pool=args.gqa_mean_pool)
        passes += 1
    dt = time.perf_counter() - t0
    return {"value": passes * seqs * spec.n_kv_heads * n / dt, "unit": UNIT, "cores": res.threads, "kind": "oracle",
            "sample": f"first {seqs * spec.n_kv_heads} of {spec.head_problems} head-problems, {passes} passes, {dt:.1f} s"}


def measure_attention(rkv, dev, wl, peaks, reps=5):
    """rkv_decode_attention over the workload's full caches (every K and V row read once): ms and GB/s."""
    spec = wl.spec
    d = rkv.rkv_desc_default()
    d.batch, d.n_kv_heads, d.n_q_heads = spec.folded_batch, spec.n_kv_heads, spec.n_q_heads
    d.head_dim = spec.head_dim
    d.dtype = {"bf16": rkv.RKV_BF16, "f32": rkv.RKV_F32, "fp8": rkv.RKV_FP8_E4M3}[spec.dtype]    # the caches are read as this type
    need = rkv.rkv_decode_workspace_bytes(d, spec.budget, spec.buffer)
    ws = torch.empty(max(need, 256), dtype=torch.uint8, device=dev)
    d.workspace, d.workspace_bytes = ws.data_ptr(), ws.numel()
    gen = torch.Generator(device=dev).manual_seed(ri.BASE_SEED + 99)
    q_new = torch.randn(spec.folded_batch, spec.n_q_heads, spec.head_dim, generator=gen, device=dev).to(spec.query_dtype)
    out = torch.empty(spec.folded_batch, spec.n_q_heads, spec.head_dim, dtype=torch.float32, device=dev)
    stream = torch.cuda.current_stream()
    flush = torch.empty(256 * 2 ** 20, dtype=torch.uint8, device=dev)
    ms = 0.0
    for i in range(reps + 1):
        flush.fill_(i & 255)
        e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
        e0.record(stream)
        rc = rkv.rkv_decode_attention(d, wl.k_cache, wl.v_cache, q_new, wl.seq_lens, out, spec.budget, spec.buffer, stream)
        e1.record(stream)
        torch.cuda.synchronize()
        if rc != rkv.RKV_OK:
            return {"error": rkv.rkv_status_string(rc)}
        if i > 0:
            ms += e0.elapsed_time(e1) / reps
    nbytes = 2 * wl.k_cache.numel() * wl.k_cache.element_size() + q_new.numel() * q_new.element_size() + out.numel() * 4
    gbs = nbytes / (ms * 1e-3) / 1e9
    return {"ms": ms, "gbs": gbs, "frac_of_hbm_peak": gbs / peaks["hbm_gbs"], "bytes_per_launch": nbytes,
            "what": "one decode step's attention of every sequence over its full cache (K and V read once)"}


def side_config(rkv, rd, dev, wl, kw, K, W, mem_gb, peaks):
    """A configuration other than the headline one: ms per step, rates and the per-kernel table."""
    spec = wl.spec
    timed = Timed(rkv, rd, dev, wl, mem_gb, K + W)
    comp = rkv.Compressor(spec.folded_batch, spec.n_kv_heads, spec.n_q_heads, spec.budget, spec.buffer, spec.alpha,
                          spec.lam, dtype=spec.torch_dtype, head_dim=spec.head_dim, device=dev, **kw)
    ms_total = timed.run_timed(comp, K, W)
    toks = tokens_per_step(spec)
    value, ms_slowest = rd.whole_job_rate(toks * K, ms_total, dev)
    kernels, scoring = kernel_table(rkv, timed, kw, min(K, 5), peaks)
    roofline, hbm = rooflines(spec, kernels, scoring, peaks)
    out = {"head_problems": spec.head_problems, "n": spec.cap - spec.alpha, "steps": K,
           "ms_per_step": ms_slowest / K, "tokens_per_s": value,
           "compressions_per_s": value / toks * spec.folded_batch,
           "beta": comp.desc.beta, "sim_threshold": comp.desc.sim_threshold, "l2": timed.l2_note(),
           "kernels": {nm: {k2: v2 for k2, v2 in kv.items() if not k2.endswith("_per_launch")} for nm, kv in kernels.items()},
           "scoring": scoring, "roofline": roofline and {k2: roofline[k2] for k2 in ("kernel", "achieved", "frac")},
           "roofline_hbm": {nm: {"achieved": h["achieved"], "frac": h["frac"]} for nm, h in hbm.items()}}
    del comp
    timed.close()
    if not kw:      # (once per workload, not for its variants): the decode step's attention over the same caches
        att = measure_attention(rkv, dev, wl, peaks, reps=3)
        out["decode_attention"] = {k2: att[k2] for k2 in ("ms", "gbs", "frac_of_hbm_peak", "error") if k2 in att}
    return out


def main():
    args = parse_args()
    from paper_2505_24133_b200 import dist as rd
    rank, local_rank, world = rd.env_world()
    if args.impl == "reference":
        run_reference(args, rank)
        return
    import paper_2505_24133_b200 as rkv    # fails loudly if the CUDA library is missing

    if not torch.cuda.is_available():
        raise SystemExit("bench.py needs a CUDA device (there is no CPU fallback)")
    torch.cuda.set_device(local_rank)
    dev = torch.device("cuda", local_rank)
    rank, local_rank, world = rd.init("nccl")
    spec = ri.SPECS[args.workload]
    if args.batch is not None or args.layers is not None:
        spec = ri.scaled(spec, layers=args.layers, batch=args.batch)
    if args.stream:
        run_stream(args, rkv, rd, dev, rank, world, spec)
        return
    K, W = args.steps, max(args.warmup, 3)
    peaks = measured_peaks()
    kw = variant_kwargs(args, rkv)

    # ---- the headline workload: one pristine copy per rank, restored (or replicated) so that every step compresses
    # full caches
    wl = ri.make_workload(spec, device=dev, seed=ri.BASE_SEED + 1000 * rank + list(ri.SPECS).index(args.workload))
    timed = Timed(rkv, rd, dev, wl, args.mem_gb, K + W)
    comp = rkv.Compressor(spec.folded_batch, spec.n_kv_heads, spec.n_q_heads, spec.budget, spec.buffer, spec.alpha,
                          spec.lam, dtype=spec.torch_dtype, head_dim=spec.head_dim, device=dev, **kw)
    launches_per_step = rkv.rkv_launch_count_for(comp.desc, spec.budget, spec.buffer, spec.alpha, rkv.RKV_STAGE_ALL)
    sampler = ClockSampler(local_rank)
    ms_total = timed.run_timed(comp, K, W, sampler)
    clocks = sampler.stop()
    toks = tokens_per_step(spec)
    value, ms_slowest = rd.whole_job_rate(toks * K, ms_total, dev)
    ms_per_step = ms_slowest / K
    n = spec.cap - spec.alpha

    kernels, scoring = kernel_table(rkv, timed, kw, min(K, 10), peaks)
    roofline, roofline_hbm = rooflines(spec, kernels, scoring, peaks)
    desc_view = {"pool_w": comp.desc.pool_w, "beta": comp.desc.beta, "sim_threshold": comp.desc.sim_threshold}
    l2_note = timed.l2_note()
    timed.close()

    attention = measure_attention(rkv, dev, wl, peaks)
    e2e = None
    if not args.no_e2e:
        e2e = measure_e2e(rkv, rd, dev, wl, kw, min(K, 2 if spec.head_problems > 4096 else 8), toks)
    cpu = None
    if rank == 0 and world == 1 and not args.no_cpu_baseline:
        cpu = measure_cpu(wl, comp.desc, args)
    del comp, wl
    torch.cuda.empty_cache()

    # ---- the other configurations, and the settings that defeat the two-pass shortcut, in the same run
    configs = {}
    if not args.no_configs and args.workload == DEFAULT_WORKLOAD and args.batch is None and args.layers is None and not kw:
        for name, k_side in (("llama8b_b1", 20), ("llama8b_b16", 5), ("qwen7b_b64", 5), ("mha7b_b8", 5), ("llama8b_b16_fp8", 5), ("llama1b_b64_d64", 5)):
            swl = ri.make_workload(ri.SPECS[name], device=dev, seed=ri.BASE_SEED + 1000 * rank + list(ri.SPECS).index(name))
            configs[name] = side_config(rkv, rd, dev, swl, {}, k_side, 3, args.mem_gb, peaks)
            if name == "llama8b_b16":
                configs[name + " threshold=0.9"] = side_config(rkv, rd, dev, swl, {"sim_threshold": 0.9}, 3, 3, args.mem_gb, peaks)
                configs[name + " beta=8"] = side_config(rkv, rd, dev, swl, {"beta": 8}, 3, 3, args.mem_gb, peaks)
            del swl
            torch.cuda.empty_cache()
        # the last benchmark configuration as the paper's experiments run it: a 32K-token generation stream in which
        # the step fires every `buffer` tokens (the first budget / buffer firings are no-ops); total compression time
        configs[spec.name + " stream (32768 tokens, firing every 128)"] = stream_measure(rkv, rd, dev, rank, spec, 32768)

    if rank == 0:
        line = {
            "metric": METRIC, "value": value, "unit": UNIT, "n_gpus": world, "steps": K, "warmup": W,
            "ms_per_step": ms_per_step, "higher_is_better": True, "scaling": "weak", "vs_baseline": None,
            "dtype": "bf16", "data": "synthetic",
            "config": {"workload": spec.name, "head_problems_per_gpu": spec.head_problems,
                       "layers": spec.layers, "batch": spec.batch, "n_kv_heads": spec.n_kv_heads,
                       "n_q_heads": spec.n_q_heads, "budget": spec.budget, "buffer": spec.buffer, "alpha": spec.alpha,
                       "lambda": spec.lam, **desc_view, "importance_order": "mean, then pool (Algorithm 1)"
                       if args.mean_then_pool else "pool, then mean (Eq. 4)",
                       "selection": "one set per sequence, head-averaged score (Algorithm 1)" if args.head_mean
                       else "one set per KV head",
                       "step": "one compressing firing: every cache full (budget + buffer tokens)",
                       "l2": l2_note,
                       "parallelism": f"{world} independent replicas, no collective"},
            "compressions_per_s": value / toks * spec.folded_batch,
            "head_problems_per_s": value / n,
            "gpu_launches": launches_per_step * K,
            "kernels": kernels,
            "scoring": scoring,
            "roofline": roofline,
            "roofline_hbm": roofline_hbm,
            "clocks": clocks,
            "peaks": {"hbm_gbs": peaks["hbm_gbs"], "bf16_tflops": peaks["bf16_tflops"], "source": peaks["source"]},
        }
        line["decode_attention"] = attention
        if e2e is not None:
            line["e2e"] = e2e
        if cpu is not None:
            line["cpu_baseline"] = cpu
        if configs:
            line["configs"] = configs
        print(json.dumps(line))
    if torch.distributed.is_initialized():
        torch.distributed.destroy_process_group()


if __name__ == "__main__":
    main()

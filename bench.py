"""Benchmark of the R-KV compression step on B200: one "step" = one firing of rkv_compress (prep, scores,
select, gather) over one batch of synthetic caches.

    python bench.py [--gpus N] [--steps K] [--warmup W] [--workload NAME] [--impl reference]

Prints ONE JSON line (rank 0).  value = cached tokens scored per second over all ranks with the inputs already
in HBM; e2e = the same through the host-buffer entry point with the copies inside the timed region; roofline =
the dominant kernel against the measured peak; cpu_baseline = the CPU oracle timed on this machine's host cores.
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
# DRAM traffic (dram__bytes_read.sum + dram__bytes_write.sum) of one launch, from the ncu captures summarised
# under profiles/: {workload: {kernel: bytes}}
NCU_TRAFFIC = {
    # profiles/all_kernels_llama8b_b1.md (cold caches: the scoring passes read K from DRAM there)
    # (the select stage is one kernel at this size: no row_stats / importance launches)
    "llama8b_b1": {"prep": 76.80e6, "scores_pass1": 85.95e6, "scores_list": 1.19e6, "scores_pass2": 81.84e6,
                   "select": 10.67e6, "gather": 209.43e6},
}


def parse_args():
    ap = argparse.ArgumentParser()
    ap.add_argument("--gpus", type=int, default=1)
    ap.add_argument("--steps", type=int, default=40)
    ap.add_argument("--warmup", type=int, default=5)
    ap.add_argument("--workload", default="llama8b_b1", choices=[c for c in ri.CONFIG_ORDER if c != "tiny"])
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


def local_spec(spec: ri.CacheSpec, rank: int, world: int) -> ri.CacheSpec:
    """Weak scaling: every rank gets the whole workload's shape (its own sequences), seeded by rank."""
    return spec


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
def run_stream(args, rkv, rd, dev, rank, world, spec):
    """A generation stream: every `buffer` tokens the caches of all sequences and layers fill up and the step fires.
    Appending the seeded blocks is not timed; each firing is bracketed by CUDA events on the call's stream."""
    peaks = measured_peaks()
    k, v, seq, gen, scale = ri.stream_state(spec, device=dev, seed=ri.BASE_SEED + 5 + 1000 * rank)
    comp = rkv.Compressor(spec.folded_batch, spec.n_kv_heads, spec.n_q_heads, spec.budget, spec.buffer, spec.alpha,
                          spec.lam, dtype=spec.torch_dtype, device=dev)
    stream = torch.cuda.current_stream()
    firings = args.stream_tokens // spec.buffer
    sampler = ClockSampler(dev.index or 0)
    sampler.start()
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
    clocks = sampler.stop()
    value, ms_slowest = rd.whole_job_rate(scored, total_ms, dev)
    if rank == 0:
        print(json.dumps({
            "metric": METRIC, "value": value, "unit": UNIT, "n_gpus": world, "steps": firings, "warmup": 0,
            "ms_per_step": ms_slowest / max(firings, 1), "higher_is_better": True, "scaling": "weak",
            "vs_baseline": None, "dtype": "bf16", "data": "synthetic",
            "config": {"workload": spec.name + " stream", "tokens_generated_per_sequence": args.stream_tokens,
                       "head_problems_per_gpu": spec.head_problems, "budget": spec.budget, "buffer": spec.buffer,
                       "l2": f"caches of {2 * k.numel() * k.element_size() / 2**30:.1f} GiB, far beyond L2",
                       "parallelism": f"{world} independent replicas, no collective"},
            "stream": {"firings": firings, "compressing_firings": real, "total_compression_ms": ms_slowest,
                       "ms_per_compressing_firing": real_ms / max(real, 1),
                       "compressions": real * spec.folded_batch},
            "gpu_launches": firings * rkv.rkv_launch_count_for(comp.desc, spec.budget, spec.buffer, spec.alpha, rkv.RKV_STAGE_ALL),
            "clocks": clocks, "peaks": peaks["source"]}))
    if torch.distributed.is_initialized():
        torch.distributed.destroy_process_group()


# ------------------------------------------------------------------------------------------------- main arm
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

    # ---- inputs: one pristine workload per rank, replicated so that every step compresses fresh caches
    wl = ri.make_workload(spec, device=dev, seed=ri.BASE_SEED + 1000 * rank + ri.CONFIG_ORDER.index(args.workload))
    bytes_per_replica = 2 * wl.k_cache.numel() * wl.k_cache.element_size()
    budget_bytes = int(args.mem_gb * 2 ** 30)
    n_rep = max(1, min(K + W, budget_bytes // bytes_per_replica))
    contiguous = n_rep >= K + W                     # else: restore between steps, outside the timed events
    reps = [(wl.k_cache.clone(), wl.v_cache.clone(), wl.seq_lens.clone()) for _ in range(n_rep)]
    flush = torch.empty(256 * 2 ** 20, dtype=torch.uint8, device=dev)     # > L2 (126 MB)

    def restore(i):
        reps[i][0].copy_(wl.k_cache)
        reps[i][1].copy_(wl.v_cache)
        reps[i][2].copy_(wl.seq_lens)

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
    comp = rkv.Compressor(spec.folded_batch, spec.n_kv_heads, spec.n_q_heads, spec.budget, spec.buffer, spec.alpha,
                          spec.lam, dtype=spec.torch_dtype, device=dev, **kw)
    launches_per_step = rkv.rkv_launch_count_for(comp.desc, spec.budget, spec.buffer, spec.alpha, rkv.RKV_STAGE_ALL)
    stream = torch.cuda.current_stream()

    def step(i, c=comp):
        k, v, s = reps[i % n_rep]
        c.compress(k, v, wl.q_window, s, stream=stream)

    # ---- pass A: the headline number
    for i in range(W):
        step(i)
    torch.cuda.synchronize()
    comp.check_status()
    sampler = ClockSampler(local_rank)
    sampler.start()
    time.sleep(0.3)
    rd.barrier()
    torch.cuda.synchronize()
    if contiguous:
        e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
        e0.record(stream)
        for i in range(K):
            step(W + i)
        e1.record(stream)
        torch.cuda.synchronize()
        ms_total = e0.elapsed_time(e1)
    else:
        ms_total = 0.0
        for i in range(K):
            restore(i % n_rep)
            flush.fill_(i & 255)                   # evicts the restored caches from L2
            e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
            e0.record(stream)
            step(i)
            e1.record(stream)
            torch.cuda.synchronize()
            ms_total += e0.elapsed_time(e1)
    rd.barrier()
    torch.cuda.synchronize()
    clocks = sampler.stop()
    comp.check_status()
    toks = tokens_per_step(spec)
    value, ms_slowest = rd.whole_job_rate(toks * K, ms_total, dev)
    ms_per_step = ms_slowest / K

    # ---- pass B: the same steps with per-kernel events, for the roofline of the dominant kernel
    comp_ev = rkv.Compressor(spec.folded_batch, spec.n_kv_heads, spec.n_q_heads, spec.budget, spec.buffer, spec.alpha,
                             spec.lam, dtype=spec.torch_dtype, device=dev, stage_events=True, **kw)
    names = list(comp_ev.KERNEL_NAMES)
    kernel_ms = [0.0] * len(names)
    KB = min(K, 20)
    tiles_executed = moved_rows = 0
    for i in range(KB):
        restore(i % n_rep)
        flush.fill_(i & 255)
        step(i, comp_ev)
        torch.cuda.synchronize()
        for s_i, t in enumerate(comp_ev.kernel_ms()):
            kernel_ms[s_i] += t / KB
        if i == 0:
            tiles_executed = int(comp_ev.counters[0].item())
            idx = comp_ev.out_idx
            moved_rows = int((idx != torch.arange(spec.budget, device=dev, dtype=idx.dtype)).sum().item())
    n = spec.cap - spec.alpha
    esz = wl.k_cache.element_size()
    row = spec.head_dim * esz
    P = spec.head_problems
    T = (n + 127) // 128
    depth = 1                                          # key tiles every token meets in the first scoring pass
    q_cols = -(-(spec.n_q_heads // spec.n_kv_heads) * spec.alpha // 16) * 16 + 16
    tile_flops = 2.0 * 128 ** 3
    pass1_tiles = P * sum(min(T - I, depth) for I in range(T))
    pass1_flops = pass1_tiles * tile_flops + P * T * 2.0 * 128 * q_cols * 128
    pass2_flops = max(tiles_executed - pass1_tiles, 0) * tile_flops
    # algorithmic work per launch: bytes a kernel has to move / flops it has to execute, nothing it merely could
    work = {
        "prep": ("hbm", P * (n * row + spec.cap * 8)),                          # K once; r_i and Kbar_i.Kbar_i out
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
        kernels[nm] = {"ms": ms, ("tflops" if bound == "tensor" else "gbs"): rate / (1e12 if bound == "tensor" else 1e9)}
    dom = max(range(len(names)), key=lambda s_i: kernel_ms[s_i])
    dom_name = names[dom]
    bound, amount = work[dom_name]
    full_matrix_tflops = sim_flops_per_step(spec) / ((kernel_ms[1] + kernel_ms[2] + kernel_ms[3]) * 1e-3) / 1e12
    if bound == "tensor":
        ach = kernels[dom_name]["tflops"]
        roofline = {"kernel": dom_name, "bound": "tensor", "achieved": ach, "peak": peaks["bf16_tflops"],
                    "unit": "TFLOP/s", "frac": ach / peaks["bf16_tflops"],
                    "peak_source": f"{peaks['source']} burst cuBLAS bf16",
                    "traffic": NCU_TRAFFIC.get(spec.name, {}).get(dom_name),
                    "flops_per_launch": amount}
    else:
        ach = kernels[dom_name]["gbs"]
        roofline = {"kernel": dom_name, "bound": "hbm", "achieved": ach, "peak": peaks["hbm_gbs"], "unit": "GB/s",
                    "frac": ach / peaks["hbm_gbs"], "peak_source": f"{peaks['source']} copy",
                    "traffic": NCU_TRAFFIC.get(spec.name, {}).get(dom_name), "bytes_per_launch": amount}
    scoring = {"tiles_executed": tiles_executed, "tiles_full_matrix": P * T * T,
               "executed_tflops": (pass1_flops + pass2_flops) / ((kernel_ms[1] + kernel_ms[2] + kernel_ms[3]) * 1e-3) / 1e12,
               "full_matrix_equivalent_tflops": full_matrix_tflops}

    # ---- e2e: the host-buffer entry point, copies inside the timed region
    e2e = None
    if not args.no_e2e:
        KE = min(K, 8)
        ch = rkv.Compressor(spec.folded_batch, spec.n_kv_heads, spec.n_q_heads, spec.budget, spec.buffer, spec.alpha,
                            spec.lam, dtype=spec.torch_dtype, device=dev, host_staging=True, **kw)
        hk0, hv0 = wl.k_cache.cpu(), wl.v_cache.cpu()
        hq = wl.q_window.cpu().pin_memory()
        hosts = [(hk0.clone().pin_memory(), hv0.clone().pin_memory(), wl.seq_lens.cpu().pin_memory(),
                  torch.empty(spec.folded_batch, spec.n_kv_heads, spec.budget, dtype=torch.int32).pin_memory())
                 for _ in range(min(KE + 1, 3))]

        def host_step(i):
            hk, hv, hs, hi = hosts[i % len(hosts)]
            ch.compress_host(hk, hv, hq, hs, hi, stream=stream)

        host_step(0)
        torch.cuda.synchronize()
        ms_e2e = 0.0
        for i in range(KE):
            hk, hv, hs, hi = hosts[i % len(hosts)]
            hk.copy_(hk0)
            hv.copy_(hv0)
            hs.copy_(wl.seq_lens.cpu())
            rd.barrier()
            torch.cuda.synchronize()
            t0 = time.perf_counter()
            host_step(i)
            torch.cuda.synchronize()              # the step's results are on the host from here
            ms_e2e += (time.perf_counter() - t0) * 1e3
        ch.check_status()
        e2e_value, _ = rd.whole_job_rate(toks * KE, ms_e2e, dev)
        h2d = 2 * wl.k_cache.numel() * esz + wl.q_window.numel() * esz + wl.seq_lens.numel() * 4
        d2h = 2 * spec.head_problems * spec.budget * row + spec.head_problems * spec.budget * 4 + wl.seq_lens.numel() * 4
        e2e = {"value": e2e_value, "unit": UNIT, "h2d_bytes_per_step": h2d, "d2h_bytes_per_step": d2h,
               "steps": KE, "ms_per_step": ms_e2e / KE}

    # ---- cpu baseline: the oracle on this machine's cores, a bounded sample of the same workload (rank 0, N = 1)
    cpu = None
    if rank == 0 and world == 1 and not args.no_cpu_baseline:
        import oracle
        cores = os.cpu_count() or 1
        heads = max(spec.n_kv_heads, min(spec.head_problems, int(cores * 2.5e9 / (n * n * spec.head_dim))))
        seqs = max(1, heads // spec.n_kv_heads)
        d = comp.desc
        Kh = wl.k_cache[:seqs].float().cpu().numpy()
        Qh = wl.q_window[:seqs].float().cpu().numpy()
        oracle.build()
        seq_h = wl.seq_lens[:seqs].cpu().numpy()
        passes, t0 = 0, time.perf_counter()
        while passes < 1 or (time.perf_counter() - t0 < 12.0 and passes < 200):      # about 12 s of CPU work
            res = oracle.oracle_batch(Kh, Qh, seq_h, budget=spec.budget, alpha=spec.alpha, lam=spec.lam, W=d.pool_w,
                                      beta=d.beta, T=d.sim_threshold, eps=d.eps, want_scores=False,
                                      mean_then_pool=args.mean_then_pool, head_mean=args.head_mean, gqa_mean_pool=args.gqa_mean_pool)
            passes += 1
        dt = time.perf_counter() - t0
        cpu = {"value": passes * seqs * spec.n_kv_heads * n / dt, "unit": UNIT, "cores": res.threads, "kind": "oracle",
               "sample": f"first {seqs * spec.n_kv_heads} of {spec.head_problems} head-problems, {passes} passes, {dt:.1f} s"}

    if rank == 0:
        line = {
            "metric": METRIC, "value": value, "unit": UNIT, "n_gpus": world, "steps": K, "warmup": W,
            "ms_per_step": ms_per_step, "higher_is_better": True, "scaling": "weak", "vs_baseline": None,
            "dtype": "bf16", "data": "synthetic",
            "config": {"workload": spec.name, "head_problems_per_gpu": spec.head_problems,
                       "layers": spec.layers, "batch": spec.batch, "n_kv_heads": spec.n_kv_heads,
                       "n_q_heads": spec.n_q_heads, "budget": spec.budget, "buffer": spec.buffer, "alpha": spec.alpha,
                       "lambda": spec.lam, "pool_w": comp.desc.pool_w, "beta": comp.desc.beta,
                       "sim_threshold": comp.desc.sim_threshold, "importance_order": "mean, then pool (Algorithm 1)"
                       if args.mean_then_pool else "pool, then mean (Eq. 4)",
                       "selection": "one set per sequence, head-averaged score (Algorithm 1)" if args.head_mean
                       else "one set per KV head",
                       "l2": (f"{n_rep} input replicas of {bytes_per_replica / 2**20:.0f} MiB cycled, each used once"
                              if contiguous else "inputs restored and a 256 MiB buffer written between timed steps"),
                       "parallelism": f"{world} independent replicas, no collective"},
            "compressions_per_s": value / toks * spec.folded_batch,
            "head_problems_per_s": value / n,
            "gpu_launches": launches_per_step * K,
            "kernels": kernels,
            "scoring": scoring,
            "roofline": roofline,
            "clocks": clocks,
        }
        if e2e is not None:
            line["e2e"] = e2e
        if cpu is not None:
            line["cpu_baseline"] = cpu
        print(json.dumps(line))
    if torch.distributed.is_initialized():
        torch.distributed.destroy_process_group()


if __name__ == "__main__":
    main()

#!/usr/bin/env python
"""Benchmark of the aLoRA suffix-prefill hot path on B200.

One "step" = one alora_prefill_layer call (batch metadata, gated q/k/v projection, KV append, paged
causal GQA attention) on the 8B-shape single-layer workload: 8 requests, 4096 cached base-model
positions each, 256 new suffix tokens each starting at the activation offset, rank-32 adapter.
Metric: suffix tokens per second.  Prints ONE JSON line (rank 0).

    python bench.py [--gpus N] [--steps K] [--warmup W] [--impl reference] [--no-recompute]

--impl reference times the CPU oracle (oracle/) on the host cores on a bounded sample of the same
workload.  With N > 1 (torchrun) every rank runs the same per-GPU batch on its own GPU (requests are
independent: weak scaling, no data-path collective).
"""
from __future__ import annotations

import argparse
import json
import os
import subprocess
import sys
import threading
import time

import numpy as np

ROOT = os.path.dirname(os.path.abspath(__file__))
sys.path.insert(0, ROOT)
sys.path.insert(0, os.path.join(ROOT, "tests"))

from paper_2504_12397_b200 import workloads as wl  # noqa: E402

METRIC = "aLoRA suffix-prefill tokens/s on reused base KV"
UNIT = "tokens/s"
WORKLOAD = "config2: 8B-shape layer bf16, 8 requests x (4096 cached + 256 suffix), rank-32 adapter, 16-token pages"
SEED = 2


def measured_peaks():
    p = os.path.join(ROOT, "MEASURED_PEAKS.json")
    if os.path.exists(p):
        d = json.load(open(p))
        return dict(hbm_gbs=d["hbm_gbs"], bf16_tflops=d["bf16_tflops"],
                    bf16_tflops_sustained=d.get("bf16_tflops_sustained", d["bf16_tflops"]), source="measured")
    return dict(hbm_gbs=6650.0, bf16_tflops=1590.0, bf16_tflops_sustained=1400.0, source="fallback")


class ClockSampler:
    """Samples SM clock and throttle reasons through NVML in a background thread while the timed work runs
    (read-only queries; nothing is set)."""
    REASONS = {"hw_slowdown": 0x8, "sw_power_cap": 0x4, "sw_thermal_slowdown": 0x20, "hw_thermal_slowdown": 0x40,
               "hw_power_brake_slowdown": 0x80}

    def __init__(self, gpu_index: int, period_s: float = 0.005):
        self.gpu, self.period = gpu_index, period_s
        self.sm, self.reasons, self.power = [], set(), []
        self.stop_flag = threading.Event()
        self.thread = None
        self.err = None
        self.max_mhz = None

    def _physical_index(self) -> int:
        vis = os.environ.get("CUDA_VISIBLE_DEVICES")
        if vis:
            ids = [v.strip() for v in vis.split(",") if v.strip()]
            if self.gpu < len(ids) and ids[self.gpu].isdigit():
                return int(ids[self.gpu])
        return self.gpu

    def start(self):
        try:
            import pynvml
            pynvml.nvmlInit()
            self.nv = pynvml
            vis = os.environ.get("CUDA_VISIBLE_DEVICES", "").split(",")
            if self.gpu < len(vis) and vis[self.gpu].strip().startswith("GPU-"):
                self.h = pynvml.nvmlDeviceGetHandleByUUID(vis[self.gpu].strip())
            else:
                self.h = pynvml.nvmlDeviceGetHandleByIndex(self._physical_index())
            self.max_mhz = float(pynvml.nvmlDeviceGetMaxClockInfo(self.h, pynvml.NVML_CLOCK_SM))
        except Exception as e:  # noqa: BLE001 - any NVML failure just disables the sampler
            self.err = f"nvml unavailable: {e}"
            return
        self.thread = threading.Thread(target=self._run, daemon=True)
        self.thread.start()

    def _run(self):
        nv = self.nv
        while not self.stop_flag.is_set():
            try:
                self.sm.append(float(nv.nvmlDeviceGetClockInfo(self.h, nv.NVML_CLOCK_SM)))
                bits = int(nv.nvmlDeviceGetCurrentClocksEventReasons(self.h))
                for name, bit in self.REASONS.items():
                    if bits & bit:
                        self.reasons.add(name)
                self.power.append(nv.nvmlDeviceGetPowerUsage(self.h) / 1e3)
            except Exception as e:  # noqa: BLE001
                self.err = str(e)
                return
            time.sleep(self.period)

    def stop(self) -> dict:
        if self.thread is None:
            return {"sm_mhz": None, "sm_max_mhz": None, "reasons": [self.err or "not started"], "samples": 0}
        self.stop_flag.set()
        self.thread.join(timeout=2)
        return {"sm_mhz": float(np.median(self.sm)) if self.sm else None, "sm_max_mhz": self.max_mhz,
                "reasons": sorted(self.reasons), "samples": len(self.sm),
                "power_w_max": max(self.power) if self.power else None}


def oracle_sample_rate(w: wl.Workload, pool_np: np.ndarray, n_tokens: int, requests=(0,), budget_s: float = 1e9):
    """Times the CPU oracle on the first n_tokens suffix tokens of each listed request (projection of those
    rows + their attention over the request's cache), stopping once budget_s has been spent.
    Returns (tokens/s, threads, seconds, tokens done)."""
    from oracle import Oracle
    import helpers as hp
    orc = Oracle("f64")
    shape, b = w.shape, w.batch
    total_s, done = 0.0, 0
    for r in requests:
        P = int(b.prefix_lens[r])
        q0 = int(b.query_start_loc[r])
        n = min(n_tokens, int(b.query_start_loc[r + 1]) - q0)
        K0, V0 = orc.paged_gather(pool_np, b.block_tables[r], P, shape.n_kv_heads, shape.page_size, shape.head_dim)
        sub = wl.Batch(positions=b.positions[q0:q0 + n], query_start_loc=np.array([0, n], np.int32),
                       seq_lens=np.array([P + n], np.int32), prefix_lens=b.prefix_lens[r:r + 1],
                       activation_offsets=b.activation_offsets[r:r + 1], adapter_ids=b.adapter_ids[r:r + 1],
                       block_tables=b.block_tables[r:r + 1], num_pages=b.num_pages, hidden=b.hidden[q0:q0 + n])
        t0 = time.perf_counter()
        hp.oracle_block(orc, shape, w.wqkv, w.adapters, sub, [K0], [V0])
        total_s += time.perf_counter() - t0
        done += n
        if total_s > budget_s:
            break
    return done / total_s, orc.threads, total_s, done


def run_reference(args):
    rank = int(os.environ.get("RANK", "0"))
    if rank != 0:
        return
    w = wl.config2(seed=SEED)
    rng = np.random.default_rng(SEED + 1000)
    pool_np = wl.random_kv_pool(w.shape, w.batch.num_pages, rng)
    n_tok = 32
    for _ in range(args.warmup):
        oracle_sample_rate(w, pool_np, 2)
    times = []
    for _ in range(args.steps):
        rate, threads, dt, _ = oracle_sample_rate(w, pool_np, n_tok)
        times.append(dt)
    ms = 1e3 * float(np.mean(times))
    value = n_tok / (ms / 1e3)
    sample = f"{n_tok} suffix tokens of request 0 per step (projection rows + attention over 4096+ cached keys)"
    print(json.dumps({
        "impl": "reference", "metric": METRIC, "value": value, "unit": UNIT, "n_gpus": args.gpus,
        "steps": args.steps, "warmup": args.warmup, "ms_per_step": ms, "higher_is_better": True,
        "scaling": "weak", "vs_baseline": None, "dtype": "f64", "data": "synthetic",
        "config": {"workload": WORKLOAD, "sample": sample},
        "cpu_baseline": {"value": value, "unit": UNIT, "cores": threads, "kind": "oracle", "sample": sample},
        "e2e": {"value": value, "unit": UNIT, "h2d_bytes_per_step": 0, "d2h_bytes_per_step": 0},
    }))


def main():
    ap = argparse.ArgumentParser()
    ap.add_argument("--gpus", type=int, default=1)
    ap.add_argument("--steps", type=int, default=200)
    ap.add_argument("--warmup", type=int, default=10)
    ap.add_argument("--impl", default="ours")
    ap.add_argument("--no-recompute", action="store_true", help="skip the full-LoRA recompute comparison")
    ap.add_argument("--no-cpu-baseline", action="store_true")
    ap.add_argument("--requests", type=int, default=8)
    ap.add_argument("--prefix", type=int, default=4096)
    ap.add_argument("--suffix", type=int, default=256)
    args = ap.parse_args()
    if args.impl == "reference":
        return run_reference(args)

    import torch
    import helpers as hp
    from paper_2504_12397_b200 import binding as ab
    from paper_2504_12397_b200.build import build_library
    build_library()

    world = int(os.environ.get("WORLD_SIZE", "1"))
    rank = int(os.environ.get("RANK", "0"))
    local = int(os.environ.get("LOCAL_RANK", "0"))
    torch.cuda.set_device(local)
    if world > 1:
        import torch.distributed as dist
        dist.init_process_group("nccl", device_id=torch.device("cuda", local))

    def barrier():
        if world > 1:
            dist.barrier()
        torch.cuda.synchronize()

    w = wl.config2(seed=SEED, requests=args.requests, prefix=args.prefix, suffix=args.suffix)
    shape, b = w.shape, w.batch
    rng = np.random.default_rng(SEED + 1000)
    pool_np = wl.random_kv_pool(shape, b.num_pages, rng)   # stands in for the base model's prefix cache
    T, R = b.T, b.R
    full_T = int(b.seq_lens.sum())
    cfg = ab.make_config(hidden=shape.hidden, n_q_heads=shape.n_q_heads, n_kv_heads=shape.n_kv_heads,
                         head_dim=shape.head_dim, page_size=shape.page_size, max_adapters=1, max_rank=32,
                         dtype=ab.DTYPE_BF16, device=local, max_tokens=max(T, 0 if args.no_recompute else full_T),
                         max_requests=R)
    ctx = ab.alora_create(cfg)
    wq = hp.to_dev(w.wqkv, "bf16")
    ab.alora_set_layer_weights(ctx, 0, wq)
    a = w.adapters[0]
    mats = [hp.to_dev(getattr(a, n), "bf16") for n in ("Aq", "Bq", "Ak", "Bk", "Av", "Bv")]
    ab.alora_register_adapter(ctx, 0, 0, a.rank, a.scale, *mats)
    d = hp.DevBatch(b, "bf16")
    pool = hp.to_dev(pool_np, "bf16")
    out = torch.empty((T, shape.Nq), dtype=torch.bfloat16, device="cuda")
    flush = torch.empty(256 * 1024 * 1024, dtype=torch.uint8, device="cuda")  # > L2 (126 MB)
    stream = torch.cuda.current_stream()

    def step():
        ab.alora_prefill_layer(ctx, 0, d.hidden, d.positions, d.a_req, d.ids, d.qsl, d.seq_lens, pool, d.bt,
                               d.max_blocks, b.num_pages, T, R, out, stream)

    for _ in range(args.warmup):
        step()
    torch.cuda.synchronize()
    assert ab.alora_get_status(ctx) == 0, "device-side finding during warm-up"

    # ---- timed region: K steps, each bracketed by CUDA events, L2 flushed between steps ----------
    sampler = ClockSampler(local)
    ev = [(torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)) for _ in range(args.steps)]
    ab.alora_profile_enable(ctx, True)
    launches0 = ab.alora_launch_count(ctx)
    barrier()
    sampler.start()
    for e0, e1 in ev:
        flush.zero_()
        e0.record(stream)
        step()
        e1.record(stream)
    barrier()
    clocks = sampler.stop()
    launches = ab.alora_launch_count(ctx) - launches0
    prof = ab.alora_profile_read(ctx)
    ab.alora_profile_enable(ctx, False)
    step_ms = float(np.mean([e0.elapsed_time(e1) for e0, e1 in ev]))
    if world > 1:
        tmax = torch.tensor([step_ms], device="cuda")
        dist.all_reduce(tmax, op=dist.ReduceOp.MAX)
        step_ms = float(tmax.item())
    value = world * T / (step_ms / 1e3)

    # ---- end to end through the C ABI with host buffers: H2D of the step's inputs, D2H of the result ----
    h_hidden = d.hidden.cpu().pin_memory()
    ints = [d.positions, d.a_req, d.ids, d.qsl, d.seq_lens, d.bt]
    h_ints = [t.cpu().pin_memory() for t in ints]
    h_out = torch.empty((T, shape.Nq), dtype=torch.bfloat16).pin_memory()
    d_hidden2 = torch.empty_like(d.hidden)
    d_ints2 = [torch.empty_like(t) for t in ints]

    def e2e_step():
        d_hidden2.copy_(h_hidden, non_blocking=True)
        for dst, src in zip(d_ints2, h_ints):
            dst.copy_(src, non_blocking=True)
        ab.alora_prefill_layer(ctx, 0, d_hidden2, d_ints2[0], d_ints2[1], d_ints2[2], d_ints2[3], d_ints2[4], pool,
                               d_ints2[5], d.max_blocks, b.num_pages, T, R, out, stream)
        h_out.copy_(out, non_blocking=True)

    for _ in range(3):
        e2e_step()
    barrier()
    e2e_ev = [(torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)) for _ in range(args.steps)]
    for e0, e1 in e2e_ev:
        flush.zero_()
        e0.record(stream)
        e2e_step()
        e1.record(stream)
    barrier()
    e2e_ms = float(np.mean([e0.elapsed_time(e1) for e0, e1 in e2e_ev]))
    if world > 1:
        tmax = torch.tensor([e2e_ms], device="cuda")
        dist.all_reduce(tmax, op=dist.ReduceOp.MAX)
        e2e_ms = float(tmax.item())
    h2d = h_hidden.numel() * 2 + sum(t.numel() * 4 for t in h_ints)
    d2h = h_out.numel() * 2

    # ---- roofline of the dominant kernel (per-kernel event times gathered during the timed region) ----
    peaks = measured_peaks()
    H, N, Nq, hd, Hq = shape.hidden, shape.N, shape.Nq, shape.head_dim, shape.n_q_heads
    r = a.rank
    P_, S_ = b.prefix_lens.astype(np.int64), (b.seq_lens - b.prefix_lens).astype(np.int64)
    proj_flops = 2.0 * T * H * (N + 3 * r) + 2.0 * T * r * N
    pairs = float((S_ * P_ + S_ * (S_ + 1) // 2).sum())
    attn_flops = 4.0 * hd * Hq * pairs
    attn_bytes = float(b.seq_lens.sum()) * shape.n_kv_heads * hd * 2 * 2 + 2.0 * T * Nq * 2
    kern = {k: (ms / max(n, 1)) for k, (ms, n) in prof.items() if n > 0}
    proj_ms = kern.get("project_qkv", 0.0) + kern.get("shrink", 0.0)
    attn_ms = kern.get("attention", 0.0) + kern.get("attn_merge", 0.0)
    dominant = "attention" if attn_ms >= proj_ms else "project_qkv"
    dom_ms = attn_ms if dominant == "attention" else proj_ms
    dom_flops = attn_flops if dominant == "attention" else proj_flops
    achieved = dom_flops / (dom_ms / 1e3) / 1e12 if dom_ms > 0 else 0.0
    peak = peaks["bf16_tflops"]
    roofline = {"bound": "tensor", "kernel": dominant, "achieved": achieved, "peak": peak, "unit": "TFLOP/s",
                "frac": achieved / peak, "traffic": None, "peak_source": peaks["source"] + " (burst bf16 GEMM)",
                "ms_per_launch": dom_ms,
                "per_kernel_ms": {k: round(v, 4) for k, v in kern.items()},
                "projection": {"tflops": proj_flops / (proj_ms / 1e3) / 1e12 if proj_ms else None,
                               "frac_of_tensor_peak": proj_flops / (proj_ms / 1e3) / 1e12 / peak if proj_ms else None},
                "attention": {"tflops": attn_flops / (attn_ms / 1e3) / 1e12 if attn_ms else None,
                              "hbm_gbs": attn_bytes / (attn_ms / 1e3) / 1e9 if attn_ms else None,
                              "frac_of_hbm_peak": attn_bytes / (attn_ms / 1e3) / 1e9 / peaks["hbm_gbs"] if attn_ms else None,
                              "frac_of_tensor_peak": attn_flops / (attn_ms / 1e3) / 1e12 / peak if attn_ms else None}}

    # ---- the comparison path: full-LoRA recompute of prefix + suffix on the same box -------------
    recompute = None
    if not args.no_recompute:
        fpos = torch.cat([torch.arange(int(n), dtype=torch.int32) for n in b.seq_lens]).cuda()
        fqsl = torch.from_numpy(np.concatenate([[0], np.cumsum(b.seq_lens)]).astype(np.int32)).cuda()
        g = torch.Generator(device="cuda"); g.manual_seed(SEED)
        fhid = torch.randn((full_T, H), generator=g, device="cuda", dtype=torch.float32).to(torch.bfloat16)
        fpool = torch.zeros_like(pool)
        fout = torch.empty((full_T, Nq), dtype=torch.bfloat16, device="cuda")

        def rstep():
            ab.alora_full_lora_prefill_layer(ctx, 0, fhid, fpos, d.ids, fqsl, d.seq_lens, fpool, d.bt, d.max_blocks,
                                             b.num_pages, full_T, R, fout, stream)
        rstep()
        torch.cuda.synchronize()
        n_rec = max(1, min(args.steps, 5))
        rev = [(torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)) for _ in range(n_rec)]
        for e0, e1 in rev:
            flush.zero_()
            e0.record(stream); rstep(); e1.record(stream)
        torch.cuda.synchronize()
        rms = float(np.mean([e0.elapsed_time(e1) for e0, e1 in rev]))
        recompute = {"ms_per_step": rms, "tokens": full_T, "speedup_alora_vs_full_lora": rms / step_ms,
                     "prefix_plus_suffix_over_suffix": float(full_T) / T}
    status = ab.alora_get_status(ctx)
    ab.alora_destroy(ctx)

    cpu = None
    if rank == 0 and world == 1 and not args.no_cpu_baseline:
        rate, threads, dt, done = oracle_sample_rate(w, pool_np, int(S_.max()), requests=range(R), budget_s=20.0)
        cpu = {"value": rate, "unit": UNIT, "cores": threads, "kind": "oracle",
               "sample": f"{done} of the step's {T} suffix tokens, whole requests in order (projection + attention "
                         f"over each request's cached keys), {dt:.1f} s of oracle time"}

    if rank == 0:
        print(json.dumps({
            "metric": METRIC, "value": value, "unit": UNIT, "n_gpus": world, "steps": args.steps,
            "warmup": args.warmup, "ms_per_step": step_ms, "higher_is_better": True, "scaling": "weak",
            "vs_baseline": None, "dtype": "bf16", "data": "synthetic",
            "config": {"workload": WORKLOAD, "requests_per_gpu": R, "prefix": args.prefix, "suffix": args.suffix,
                       "tokens_per_step_per_gpu": T, "l2": "flushed between steps (256 MB memset outside the timed events)",
                       "timing": "mean of per-step CUDA-event durations on the launching stream, max over ranks"},
            "clocks": clocks, "e2e": {"value": world * T / (e2e_ms / 1e3), "unit": UNIT, "h2d_bytes_per_step": h2d,
                                      "d2h_bytes_per_step": d2h, "ms_per_step": e2e_ms},
            "gpu_launches": int(launches), "roofline": roofline, "cpu_baseline": cpu,
            "full_lora_recompute": recompute, "device_status": status,
        }))
    if world > 1:
        dist.destroy_process_group()


if __name__ == "__main__":
    main()

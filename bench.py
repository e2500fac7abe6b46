#!/usr/bin/env python
"""Benchmark of the aLoRA suffix-prefill hot path on B200.

One "step" = one alora_prefill_layer call (batch metadata, gated q/k/v projection, KV append, paged
causal GQA attention) on the 8B-shape single-layer workload: 8 requests, 4096 cached base-model
positions each, 256 new suffix tokens each starting at the activation offset, rank-32 adapter.
Metric: suffix tokens per second.  Prints ONE JSON line (rank 0).

    python bench.py [--gpus N] [--steps K] [--warmup W] [--impl reference] [--no-recompute]

With --gpus N > 1 and no launcher around it, the script starts N ranks of itself (torch.distributed.run on
127.0.0.1); under torchrun it reads RANK / LOCAL_RANK / WORLD_SIZE as usual.

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

from paper_2504_12397_b200 import sharding  # noqa: E402
from paper_2504_12397_b200 import workloads as wl  # noqa: E402

METRIC = "aLoRA suffix-prefill tokens/s on reused base KV"
UNIT = "tokens/s"
WORKLOAD = "config2: 8B-shape layer bf16, 8 requests x (4096 cached + 256 suffix), rank-32 adapter, 16-token pages"
SEED = 2
NOMINAL_BF16_TFLOPS, NOMINAL_HBM_GBS = 2250.0, 8000.0   # the data-sheet figures the target statement quotes
# dram__bytes_read.sum + dram__bytes_write.sum per launch of the default workload's kernels, from the ncu captures
# summarised under profiles/ (valid only for the default requests / prefix / suffix and the kernels as profiled)
NCU_TRAFFIC_BYTES = {"attention": 159.465216e6 + 5.905408e6, "project_qkv": 99.755008e6 + 16.834816e6}


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

    def __init__(self, gpu_index: int, period_s: float = 0.002):
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
    from oracle import Adapter, Oracle
    orc = Oracle("f64")
    shape, b = w.shape, w.batch
    ads = [Adapter(a.rank, a.scale, a.Aq, a.Bq, a.Ak, a.Bk, a.Av, a.Bv) for a in w.adapters]
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
        orc.attention_block(sub.hidden, w.wqkv, shape.Nq, shape.Nkv, shape.n_q_heads, shape.n_kv_heads, shape.head_dim,
                            sub.positions, sub.query_start_loc, sub.activation_offsets, sub.adapter_ids, ads, [K0], [V0])
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
    # bounded sample: about 2000 suffix tokens over the whole run, at most 32 per step
    n_tok = max(2, min(32, 2000 // max(args.steps, 1)))
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


def launch_ranks(n: int) -> int:
    """`python bench.py --gpus N` without a launcher: start N ranks of this script on this node (one per GPU) under
    torch.distributed.run, with the same arguments, and pass their exit status on."""
    import socket
    with socket.socket() as sk:
        sk.bind(("127.0.0.1", 0))
        port = sk.getsockname()[1]
    cmd = [sys.executable, "-m", "torch.distributed.run", "--nnodes=1", f"--nproc-per-node={n}",
           "--master-addr", "127.0.0.1", "--master-port", str(port), os.path.abspath(__file__)] + sys.argv[1:]
    rc = subprocess.call(cmd)
    if rc != 0:
        sys.exit(rc)
    return rc


def dry_run(args, world: int, rank: int) -> None:
    """The multi-rank plumbing without a GPU: every rank joins the process group, takes its share of a request
    partition and its batch seed, the ranks agree on a (made-up) per-rank time by barrier + max over ranks, and rank
    0 prints the JSON line with the number of ranks that really took part.  Nothing is measured."""
    import torch
    import torch.distributed as dist
    if world > 1:
        dist.init_process_group(args.backend)
    try:
        lo, hi = sharding.partition_requests(args.requests * world, world)[rank]
        fake_ms = 1.0 + rank
        if world > 1:
            dist.barrier()
        ms = sharding.max_over_ranks(fake_ms)
        took_part = torch.ones(1, dtype=torch.int64)
        if world > 1:
            dist.all_reduce(took_part)
        if rank == 0:
            print(json.dumps({"metric": METRIC, "value": None, "unit": UNIT, "n_gpus": int(took_part.item()),
                              "steps": args.steps, "warmup": args.warmup, "ms_per_step": ms, "scaling": "weak",
                              "dry_run": True, "backend": args.backend if world > 1 else None,
                              "config": {"workload": WORKLOAD, "requests_per_gpu": hi - lo,
                                         "rank_seeds": [sharding.rank_seed(SEED, r) for r in range(world)]}}))
    finally:
        if world > 1:
            dist.destroy_process_group()


def fractions(peaks, roofline, sustained, config3, decode, short, recompute_8k, stack_8k, stack, evaluators,
              evaluators_stack=None, mlp_adapters=None, regime2=None):
    """Compact summary of the roofline fractions and speed-ups of all legs (None where a leg did not run)."""
    r3 = lambda x: None if x is None else round(float(x), 3)   # noqa: E731
    out = {"peaks": {"bf16_tflops": peaks["bf16_tflops"], "bf16_tflops_sustained": peaks["bf16_tflops_sustained"],
                     "hbm_gbs": peaks["hbm_gbs"], "source": peaks["source"]},
           "config2_projection_tensor": r3(roofline["projection"]["frac_of_tensor_peak"]),
           "config2_attention_tensor": r3(roofline["attention"]["frac_of_tensor_peak"])}
    if sustained:
        out["config2_step_of_sustained_tensor"] = r3(sustained["frac_of_sustained_bf16_peak"])
    if config3:
        out["config3_projection_tensor"] = r3(config3["projection_frac_of_tensor_peak"])
        out["config3_attention_tensor"] = r3(config3["attention_frac_of_tensor_peak"])
        out["config3_tokens_per_s"] = r3(config3["suffix_tokens_per_s"])
    if decode:
        out["config5_decode_attention_hbm"] = r3(decode["attention_frac_of_hbm_peak"])
        out["config5_decode_ms_per_step"] = r3(decode["ms_per_step"])
        out["config5_decode_projection_ms"] = r3(decode["per_kernel_ms"].get("project_qkv", 0.0) + decode["per_kernel_ms"].get("shrink", 0.0))
    if short:
        for s_ in short:
            key = f"short_{s_['requests']}x{s_['suffix']}" + ("" if s_["prefix"] == 4096 else f"_at{s_['prefix']}")
            out[key + "_attention_hbm"] = r3(s_["attention_frac_of_hbm_peak"])
            out[key + "_ms_per_step"] = r3(s_["ms_per_step"])
            out[key + "_projection_ms"] = r3(s_["per_kernel_ms"].get("project_qkv", 0.0) + s_["per_kernel_ms"].get("shrink", 0.0))
    if regime2:
        out["chunk_straddling_ms_per_step"] = r3(regime2["ms_per_step"])
        out["chunk_straddling_vs_activation_at_chunk_start"] = r3(regime2["ms_per_step"] / regime2["ms_per_step_activation_at_chunk_start"])
    if recompute_8k:
        out["speedup_8k_prefix_qkv_attention"] = r3(recompute_8k["speedup_alora_vs_full_lora"])
    if stack_8k:
        out["speedup_8k_prefix_whole_layers"] = r3(stack_8k["speedup_alora_vs_full_lora"])
        out["flop_ratio_8k_prefix_whole_layers"] = r3(stack_8k["flop_ratio"])
        out["token_ratio_8k_prefix"] = r3(stack_8k["prefix_plus_suffix_over_suffix"])
    if mlp_adapters and mlp_adapters.get("with_mlp_adapters"):
        out["mlp_adapters_alora_overhead"] = r3(mlp_adapters["with_mlp_adapters"]["alora_overhead"])
        out["mlp_adapters_recompute_overhead"] = r3(mlp_adapters["with_mlp_adapters"]["recompute_overhead"])
        out["speedup_8k_prefix_mlp_adapters"] = r3(mlp_adapters["with_mlp_adapters"]["speedup_alora_vs_full_lora"])
    if stack:
        out["speedup_config4_stack"] = r3(stack["speedup_alora_vs_full_lora"])
        out["flop_ratio_config4_stack"] = r3(stack["flop_ratio"])
    if evaluators:
        out["evaluator_stage_speedup"] = [r3(e["evaluator_stage_speedup"]) for e in evaluators]
        out["evaluator_pipeline_speedup"] = [r3(e["pipeline_speedup"]) for e in evaluators]
    if evaluators_stack:
        out["evaluator_stage_speedup_32_layers"] = [r3(e["evaluator_stage_speedup"]) for e in evaluators_stack]
        out["evaluator_pipeline_speedup_32_layers"] = [r3(e["pipeline_speedup"]) for e in evaluators_stack]
    return out


class L2Flush:
    """Empties the L2 of a step's inputs between timed steps: a 256 MB memset (twice the 126 MB L2), then a read
    sweep over a second 256 MB buffer.  The memset alone leaves the L2 full of DIRTY lines, whose write-back the next
    kernel's first 126 MB of reads would pay for, which no serving step does; after the read sweep the L2 holds clean
    lines of a buffer nobody uses.  `zero_()` keeps the call sites those of a plain buffer."""

    def __init__(self, how="write+read"):
        import torch
        self.how = how
        self.w = torch.empty(256 * 1024 * 1024, dtype=torch.uint8, device="cuda")
        self.r = torch.zeros(64 * 1024 * 1024, dtype=torch.float32, device="cuda") if how == "write+read" else None
        self.acc = None

    def zero_(self):
        self.w.zero_()
        if self.r is not None:
            self.acc = self.r.sum()


def attention_ms(kern):
    """Time of the attention kernel that did the batch's work, from the library's per-family event pairs.  A layer call
    launches the tensor-core kernel and the few-row kernel one after the other; when one of them found an empty work
    list its event pair holds a few microseconds of launch and event overhead, which is not the other kernel's time:
    then the working kernel's pair alone counts.  When both had work (mixed batches) the two add up."""
    tc, few = kern.get("attention", 0.0), kern.get("attention_few_row", 0.0)
    return max(tc, few) if min(tc, few) < 0.25 * max(tc, few) else tc + few


def _events(n):
    import torch
    return [(torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)) for _ in range(n)]


def timed(step, n, stream, flush):
    """Mean CUDA-event duration (ms) of n calls of step() on `stream`, L2 flushed before each call."""
    import torch
    ev = _events(n)
    for e0, e1 in ev:
        if flush is not None:
            flush.zero_()
        e0.record(stream)
        step()
        e1.record(stream)
    torch.cuda.synchronize()
    return float(np.mean([e0.elapsed_time(e1) for e0, e1 in ev]))


def profiled(ab, ctx, step, n, flush):
    """Per kernel family: mean milliseconds per step over n steps (event pairs recorded by the library)."""
    import torch
    ab.alora_profile_enable(ctx, True)
    for _ in range(n):
        if flush is not None:
            flush.zero_()
        step()
    torch.cuda.synchronize()
    prof = ab.alora_profile_read(ctx)
    ab.alora_profile_enable(ctx, False)
    return {k: ms / n for k, (ms, cnt) in prof.items() if cnt > 0}


class PrefillCase:
    """Device buffers of one suffix-prefill batch at the 8B layer shape plus its full-LoRA recompute twin."""

    def __init__(self, hp, shape, requests, prefix, suffix, seed, with_recompute, activation_shift=0, shuffle_pages=False):
        import torch
        self.w = wl.config2(seed=seed, requests=requests, prefix=prefix, suffix=suffix, activation_shift=activation_shift,
                            shuffle_pages=shuffle_pages)
        b = self.b = self.w.batch
        self.T, self.R = b.T, b.R
        self.full_T = int(b.seq_lens.sum())
        self.d = hp.DevBatch(b, "bf16")
        g = torch.Generator(device="cuda"); g.manual_seed(seed + 1000)
        # stands in for the base model's prefix cache: N(0,1) values (the byte and flop counts do not depend on them)
        self.pool = torch.randn((b.num_pages, 2, shape.n_kv_heads, shape.page_size, shape.head_dim), generator=g,
                                device="cuda", dtype=torch.float32).to(torch.bfloat16)
        self.out = torch.empty((self.T, shape.Nq), dtype=torch.bfloat16, device="cuda")
        if with_recompute:
            self.fpos = torch.cat([torch.arange(int(n), dtype=torch.int32) for n in b.seq_lens]).cuda()
            self.fqsl = torch.from_numpy(np.concatenate([[0], np.cumsum(b.seq_lens)]).astype(np.int32)).cuda()
            self.fhid = torch.randn((self.full_T, shape.hidden), generator=g, device="cuda",
                                    dtype=torch.float32).to(torch.bfloat16)
            self.fpool = torch.zeros_like(self.pool)
            self.fout = torch.empty((self.full_T, shape.Nq), dtype=torch.bfloat16, device="cuda")

    def step(self, ab, ctx, stream):
        d, b = self.d, self.b
        ab.alora_prefill_layer(ctx, 0, d.hidden, d.positions, d.a_req, d.ids, d.qsl, d.seq_lens, self.pool, d.bt,
                               d.max_blocks, b.num_pages, self.T, self.R, self.out, stream)

    def recompute_step(self, ab, ctx, stream):
        d, b = self.d, self.b
        ab.alora_full_lora_prefill_layer(ctx, 0, self.fhid, self.fpos, d.ids, self.fqsl, d.seq_lens, self.fpool, d.bt,
                                         d.max_blocks, b.num_pages, self.full_T, self.R, self.fout, stream)

    def flops_bytes(self, shape, rank):
        b = self.b
        H, N, Nq, hd, Hq = shape.hidden, shape.N, shape.Nq, shape.head_dim, shape.n_q_heads
        P_, S_ = b.prefix_lens.astype(np.int64), (b.seq_lens - b.prefix_lens).astype(np.int64)
        proj = 2.0 * self.T * H * (N + 3 * rank) + 2.0 * self.T * rank * N
        pairs = float((S_ * P_ + S_ * (S_ + 1) // 2).sum())
        attn = 4.0 * hd * Hq * pairs
        kv_bytes = float(b.seq_lens.sum()) * shape.n_kv_heads * hd * 2 * 2
        return proj, attn, kv_bytes + 2.0 * self.T * Nq * 2


def decode_leg(ab, hp, ctx, shape, stream, flush, peaks, steps=256, seed=5, ctx_max=32768):
    """Config 5: 64 requests (base + 4 rank-32 adapters), contexts U[1024, 32768], one token per request per
    step, `steps` steps with the cache growing by one position per step."""
    import torch
    rng = np.random.default_rng(seed)
    R = 64
    ctx_len = rng.integers(min(1024, ctx_max), ctx_max + 1, R)
    ids = rng.integers(-1, 4, R).astype(np.int32)
    a_req = np.maximum(ctx_len - 1 - rng.integers(0, 64, R), 0).astype(np.int32)
    ps = shape.page_size
    blocks = (ctx_len + steps + ps - 1) // ps
    num_pages = int(blocks.sum()) + 3
    order = rng.permutation(num_pages)
    bt = np.zeros((R, int(blocks.max())), np.int32)
    nxt = 0
    for r in range(R):
        bt[r, :blocks[r]] = order[nxt:nxt + blocks[r]]
        nxt += int(blocks[r])
    g = torch.Generator(device="cuda"); g.manual_seed(seed)
    pool = torch.empty((num_pages, 2, shape.n_kv_heads, ps, shape.head_dim), device="cuda", dtype=torch.bfloat16)
    for i in range(0, num_pages, 8192):  # filled in slices: no fp32 copy of the whole pool
        n = min(8192, num_pages - i)
        pool[i:i + n] = torch.randn((n,) + tuple(pool.shape[1:]), generator=g, device="cuda",
                                    dtype=torch.float32).to(torch.bfloat16)
    hidden = torch.randn((R, shape.hidden), generator=g, device="cuda", dtype=torch.float32).to(torch.bfloat16)
    out = torch.empty((R, shape.Nq), dtype=torch.bfloat16, device="cuda")
    # positions / sequence lengths of every step, resident on the device
    pos_all = torch.from_numpy((ctx_len[None, :] - 1 + np.arange(steps)[:, None]).astype(np.int32)).cuda()
    len_all = (pos_all + 1).contiguous()
    d_bt, d_ids, d_areq = hp.idev(bt), hp.idev(ids), hp.idev(a_req)

    def run(n):
        for i in range(n):
            ab.alora_decode_step(ctx, 0, hidden, pos_all[i], d_areq, d_ids, len_all[i], pool, d_bt, bt.shape[1],
                                 num_pages, R, out, stream)
    run(min(8, steps))
    torch.cuda.synchronize()
    assert ab.alora_get_status(ctx) == 0, "device-side finding in the decode leg"
    e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
    e0.record(stream); run(steps); e1.record(stream)
    torch.cuda.synchronize()
    ms = e0.elapsed_time(e1) / steps
    kern = profiled(ab, ctx, lambda: run(1), 32, None)
    attn_ms = attention_ms(kern)
    kv_bytes = float((ctx_len + steps / 2.0).sum()) * shape.n_kv_heads * shape.head_dim * 2 * 2
    kv_bytes_prof = float(ctx_len.sum()) * shape.n_kv_heads * shape.head_dim * 2 * 2
    gbs = kv_bytes_prof / (attn_ms / 1e3) / 1e9 if attn_ms else None
    return {"workload": f"config5: {R} requests, contexts U[1024,{ctx_max}] (mean {ctx_len.mean():.0f}), base + 4 rank-32 "
                        f"adapters, {steps} steps, shuffled 16-token pages; the {kv_bytes_prof / 1e9:.2f} GB cache read per "
                        "step exceeds L2",
            "ms_per_step": ms, "decode_tokens_per_s": R / (ms / 1e3),
            "kv_bytes_per_step": kv_bytes, "per_kernel_ms": {k: round(v, 4) for k, v in kern.items()},
            "attention_hbm_gbs": gbs, "attention_frac_of_hbm_peak": gbs / peaks["hbm_gbs"] if gbs else None,
            "step_hbm_gbs": (kv_bytes + 2.0 * shape.N * shape.hidden) / (ms / 1e3) / 1e9,
            "peak_source": peaks["source"]}


def parse_short_case(text):
    """'8x4' -> (8 requests, 4 new tokens, 4096 cached); '64x16@16384' names the cached length too."""
    shape, _, prefix = text.partition("@")
    r, s = (int(v) for v in shape.split("x"))
    return r, s, int(prefix) if prefix else 4096


def short_suffix_leg(ab, hp, ctx, shape, stream, flush, peaks, requests, prefix, suffix, seed=7, activation_shift=0,
                     shuffle_pages=False):
    """The paper-shaped short invocation: `suffix` new tokens per request on a reused cache (HBM-bound attention).
    With `activation_shift` the adapter activates that many tokens into the new chunk (an uncached context tail
    prefilled with the base weights in the same call as the invocation)."""
    c = PrefillCase(hp, shape, requests, prefix, suffix, seed, with_recompute=False, activation_shift=activation_shift,
                    shuffle_pages=shuffle_pages)
    for _ in range(5):
        c.step(ab, ctx, stream)
    ms = timed(lambda: c.step(ab, ctx, stream), 50, stream, flush)
    kern = profiled(ab, ctx, lambda: c.step(ab, ctx, stream), 50, flush)
    attn_ms = attention_ms(kern)
    _, _, attn_bytes = c.flops_bytes(shape, 32)
    gbs = attn_bytes / (attn_ms / 1e3) / 1e9 if attn_ms else None
    return {"requests": requests, "prefix": prefix, "suffix": suffix, "activation_shift": activation_shift,
            "pages": "shuffled" if shuffle_pages else "contiguous", "ms_per_step": ms,
            "tokens_per_s": c.T / (ms / 1e3), "per_kernel_ms": {k: round(v, 4) for k, v in kern.items()},
            "attention_hbm_gbs": gbs, "attention_frac_of_hbm_peak": gbs / peaks["hbm_gbs"] if gbs else None}


def config3_leg(ab, hp, stream, local, flush, peaks, seed=3):
    """Config 3: ragged multi-adapter batch at the 8B layer shape: 32 requests over adapters of ranks 8/16/32/64,
    prefixes U[512, 16384], suffixes U[16, 512], activation at the prefix end, shuffled 16-token pages."""
    import torch
    w = wl.config3(seed=seed)
    shape, b = w.shape, w.batch
    cfg = ab.make_config(hidden=shape.hidden, n_q_heads=shape.n_q_heads, n_kv_heads=shape.n_kv_heads,
                         head_dim=shape.head_dim, page_size=shape.page_size, max_adapters=len(w.adapters), max_rank=64,
                         dtype=ab.DTYPE_BF16, device=local, max_tokens=b.T, max_requests=b.R)
    ctx = ab.alora_create(cfg)
    try:
        wq = hp.to_dev(w.wqkv, "bf16")
        ab.alora_set_layer_weights(ctx, 0, wq)
        keep = []
        for i, a in enumerate(w.adapters):
            mats = [hp.to_dev(getattr(a, n), "bf16") for n in ("Aq", "Bq", "Ak", "Bk", "Av", "Bv")]
            keep.append(mats)
            ab.alora_register_adapter(ctx, i, 0, a.rank, a.scale, *mats)
        d = hp.DevBatch(b, "bf16")
        g = torch.Generator(device="cuda"); g.manual_seed(seed + 1000)
        pool = torch.empty((b.num_pages, 2, shape.n_kv_heads, shape.page_size, shape.head_dim), device="cuda", dtype=torch.bfloat16)
        for i in range(0, b.num_pages, 8192):
            n = min(8192, b.num_pages - i)
            pool[i:i + n] = torch.randn((n,) + tuple(pool.shape[1:]), generator=g, device="cuda", dtype=torch.float32).to(torch.bfloat16)
        out = torch.empty((b.T, shape.Nq), dtype=torch.bfloat16, device="cuda")

        def step():
            ab.alora_prefill_layer(ctx, 0, d.hidden, d.positions, d.a_req, d.ids, d.qsl, d.seq_lens, pool, d.bt,
                                   d.max_blocks, b.num_pages, b.T, b.R, out, stream)
        for _ in range(5):
            step()
        ms = timed(step, 30, stream, flush)
        kern = profiled(ab, ctx, step, 30, flush)
        status = ab.alora_get_status(ctx)
    finally:
        ab.alora_destroy(ctx)
    H, N, hd, Hq = shape.hidden, shape.N, shape.head_dim, shape.n_q_heads
    P_, S_ = b.prefix_lens.astype(np.int64), (b.seq_lens - b.prefix_lens).astype(np.int64)
    ranks = np.array([w.adapters[k].rank for k in b.adapter_ids], np.int64)
    proj = float((2.0 * S_ * H * (N + 3 * ranks) + 2.0 * S_ * ranks * N).sum())
    attn = 4.0 * hd * Hq * float((S_ * P_ + S_ * (S_ + 1) // 2).sum())
    kv_bytes = float(b.seq_lens.sum()) * shape.n_kv_heads * hd * 2 * 2 + 2.0 * b.T * shape.Nq * 2
    proj_ms = kern.get("project_qkv", 0.0) + kern.get("shrink", 0.0)
    attn_ms = attention_ms(kern)
    peak = peaks["bf16_tflops"]
    return {"workload": f"config3: {b.R} requests over adapters of ranks 8/16/32/64, prefixes U[512,16384] (sum "
                        f"{int(P_.sum())}), suffixes U[16,512] (sum {b.T}), shuffled 16-token pages; KV read "
                        f"{kv_bytes / 1e9:.2f} GB per step exceeds L2",
            "ms_per_step": ms, "suffix_tokens_per_s": b.T / (ms / 1e3),
            "per_kernel_ms": {k: round(v, 4) for k, v in kern.items()},
            "projection_tflops": proj / (proj_ms / 1e3) / 1e12 if proj_ms else None,
            "projection_frac_of_tensor_peak": proj / (proj_ms / 1e3) / 1e12 / peak if proj_ms else None,
            "attention_tflops": attn / (attn_ms / 1e3) / 1e12 if attn_ms else None,
            "attention_frac_of_tensor_peak": attn / (attn_ms / 1e3) / 1e12 / peak if attn_ms else None,
            "attention_hbm_gbs": kv_bytes / (attn_ms / 1e3) / 1e9 if attn_ms else None,
            "attention_frac_of_hbm_peak": kv_bytes / (attn_ms / 1e3) / 1e9 / peaks["hbm_gbs"] if attn_ms else None,
            "step_tflops": (proj + attn) / (ms / 1e3) / 1e12, "device_status": status}


def sustained_leg(step, stream, flush, local, min_seconds, step_flops, peaks):
    """The headline step repeated until at least `min_seconds` of step time have been timed (per-step CUDA events,
    L2 flushed between steps), with the SM clock sampled every millisecond: the layer call under the power cap."""
    import torch
    sampler = ClockSampler(local, period_s=0.001)
    sampler.start()
    total_ms, times = 0.0, []
    while total_ms < min_seconds * 1e3 and len(times) < 200000:
        n = 200
        ev = _events(n)
        for e0, e1 in ev:
            flush.zero_()
            e0.record(stream)
            step()
            e1.record(stream)
        torch.cuda.synchronize()
        batch = [e0.elapsed_time(e1) for e0, e1 in ev]
        times += batch
        total_ms += sum(batch)
    clocks = sampler.stop()
    ms = float(np.mean(times))
    tail = float(np.mean(times[len(times) // 2:]))   # the second half: clocks have settled
    mhz = clocks.get("sm_mhz")
    return {"steps": len(times), "timed_seconds": total_ms / 1e3, "ms_per_step": ms, "ms_per_step_second_half": tail,
            "sm_mhz_median": mhz, "ms_x_sm_mhz": ms * mhz if mhz else None, "clocks": clocks,
            "step_tflops": step_flops / (tail / 1e3) / 1e12,
            "frac_of_sustained_bf16_peak": step_flops / (tail / 1e3) / 1e12 / peaks["bf16_tflops_sustained"],
            "peak": peaks["bf16_tflops_sustained"], "peak_source": peaks["source"] + " (sustained bf16 GEMM)"}


def evaluator_leg(ab, hp, shape, stream, local, n_eval, seed=9, convs=8, prompt=4096, gen=256, inv=16, eval_steps=16):
    """The paper's evaluator workload on one layer: `convs` conversations get a base-model prefill of `prompt` tokens
    and `gen` base decode steps; then `n_eval` adapters each read the conversation and answer: `inv` invocation
    tokens prefilled, `eval_steps` tokens decoded.  aLoRA: the evaluators' block tables point at the conversation's
    own pages (the base model's cache, reused as it is) and only the invocation is prefilled, adapted from its
    first token on.  LoRA: every evaluator prefills prompt + generation + invocation again with its adapter on all
    tokens, into pages of its own.  Both pipelines are timed as a whole with CUDA events."""
    import torch
    rng = np.random.default_rng(seed)
    ps = shape.page_size
    ctx_len = prompt + gen
    assert ctx_len % ps == 0, "the evaluators' own tokens start on a fresh page"
    R2 = convs * n_eval
    conv_blocks, own_blocks = ctx_len // ps, (inv + eval_steps + ps - 1) // ps
    full_blocks = conv_blocks + own_blocks
    num_pages = convs * conv_blocks + R2 * own_blocks + R2 * full_blocks + 3
    order = rng.permutation(num_pages).astype(np.int32)
    nxt = 0

    def take(n):
        nonlocal nxt
        out = order[nxt:nxt + n]
        nxt += n
        return out
    bt_conv = np.zeros((convs, full_blocks), np.int32)
    for c in range(convs):
        bt_conv[c, :conv_blocks] = take(conv_blocks)
    bt_alora = np.zeros((R2, full_blocks), np.int32)
    bt_lora = np.zeros((R2, full_blocks), np.int32)
    for c in range(convs):
        for n in range(n_eval):
            r = c * n_eval + n
            bt_alora[r, :conv_blocks] = bt_conv[c, :conv_blocks]
            bt_alora[r, conv_blocks:] = take(own_blocks)
            bt_lora[r] = take(full_blocks)
    ids_eval = np.tile(np.arange(n_eval, dtype=np.int32), convs)
    T_re = R2 * (ctx_len + inv)
    cfg = ab.make_config(hidden=shape.hidden, n_q_heads=shape.n_q_heads, n_kv_heads=shape.n_kv_heads,
                         head_dim=shape.head_dim, page_size=ps, max_adapters=max(n_eval, 1), max_rank=32,
                         dtype=ab.DTYPE_BF16, device=local, max_tokens=max(T_re, convs * prompt), max_requests=max(R2, convs))
    ctx = ab.alora_create(cfg)
    keep = []
    g = torch.Generator(device="cuda"); g.manual_seed(seed)

    def rnd(*dims, std=1.0):
        return (torch.randn(dims, generator=g, device="cuda", dtype=torch.float32) * std).to(torch.bfloat16)
    wq = rnd(shape.N, shape.hidden, std=0.02)
    ab.alora_set_layer_weights(ctx, 0, wq)
    for i in range(n_eval):
        mats = []
        for blk in (shape.Nq, shape.Nkv, shape.Nkv):
            mats += [rnd(32, shape.hidden, std=0.02), rnd(blk, 32, std=0.02)]
        keep.append(mats)
        ab.alora_register_adapter(ctx, i, 0, 32, 1.0, *mats)
    pool = torch.zeros((num_pages, 2, shape.n_kv_heads, ps, shape.head_dim), device="cuda", dtype=torch.bfloat16)
    hid = rnd(max(T_re, convs * prompt), shape.hidden)
    out = torch.empty((max(T_re, convs * prompt), shape.Nq), dtype=torch.bfloat16, device="cuda")
    i32 = lambda a: hp.idev(np.ascontiguousarray(a, dtype=np.int32))  # noqa: E731
    # phase 1: base prefill of the prompts
    p1 = dict(pos=i32(np.tile(np.arange(prompt), convs)), qsl=i32(np.arange(convs + 1) * prompt),
              lens=i32(np.full(convs, prompt)), ids=i32(np.full(convs, -1)), bt=i32(bt_conv))
    # phase 2: base decode steps
    p2_pos = i32(prompt + np.arange(gen)[:, None] + np.zeros((1, convs), np.int64))
    p2_len = (p2_pos + 1).contiguous()
    areq_conv = i32(np.zeros(convs))
    # phase 3 (aLoRA): invocation prefill on the reused cache, adapted from its first token on
    p3 = dict(pos=i32(np.tile(ctx_len + np.arange(inv), R2)), qsl=i32(np.arange(R2 + 1) * inv),
              lens=i32(np.full(R2, ctx_len + inv)), ids=i32(ids_eval), areq=i32(np.full(R2, ctx_len)), bt=i32(bt_alora))
    # phase 3' (LoRA): the whole sequence again with the adapter on every token
    L3 = ctx_len + inv
    p3l = dict(pos=i32(np.tile(np.arange(L3), R2)), qsl=i32(np.arange(R2 + 1) * L3), lens=i32(np.full(R2, L3)),
               ids=i32(ids_eval), bt=i32(bt_lora))
    # phase 4: the evaluators' decode steps (aLoRA: gate opens at the invocation; LoRA: open everywhere)
    p4_pos = i32(L3 + np.arange(eval_steps)[:, None] + np.zeros((1, R2), np.int64))
    p4_len = (p4_pos + 1).contiguous()
    areq_open = i32(np.zeros(R2))

    def base_phases():
        ab.alora_full_lora_prefill_layer(ctx, 0, hid, p1["pos"], p1["ids"], p1["qsl"], p1["lens"], pool, p1["bt"],
                                         full_blocks, num_pages, convs * prompt, convs, out, stream)
        for i in range(gen):
            ab.alora_decode_step(ctx, 0, hid, p2_pos[i], areq_conv, p1["ids"], p2_len[i], pool, p1["bt"], full_blocks,
                                 num_pages, convs, out, stream)

    def alora_eval():
        ab.alora_prefill_layer(ctx, 0, hid, p3["pos"], p3["areq"], p3["ids"], p3["qsl"], p3["lens"], pool, p3["bt"],
                               full_blocks, num_pages, R2 * inv, R2, out, stream)
        for i in range(eval_steps):
            ab.alora_decode_step(ctx, 0, hid, p4_pos[i], p3["areq"], p3["ids"], p4_len[i], pool, p3["bt"], full_blocks,
                                 num_pages, R2, out, stream)

    def lora_eval():
        ab.alora_full_lora_prefill_layer(ctx, 0, hid, p3l["pos"], p3l["ids"], p3l["qsl"], p3l["lens"], pool, p3l["bt"],
                                         full_blocks, num_pages, T_re, R2, out, stream)
        for i in range(eval_steps):
            ab.alora_decode_step(ctx, 0, hid, p4_pos[i], areq_open, p3l["ids"], p4_len[i], pool, p3l["bt"], full_blocks,
                                 num_pages, R2, out, stream)

    def once(fn, reps):
        fn()
        torch.cuda.synchronize()
        e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
        e0.record(stream)
        for _ in range(reps):
            fn()
        e1.record(stream)
        torch.cuda.synchronize()
        return e0.elapsed_time(e1) / reps
    base_ms = once(base_phases, 2)
    alora_ms = once(alora_eval, 5)
    lora_ms = once(lora_eval, 2)
    status = ab.alora_get_status(ctx)
    finite = bool(torch.isfinite(out[:R2].float()).all())
    ab.alora_destroy(ctx)
    page_bytes = 2 * shape.n_kv_heads * ps * shape.head_dim * 2
    return {"workload": f"one 8B-shape layer: {convs} conversations x ({prompt} prompt tokens, {gen} base decode steps), then "
                        f"{n_eval} evaluator adapter(s) x ({inv} invocation tokens + {eval_steps} decode steps)",
            "base_prefill_and_generation_ms": base_ms,
            "evaluators_alora_ms": alora_ms, "evaluators_lora_ms": lora_ms,
            "evaluator_stage_speedup": lora_ms / alora_ms,
            "pipeline_alora_ms": base_ms + alora_ms, "pipeline_lora_ms": base_ms + lora_ms,
            "pipeline_speedup": (base_ms + lora_ms) / (base_ms + alora_ms),
            "evaluator_cache_bytes_alora": R2 * own_blocks * page_bytes,
            "evaluator_cache_bytes_lora": R2 * full_blocks * page_bytes,
            "device_status": status, "output_finite": finite}


def evaluator_stack_leg(ab, hp, shape, stream, local, n_eval, n_layers=32, seed=9, convs=8, prompt=4096, gen=256, inv=16,
                        eval_steps=16):
    """The evaluator workload of evaluator_leg through the whole decoder stack (n_layers layers: RMSNorm, attention
    block with adapters on q/k/v, o_proj, SwiGLU MLP; random bf16 weights): base prefill of the prompts, `gen` base
    decode steps, then `n_eval` adapters per conversation x (`inv` invocation tokens + `eval_steps` decode steps).
    aLoRA evaluators reuse the conversation's pages in every layer; LoRA evaluators prefill everything again."""
    import torch
    rng = np.random.default_rng(seed)
    ps = shape.page_size
    ctx_len = prompt + gen
    assert ctx_len % ps == 0
    R2 = convs * n_eval
    conv_blocks, own_blocks = ctx_len // ps, (inv + eval_steps + ps - 1) // ps
    full_blocks = conv_blocks + own_blocks
    num_pages = convs * conv_blocks + R2 * own_blocks + R2 * full_blocks + 3
    order = rng.permutation(num_pages).astype(np.int32)
    nxt = 0

    def take(n):
        nonlocal nxt
        out = order[nxt:nxt + n]
        nxt += n
        return out
    bt_conv = np.zeros((convs, full_blocks), np.int32)
    for c in range(convs):
        bt_conv[c, :conv_blocks] = take(conv_blocks)
    bt_alora = np.zeros((R2, full_blocks), np.int32)
    bt_lora = np.zeros((R2, full_blocks), np.int32)
    for c in range(convs):
        for n in range(n_eval):
            r = c * n_eval + n
            bt_alora[r, :conv_blocks] = bt_conv[c, :conv_blocks]
            bt_alora[r, conv_blocks:] = take(own_blocks)
            bt_lora[r] = take(full_blocks)
    ids_eval = np.tile(np.arange(n_eval, dtype=np.int32), convs)
    T_re = R2 * (ctx_len + inv)
    T_max = max(T_re, convs * prompt)
    H, I, Nq, Nkv = shape.hidden, shape.intermediate, shape.Nq, shape.Nkv
    cfg = ab.make_config(hidden=H, n_q_heads=shape.n_q_heads, n_kv_heads=shape.n_kv_heads, head_dim=shape.head_dim,
                         page_size=ps, n_layers=n_layers, intermediate=I, max_adapters=max(n_eval, 1), max_rank=32,
                         dtype=ab.DTYPE_BF16, device=local, max_tokens=T_max, max_requests=max(R2, convs))
    ctx = ab.alora_create(cfg)
    try:
        keep = []
        g = torch.Generator(device="cuda"); g.manual_seed(seed)

        def rnd(*dims, std=0.02):
            return (torch.randn(dims, generator=g, device="cuda", dtype=torch.float32) * std).to(torch.bfloat16)
        for l in range(n_layers):
            wts = [rnd(shape.N, H), rnd(H, Nq), rnd(2 * I, H), rnd(H, I),
                   (1.0 + 0.1 * torch.randn(H, generator=g, device="cuda")).to(torch.bfloat16),
                   (1.0 + 0.1 * torch.randn(H, generator=g, device="cuda")).to(torch.bfloat16)]
            keep.append(wts)
            ab.alora_set_layer_weights(ctx, l, *wts)
            for i in range(n_eval):
                ad = [rnd(32, H), rnd(Nq, 32), rnd(32, H), rnd(Nkv, 32), rnd(32, H), rnd(Nkv, 32)]
                keep.append(ad)
                ab.alora_register_adapter(ctx, i, l, 32, 1.0, *ad)
        pools = [torch.zeros((num_pages, 2, shape.n_kv_heads, ps, shape.head_dim), device="cuda", dtype=torch.bfloat16)
                 for _ in range(n_layers)]
        hid = rnd(T_max, H, std=1.0)
        out = torch.empty((T_max, H), dtype=torch.bfloat16, device="cuda")
        i32 = lambda a: hp.idev(np.ascontiguousarray(a, dtype=np.int32))  # noqa: E731
        p1 = dict(pos=i32(np.tile(np.arange(prompt), convs)), qsl=i32(np.arange(convs + 1) * prompt),
                  lens=i32(np.full(convs, prompt)), ids=i32(np.full(convs, -1)), bt=i32(bt_conv))
        p2_pos = i32(prompt + np.arange(gen)[:, None] + np.zeros((1, convs), np.int64))
        p2_len = (p2_pos + 1).contiguous()
        areq_conv = i32(np.zeros(convs))
        p3 = dict(pos=i32(np.tile(ctx_len + np.arange(inv), R2)), qsl=i32(np.arange(R2 + 1) * inv),
                  lens=i32(np.full(R2, ctx_len + inv)), ids=i32(ids_eval), areq=i32(np.full(R2, ctx_len)), bt=i32(bt_alora))
        L3 = ctx_len + inv
        p3l = dict(pos=i32(np.tile(np.arange(L3), R2)), qsl=i32(np.arange(R2 + 1) * L3), lens=i32(np.full(R2, L3)),
                   ids=i32(ids_eval), bt=i32(bt_lora))
        p4_pos = i32(L3 + np.arange(eval_steps)[:, None] + np.zeros((1, R2), np.int64))
        p4_len = (p4_pos + 1).contiguous()
        areq_open = i32(np.zeros(R2))

        def base_phases():
            ab.alora_forward_stack(ctx, ab.MODE_BASE, hid, p1["pos"], None, p1["ids"], p1["qsl"], p1["lens"], pools, p1["bt"],
                                   full_blocks, num_pages, convs * prompt, convs, out, stream)
            for i in range(gen):
                ab.alora_decode_stack(ctx, hid, p2_pos[i], areq_conv, p1["ids"], p2_len[i], pools, p1["bt"], full_blocks,
                                      num_pages, convs, out, stream)

        def alora_eval():
            ab.alora_forward_stack(ctx, ab.MODE_ALORA, hid, p3["pos"], p3["areq"], p3["ids"], p3["qsl"], p3["lens"], pools,
                                   p3["bt"], full_blocks, num_pages, R2 * inv, R2, out, stream)
            for i in range(eval_steps):
                ab.alora_decode_stack(ctx, hid, p4_pos[i], p3["areq"], p3["ids"], p4_len[i], pools, p3["bt"], full_blocks,
                                      num_pages, R2, out, stream)

        def lora_eval():
            ab.alora_forward_stack(ctx, ab.MODE_FULL_LORA, hid, p3l["pos"], None, p3l["ids"], p3l["qsl"], p3l["lens"], pools,
                                   p3l["bt"], full_blocks, num_pages, T_re, R2, out, stream)
            for i in range(eval_steps):
                ab.alora_decode_stack(ctx, hid, p4_pos[i], areq_open, p3l["ids"], p4_len[i], pools, p3l["bt"], full_blocks,
                                      num_pages, R2, out, stream)

        def once(fn, warm):
            if warm:
                fn()
            torch.cuda.synchronize()
            e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
            e0.record(stream)
            fn()
            e1.record(stream)
            torch.cuda.synchronize()
            return e0.elapsed_time(e1)
        base_ms = once(base_phases, True)
        alora_ms = once(alora_eval, True)
        lora_ms = once(lora_eval, False)
        status = ab.alora_get_status(ctx)
        finite = bool(torch.isfinite(out[:R2].float()).all())
    finally:
        ab.alora_destroy(ctx)
    return {"workload": f"{n_layers}-layer 8B-shape stack: {convs} conversations x ({prompt} prompt tokens, {gen} base decode "
                        f"steps), then {n_eval} evaluator adapter(s) x ({inv} invocation tokens + {eval_steps} decode steps)",
            "base_prefill_and_generation_ms": base_ms, "base_decode_ms_per_step_upper_bound": base_ms / gen,
            "evaluators_alora_ms": alora_ms, "evaluators_lora_ms": lora_ms,
            "evaluator_stage_speedup": lora_ms / alora_ms,
            "pipeline_alora_ms": base_ms + alora_ms, "pipeline_lora_ms": base_ms + lora_ms,
            "pipeline_speedup": (base_ms + lora_ms) / (base_ms + alora_ms),
            "device_status": status, "output_finite": finite}


def stack_leg(ab, hp, shape, stream, local, seed=4, requests=4, prefix=32768, suffix=1024, n_layers=32, name="config4",
              with_mlp_adapters=False):
    """The decoder stack at the 8B shape (RMSNorm, attention block, o_proj, SwiGLU MLP; random bf16 weights):
    `requests` requests with `prefix` cached positions and `suffix` aLoRA suffix tokens each, against the
    full-LoRA recompute of prefix + suffix through the same stack.  Config 4 is 32 layers, 4 x (32768 + 1024);
    the 8K-prefix comparison runs 4 layers of 8 x (8192 + 256) (every layer costs the same, so the ratio is that
    of the whole stack).  `with_mlp_adapters`: both arms are then timed once more with rank-32 adapters on the gate,
    up and down projections of every layer as well (gated like q/k/v)."""
    import torch
    g = torch.Generator(device="cuda"); g.manual_seed(seed)

    def rnd(*dims, std=0.02):
        return (torch.randn(dims, generator=g, device="cuda", dtype=torch.float32) * std).to(torch.bfloat16)

    R, P, S_ = requests, prefix, suffix
    T, full_T = R * S_, R * (P + S_)
    ps = shape.page_size
    blocks = (P + S_ + ps - 1) // ps
    num_pages = R * blocks + 3
    bt = np.arange(R * blocks, dtype=np.int32).reshape(R, blocks)
    cfg = ab.make_config(hidden=shape.hidden, n_q_heads=shape.n_q_heads, n_kv_heads=shape.n_kv_heads,
                         head_dim=shape.head_dim, page_size=ps, n_layers=n_layers, intermediate=shape.intermediate,
                         max_adapters=1, max_rank=32, dtype=ab.DTYPE_BF16, device=local, max_tokens=full_T, max_requests=R)
    ctx = ab.alora_create(cfg)
    keep = []
    H, I, Nq, Nkv = shape.hidden, shape.intermediate, shape.Nq, shape.Nkv
    for l in range(n_layers):
        wts = [rnd(shape.N, H), rnd(H, Nq), rnd(2 * I, H), rnd(H, I),
               (1.0 + 0.1 * torch.randn(H, generator=g, device="cuda")).to(torch.bfloat16),
               (1.0 + 0.1 * torch.randn(H, generator=g, device="cuda")).to(torch.bfloat16)]
        ad = [rnd(32, H), rnd(Nq, 32), rnd(32, H), rnd(Nkv, 32), rnd(32, H), rnd(Nkv, 32)]
        keep.append((wts, ad))
        ab.alora_set_layer_weights(ctx, l, *wts)
        ab.alora_register_adapter(ctx, 0, l, 32, 1.0, *ad)
    pools = []
    for l in range(n_layers):   # the base model's cache of every layer: N(0,1) stand-in
        pool = torch.empty((num_pages, 2, shape.n_kv_heads, ps, shape.head_dim), device="cuda", dtype=torch.bfloat16)
        for i in range(0, num_pages, 8192):
            n = min(8192, num_pages - i)
            pool[i:i + n] = torch.randn((n,) + tuple(pool.shape[1:]), generator=g, device="cuda",
                                        dtype=torch.float32).to(torch.bfloat16)
        pools.append(pool)
    ids = hp.idev(np.zeros(R, np.int32)); d_bt = hp.idev(bt)
    seq = hp.idev(np.full(R, P + S_, np.int32))
    # aLoRA side: only the suffix tokens are new
    pos_a = hp.idev(np.concatenate([np.arange(P, P + S_, dtype=np.int32)] * R))
    qsl_a = hp.idev(np.arange(R + 1, dtype=np.int32) * S_)
    areq = hp.idev(np.full(R, P, np.int32))
    hid_a = rnd(T, H, std=1.0); out_a = torch.empty_like(hid_a)
    # recompute side: every token is new, the adapter applies everywhere
    pos_f = hp.idev(np.concatenate([np.arange(P + S_, dtype=np.int32)] * R))
    qsl_f = hp.idev(np.arange(R + 1, dtype=np.int32) * (P + S_))
    hid_f = rnd(full_T, H, std=1.0); out_f = torch.empty_like(hid_f)
    fpools = [torch.zeros_like(pools[0]) for _ in range(2)]   # two private pools, alternated: results are not reused

    def alora():
        ab.alora_forward_stack(ctx, ab.MODE_ALORA, hid_a, pos_a, areq, ids, qsl_a, seq, pools, d_bt, blocks, num_pages,
                               T, R, out_a, stream)

    def recompute():
        ab.alora_forward_stack(ctx, ab.MODE_FULL_LORA, hid_f, pos_f, None, ids, qsl_f, seq,
                               [fpools[l & 1] for l in range(n_layers)], d_bt, blocks, num_pages, full_T, R, out_f, stream)

    def once(fn, n):
        fn(); torch.cuda.synchronize()
        e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
        e0.record(stream)
        for _ in range(n):
            fn()
        e1.record(stream); torch.cuda.synchronize()
        return e0.elapsed_time(e1) / n

    a_ms = once(alora, 3)
    kern = profiled(ab, ctx, alora, 1, None)
    r_ms = once(recompute, 1)
    mlp = None
    if with_mlp_adapters:
        a_hot_ms = once(alora, 3)        # the plain stack once more, in the clock state the adapted one will see
        for l in range(n_layers):
            m = [rnd(32, H), rnd(I, 32), rnd(32, H), rnd(I, 32), rnd(32, I), rnd(H, 32)]
            keep.append(m)
            ab.alora_register_mlp_adapter(ctx, 0, l, 32, 1.0, *m)
        torch.cuda.synchronize()
        am_ms = once(alora, 3)
        kern_m = profiled(ab, ctx, alora, 1, None)
        rm_ms = once(recompute, 1)
        mlp = {"alora_ms": am_ms, "alora_ms_without": a_hot_ms, "alora_overhead": am_ms / a_hot_ms - 1.0,
               "full_lora_recompute_ms": rm_ms,
               "recompute_overhead": rm_ms / r_ms - 1.0, "speedup_alora_vs_full_lora": rm_ms / am_ms,
               "per_kernel_ms_alora": {k: round(v, 3) for k, v in kern_m.items()}}
    status = ab.alora_get_status(ctx)
    finite = bool(torch.isfinite(out_a.float()).all().item())
    ab.alora_destroy(ctx)
    lin = 2.0 * (H * shape.N + Nq * H + 3 * H * I)                    # linear FLOP per token and layer
    att = lambda s_, p_: 4.0 * shape.head_dim * shape.n_q_heads * (s_ * p_ + s_ * (s_ + 1) / 2)   # noqa: E731
    flop_a = n_layers * (T * lin + R * att(S_, P))
    flop_r = n_layers * (full_T * lin + R * att(P + S_, 0))
    return {"workload": f"{name}: {n_layers}-layer 8B-shape stack, {R} requests x ({P} cached + {S_} suffix), rank 32",
            "alora_ms": a_ms, "alora_suffix_tokens_per_s": T / (a_ms / 1e3), "alora_tflops": flop_a / (a_ms / 1e3) / 1e12,
            "full_lora_recompute_ms": r_ms, "recompute_tflops": flop_r / (r_ms / 1e3) / 1e12,
            "speedup_alora_vs_full_lora": r_ms / a_ms, "flop_ratio": flop_r / flop_a,
            "prefix_plus_suffix_over_suffix": (P + S_) / S_, "per_kernel_ms_alora": {k: round(v, 3) for k, v in kern.items()},
            "with_mlp_adapters": mlp, "device_status": status, "output_finite": finite}


def main():
    ap = argparse.ArgumentParser()
    ap.add_argument("--gpus", type=int, default=1)
    ap.add_argument("--steps", type=int, default=200)
    ap.add_argument("--warmup", type=int, default=10)
    ap.add_argument("--impl", default="ours")
    ap.add_argument("--no-recompute", action="store_true", help="skip the full-LoRA recompute comparisons")
    ap.add_argument("--no-cpu-baseline", action="store_true")
    ap.add_argument("--no-extra", action="store_true", help="skip the decode and short-suffix legs")
    ap.add_argument("--legs", default="sustained,config3,decode,short,regime2,recompute8k,stack8k,mlp,evaluators,evaluators_stack,stack",
                    help="extra legs to run after the main workload (comma list of sustained, config3, decode, short, "
                         "regime2, recompute8k, stack8k, mlp, evaluators, evaluators_stack, stack)")
    ap.add_argument("--min-seconds", type=float, default=1.0,
                    help="length of the sustained pass: the headline step repeated until this much time has been timed")
    ap.add_argument("--decode-steps", type=int, default=256)
    ap.add_argument("--decode-ctx-max", type=int, default=32768)
    ap.add_argument("--short-cases", default="8x4,8x16,64x4,64x16",
                    help="the short-suffix leg's cases as requests x suffix tokens, on 4096 cached tokens each unless "
                         "'@cached' follows (64x4@16384)")
    ap.add_argument("--short-pages", default="contiguous", choices=["contiguous", "shuffled"],
                    help="physical page order of the short-suffix leg's caches")
    ap.add_argument("--requests", type=int, default=8)
    ap.add_argument("--prefix", type=int, default=4096)
    ap.add_argument("--suffix", type=int, default=256)
    ap.add_argument("--backend", default="nccl", help="process-group backend of a multi-rank run (gloo with --dry-run)")
    ap.add_argument("--dry-run", action="store_true",
                    help="exercise the multi-rank launch, barrier and max-over-ranks without touching a GPU")
    args = ap.parse_args()
    if args.impl == "reference":
        return run_reference(args)

    if "WORLD_SIZE" not in os.environ and args.gpus > 1:
        return launch_ranks(args.gpus)
    world = int(os.environ.get("WORLD_SIZE", "1"))
    rank = int(os.environ.get("RANK", "0"))
    local = int(os.environ.get("LOCAL_RANK", "0"))
    if args.dry_run:
        return dry_run(args, world, rank)

    import torch
    from paper_2504_12397_b200 import binding as ab
    from paper_2504_12397_b200 import device as hp
    from paper_2504_12397_b200.build import build_library
    build_library()

    torch.cuda.set_device(local)
    if world > 1:
        import torch.distributed as dist
        os.environ.setdefault("NCCL_DEBUG", "INFO")   # the communicator lines (transport, NVLS) go to stderr
        dist.init_process_group("nccl", device_id=torch.device("cuda", local))

    def barrier():
        if world > 1:
            dist.barrier()
        torch.cuda.synchronize()

    def max_over_ranks(x):
        return sharding.max_over_ranks(x, device="cuda")

    shape = wl.SHAPE_8B
    extra = not args.no_extra and world == 1
    legs = set(x for x in args.legs.split(",") if x) if extra else set()
    recomp = not args.no_recompute
    main_case = PrefillCase(hp, shape, args.requests, args.prefix, args.suffix, sharding.rank_seed(SEED, rank),
                            with_recompute=recomp)   # weak scaling: every rank draws its own batch of the same shape
    case_8k = PrefillCase(hp, shape, 8, 8192, 256, SEED + 1, with_recompute=True) if (recomp and "recompute8k" in legs) else None
    T, R = main_case.T, main_case.R
    max_tokens = max([T] + ([main_case.full_T] if recomp else []) + ([case_8k.full_T] if case_8k else []))
    cfg = ab.make_config(hidden=shape.hidden, n_q_heads=shape.n_q_heads, n_kv_heads=shape.n_kv_heads,
                         head_dim=shape.head_dim, page_size=shape.page_size, max_adapters=4, max_rank=32,
                         dtype=ab.DTYPE_BF16, device=local, max_tokens=max_tokens, max_requests=max(R, 64))
    ctx = ab.alora_create(cfg)
    w = main_case.w
    wq = hp.to_dev(w.wqkv, "bf16")
    ab.alora_set_layer_weights(ctx, 0, wq)
    rng_ad = np.random.default_rng(SEED + 17)
    adapters = [w.adapters[0]] + [wl.make_adapter(shape, 32, rng_ad) for _ in range(3)]
    keep = []
    for i, a in enumerate(adapters):
        mats = [hp.to_dev(getattr(a, n), "bf16") for n in ("Aq", "Bq", "Ak", "Bk", "Av", "Bv")]
        keep.append(mats)
        ab.alora_register_adapter(ctx, i, 0, a.rank, a.scale, *mats)
    a = adapters[0]
    flush = L2Flush(os.environ.get("ALORA_BENCH_FLUSH", "write+read"))
    stream = torch.cuda.current_stream()
    step = lambda: main_case.step(ab, ctx, stream)  # noqa: E731

    for _ in range(args.warmup):
        step()
    torch.cuda.synchronize()
    assert ab.alora_get_status(ctx) == 0, "device-side finding during warm-up"

    # ---- timed region: K steps, each bracketed by CUDA events, L2 flushed between steps ----------
    sampler = ClockSampler(local)
    launches0 = ab.alora_launch_count(ctx)
    barrier()
    sampler.start()
    step_ms = timed(step, args.steps, stream, flush)
    barrier()
    clocks = sampler.stop()            # the clocks of the timed region itself
    sampler_rest = ClockSampler(local)
    sampler_rest.start()               # the other legs (end to end, recompute, decode, stack) are sampled apart
    launches = ab.alora_launch_count(ctx) - launches0
    step_ms = max_over_ranks(step_ms)
    value = sharding.aggregate_throughput(T, step_ms / 1e3, world)

    # per-kernel event times, right after the headline pass (same clocks and temperature)
    kern = profiled(ab, ctx, step, min(args.steps, 100), flush)

    # ---- end to end through the C ABI with host buffers: H2D of the step's inputs, D2H of the result ----
    d = main_case.d
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
        ab.alora_prefill_layer(ctx, 0, d_hidden2, d_ints2[0], d_ints2[1], d_ints2[2], d_ints2[3], d_ints2[4],
                               main_case.pool, d_ints2[5], d.max_blocks, main_case.b.num_pages, T, R, main_case.out,
                               stream)
        h_out.copy_(main_case.out, non_blocking=True)

    for _ in range(3):
        e2e_step()
    barrier()
    e2e_serial_ms = max_over_ranks(timed(e2e_step, args.steps, stream, flush))

    # The same steps as a pipeline, the way a server would run them: inputs and outputs double-buffered, the H2D
    # copy of step i+1 and the D2H copy of step i-1 on streams of their own beside step i's kernels.  Every step
    # still copies its own inputs in and its own result out inside the timed region.
    s_in, s_out = torch.cuda.Stream(), torch.cuda.Stream()
    # the six small integer arrays travel as one pinned buffer (each padded to 16 bytes) and one copy
    offs, tot = [], 0
    for t in h_ints:
        offs.append(tot)
        tot += (t.numel() + 3) // 4 * 4
    h_pack = torch.zeros(tot, dtype=torch.int32).pin_memory()
    for o, t in zip(offs, h_ints):
        h_pack[o:o + t.numel()] = t.reshape(-1)
    bufs = []
    for _ in range(2):
        d_pack = torch.empty(tot, dtype=torch.int32, device=d.hidden.device)
        views = [d_pack[o:o + t.numel()].view(t.shape) for o, t in zip(offs, h_ints)]
        bufs.append(dict(hidden=torch.empty_like(d.hidden), pack=d_pack, ints=views,
                         out=torch.empty_like(main_case.out),
                         h_out=torch.empty((T, shape.Nq), dtype=torch.bfloat16).pin_memory(),
                         in_ev=torch.cuda.Event(), comp_ev=torch.cuda.Event(), out_ev=torch.cuda.Event(), used=False))

    def e2e_pipeline(n):
        for i in range(n):
            bf = bufs[i % 2]
            if bf["used"]:
                s_in.wait_event(bf["comp_ev"])            # the step that last read these inputs is done
            with torch.cuda.stream(s_in):
                bf["hidden"].copy_(h_hidden, non_blocking=True)
                bf["pack"].copy_(h_pack, non_blocking=True)
                bf["in_ev"].record(s_in)
            stream.wait_event(bf["in_ev"])
            if bf["used"]:
                stream.wait_event(bf["out_ev"])           # the result last written here has been read back
            if flush is not None:
                flush.zero_()
            ab.alora_prefill_layer(ctx, 0, bf["hidden"], bf["ints"][0], bf["ints"][1], bf["ints"][2], bf["ints"][3],
                                   bf["ints"][4], main_case.pool, bf["ints"][5], d.max_blocks, main_case.b.num_pages,
                                   T, R, bf["out"], stream)
            bf["comp_ev"].record(stream)
            s_out.wait_event(bf["comp_ev"])
            with torch.cuda.stream(s_out):
                bf["h_out"].copy_(bf["out"], non_blocking=True)
                bf["out_ev"].record(s_out)
            bf["used"] = True

    e2e_pipeline(4)
    torch.cuda.synchronize()
    barrier()
    p0 = torch.cuda.Event(enable_timing=True); p1 = torch.cuda.Event(enable_timing=True)
    p0.record(stream)
    s_in.wait_event(p0); s_out.wait_event(p0)
    e2e_pipeline(args.steps)
    stream.wait_stream(s_out); stream.wait_stream(s_in)
    p1.record(stream)
    torch.cuda.synchronize()
    e2e_ms = max_over_ranks(p0.elapsed_time(p1) / args.steps)
    assert torch.equal(bufs[0]["h_out"], h_out) and torch.equal(bufs[1]["h_out"], h_out)
    h2d = h_hidden.numel() * 2 + h_pack.numel() * 4
    d2h = h_out.numel() * 2

    # ---- roofline of the dominant kernel: per-kernel event times from a separate profiled pass -----
    peaks = measured_peaks()
    proj_flops, attn_flops, attn_bytes = main_case.flops_bytes(shape, a.rank)
    proj_ms = kern.get("project_qkv", 0.0) + kern.get("shrink", 0.0)
    attn_ms = attention_ms(kern)
    dominant = "attention" if attn_ms >= proj_ms else "project_qkv"
    dom_ms = attn_ms if dominant == "attention" else proj_ms
    dom_flops = attn_flops if dominant == "attention" else proj_flops
    achieved = dom_flops / (dom_ms / 1e3) / 1e12 if dom_ms > 0 else 0.0
    peak = peaks["bf16_tflops"]
    roofline = {"bound": "tensor", "kernel": dominant, "achieved": achieved, "peak": peak, "unit": "TFLOP/s",
                "frac": achieved / peak, "frac_of_nominal": achieved / NOMINAL_BF16_TFLOPS,
                "traffic": (NCU_TRAFFIC_BYTES.get(dominant) if (args.requests, args.prefix, args.suffix) == (8, 4096, 256) else None),
                "traffic_unit": "bytes per launch (ncu dram read + write)",
                "algorithmic_bytes": attn_bytes if dominant == "attention" else 2.0 * (T * shape.hidden + shape.N * shape.hidden + T * shape.N),
                "peak_source": peaks["source"] + " (burst bf16 GEMM)",
                "ms_per_launch": dom_ms,
                "per_kernel_ms": {k: round(v, 4) for k, v in kern.items()},
                "projection": {"tflops": proj_flops / (proj_ms / 1e3) / 1e12 if proj_ms else None,
                               "frac_of_tensor_peak": proj_flops / (proj_ms / 1e3) / 1e12 / peak if proj_ms else None},
                "attention": {"tflops": attn_flops / (attn_ms / 1e3) / 1e12 if attn_ms else None,
                              "hbm_gbs": attn_bytes / (attn_ms / 1e3) / 1e9 if attn_ms else None,
                              "frac_of_hbm_peak": attn_bytes / (attn_ms / 1e3) / 1e9 / peaks["hbm_gbs"] if attn_ms else None,
                              "frac_of_tensor_peak": attn_flops / (attn_ms / 1e3) / 1e12 / peak if attn_ms else None}}

    # ---- the comparison path: full-LoRA recompute of prefix + suffix on the same box -------------
    def recompute_of(case, alora_ms):
        rs = lambda: case.recompute_step(ab, ctx, stream)  # noqa: E731
        rs(); rs()
        rms = timed(rs, max(1, min(args.steps, 10)), stream, flush)
        return {"prefix": int(case.b.prefix_lens[0]), "suffix": int(case.T // case.R), "requests": case.R,
                "alora_ms_per_step": alora_ms, "full_lora_ms_per_step": rms, "tokens": case.full_T,
                "speedup_alora_vs_full_lora": rms / alora_ms,
                "prefix_plus_suffix_over_suffix": float(case.full_T) / case.T}

    recompute = recompute_of(main_case, step_ms) if recomp else None
    recompute_8k = None
    if case_8k is not None:
        s8 = lambda: case_8k.step(ab, ctx, stream)  # noqa: E731
        for _ in range(5):
            s8()
        recompute_8k = recompute_of(case_8k, timed(s8, 50, stream, flush))

    decode = short = sustained = None
    if "sustained" in legs:
        sustained = sustained_leg(step, stream, flush, local, args.min_seconds, proj_flops + attn_flops, peaks)
    if "decode" in legs:
        decode = decode_leg(ab, hp, ctx, shape, stream, flush, peaks, steps=args.decode_steps,
                            ctx_max=args.decode_ctx_max)
    if "short" in legs:
        short = [short_suffix_leg(ab, hp, ctx, shape, stream, flush, peaks, r_, p_, s_, shuffle_pages=args.short_pages == "shuffled")
                 for r_, s_, p_ in [parse_short_case(c) for c in args.short_cases.split(",") if c]]
    regime2 = None
    if "regime2" in legs:
        # the headline shape with the activation offset 192 tokens into the 256 new ones: an uncached tail of the
        # context goes through the base weights, the 64-token invocation through the adapter, in ONE call
        regime2 = short_suffix_leg(ab, hp, ctx, shape, stream, flush, peaks, args.requests, args.prefix, args.suffix,
                                   seed=12, activation_shift=(3 * args.suffix) // 4)
        regime2["ms_per_step_activation_at_chunk_start"] = step_ms
    status = ab.alora_get_status(ctx)
    ab.alora_destroy(ctx)
    want_cpu = rank == 0 and world == 1 and not args.no_cpu_baseline
    pool_np = main_case.pool.to(torch.float32).cpu().numpy() if want_cpu else None
    stack = evaluators = config3 = stack_8k = evaluators_stack = mlp_adapters = None
    if legs & {"evaluators", "evaluators_stack", "stack", "stack8k", "config3", "mlp"}:
        del main_case.pool
        torch.cuda.empty_cache()
    if "config3" in legs:
        config3 = config3_leg(ab, hp, stream, local, flush, peaks)
        torch.cuda.empty_cache()
    if "stack8k" in legs:
        stack_8k = stack_leg(ab, hp, shape, stream, local, seed=8, requests=8, prefix=8192, suffix=256, n_layers=4,
                             name="8K-prefix comparison through whole layers")
        torch.cuda.empty_cache()
    if "mlp" in legs:
        mlp_adapters = stack_leg(ab, hp, shape, stream, local, seed=9, requests=8, prefix=8192, suffix=256, n_layers=2,
                                 name="adapters on the MLP block as well", with_mlp_adapters=True)
        torch.cuda.empty_cache()
    if "evaluators" in legs:
        evaluators = [evaluator_leg(ab, hp, shape, stream, local, n) for n in (1, 5)]
        torch.cuda.empty_cache()
    if "evaluators_stack" in legs:
        evaluators_stack = []
        for n in (1, 5):
            evaluators_stack.append(evaluator_stack_leg(ab, hp, shape, stream, local, n))
            torch.cuda.empty_cache()
    if "stack" in legs:
        stack = stack_leg(ab, hp, shape, stream, local)
    clocks_rest = sampler_rest.stop()

    cpu = None
    if want_cpu:
        S_ = (main_case.b.seq_lens - main_case.b.prefix_lens)
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
                       "tokens_per_step_per_gpu": T, "l2": "flushed between steps (256 MB memset, then a 256 MB read sweep that leaves clean lines; outside the timed events)",
                       "timing": "mean of per-step CUDA-event durations on the launching stream, max over ranks"},
            "clocks": clocks, "clocks_other_legs": clocks_rest, "e2e": {"value": world * T / (e2e_ms / 1e3), "unit": UNIT, "h2d_bytes_per_step": h2d,
                                      "d2h_bytes_per_step": d2h, "ms_per_step": e2e_ms, "serial_ms_per_step": e2e_serial_ms,
                                      "how": "K steps as a 3-stream pipeline (H2D, kernels, D2H; double-buffered), total time / K; serial = one step at a time"},
            "gpu_launches": int(launches), "roofline": roofline, "cpu_baseline": cpu,
            "full_lora_recompute": recompute, "full_lora_recompute_8k_prefix": recompute_8k,
            "sustained": sustained, "config3": config3, "decode": decode, "short_suffix": short,
            "evaluator_pipeline": evaluators, "evaluator_pipeline_32_layers": evaluators_stack,
            "chunk_straddling_prefill": regime2, "stack_8k_prefix": stack_8k, "mlp_adapters": mlp_adapters, "stack": stack, "device_status": status,
            # the figures of merit in one place, last, so that a truncated copy of this line still carries them
            "fractions": fractions(peaks, roofline, sustained, config3, decode, short, recompute_8k, stack_8k, stack, evaluators,
                                   evaluators_stack, mlp_adapters, regime2),
        }))
    if world > 1:
        dist.destroy_process_group()


if __name__ == "__main__":
    main()

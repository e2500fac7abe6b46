"""Error behaviour of the boundary on a device: what the host checks reject before any launch, what the device
reports through the status word, and that the context stays usable afterwards."""
import numpy as np
import pytest

from paper_2504_12397_b200 import binding as ab
from paper_2504_12397_b200 import workloads as wl

import helpers as hp

pytestmark = pytest.mark.gpu

SHAPE = wl.LayerShape(hidden=256, n_q_heads=4, n_kv_heads=2, head_dim=64, page_size=16, dtype="bf16")


def _layer(rng, shape=SHAPE, n_adapters=2, registered=(0,)):
    w = wl.make_wqkv(shape, rng)
    ads = [wl.make_adapter(shape, 8, rng, scale=4.0) for _ in registered]
    g = hp.GpuLayers(shape, [dict(wqkv=w)], [ads], 256, 8, n_adapters=n_adapters)
    return w, ads, g


def test_tokens_without_requests_are_rejected_before_any_launch():
    import torch
    rng = np.random.default_rng(1)
    w, ads, g = _layer(rng)
    try:
        z = torch.zeros(16, dtype=torch.int32, device="cuda")
        x = torch.zeros((4, SHAPE.hidden), dtype=torch.bfloat16, device="cuda")
        out = torch.zeros((4, SHAPE.N), dtype=torch.bfloat16, device="cuda")
        n0 = ab.alora_launch_count(g.ctx)
        with pytest.raises(ab.AloraError) as e:
            ab.alora_project_qkv(g.ctx, 0, ab.MODE_ALORA, x, z, z, z, z, z, 4, 0, out)
        assert e.value.status == 1   # ALORA_ERR_INVALID_ARG
        assert ab.alora_launch_count(g.ctx) == n0
    finally:
        g.close()


def test_open_gate_on_an_unregistered_adapter_is_reported(oracle64):
    """Adapter id 1 is inside [0, max_adapters) but was never registered on the layer: the rows that would apply it
    get the base projection and the status word reads ALORA_ERR_NO_WEIGHTS; the next call is clean."""
    rng = np.random.default_rng(2)
    w, ads, g = _layer(rng, n_adapters=2, registered=(0,))
    try:
        b = wl.make_batch(SHAPE, [5, 9], [20, 12], [0, 1], rng, activation_offsets=[5, 12])
        d = hp.DevBatch(b, "bf16")
        qkv = g.empty(b.T, SHAPE.N)
        ab.alora_project_qkv(g.ctx, 0, ab.MODE_ALORA, d.hidden, d.positions, d.a_req, d.ids, d.qsl, d.seq_lens,
                             b.T, b.R, qkv)
        assert g.status() == 4   # ALORA_ERR_NO_WEIGHTS
        ids_ok = np.array([0, -1], np.int32)
        want, _ = oracle64.project_qkv(b.hidden, w, SHAPE.Nq, SHAPE.Nkv, b.positions, b.query_start_loc,
                                       b.activation_offsets, ids_ok, hp.oracle_adapters(ads))
        hp.assert_close(hp.to_host(qkv), want, 2e-2, "rows of the unregistered adapter fall back to the base projection")
        ab.alora_project_qkv(g.ctx, 0, ab.MODE_ALORA, d.hidden, d.positions, d.a_req, hp.idev(ids_ok), d.qsl, d.seq_lens,
                             b.T, b.R, qkv)
        assert g.status() == 0
    finally:
        g.close()


def test_stack_step_with_an_unsupported_shape_stops_the_call():
    """An MLP width that is not a multiple of 8 cannot be served by the tensor-core GEMM: the stack call must
    return ALORA_ERR_UNSUPPORTED instead of skipping the step and reporting success."""
    import torch
    shape = wl.LayerShape(hidden=256, n_q_heads=4, n_kv_heads=2, head_dim=64, page_size=16, dtype="bf16",
                          intermediate=20)
    rng = np.random.default_rng(3)
    lw = wl.make_stack_weights(shape, rng)
    g = hp.GpuLayers(shape, [lw], [[]], 64, 2)
    try:
        b = wl.make_batch(shape, [0], [24], [-1], rng)
        d = hp.DevBatch(b, "bf16")
        pool = g.new_pool(b.num_pages)
        hout = g.empty(b.T, shape.hidden)
        with pytest.raises(ab.AloraError) as e:
            ab.alora_forward_stack(g.ctx, ab.MODE_BASE, d.hidden, d.positions, d.a_req, d.ids, d.qsl, d.seq_lens, [pool],
                                   d.bt, d.max_blocks, b.num_pages, b.T, b.R, hout)
        assert e.value.status == 2   # ALORA_ERR_UNSUPPORTED
        torch.cuda.synchronize()
        assert g.status() == 0
    finally:
        g.close()


def test_bounded_wait_gives_up_and_the_context_stays_usable(oracle64):
    """One block waits, with a limit of about a millisecond, on a barrier that nobody arrives at (the library's own
    bounded wait, as every tensor-core kernel uses it).  The wait must run out, the kernel must return normally, the
    status word must read ALORA_ERR_TIMEOUT, and a layer call right after must be clean and correct."""
    import time
    import torch
    rng = np.random.default_rng(4)
    w, ads, g = _layer(rng)
    try:
        t0 = time.perf_counter()
        ab.alora_selftest_wait_timeout(g.ctx, 2_000_000)     # about 1 ms at 2 GHz
        torch.cuda.synchronize()
        assert time.perf_counter() - t0 < 5.0
        assert g.status() == 8   # ALORA_ERR_TIMEOUT
        assert g.status() == 0   # reading the status clears it
        with pytest.raises(ab.AloraError):
            ab.alora_selftest_wait_timeout(g.ctx, 10**12)    # limits that would stall the GPU are refused
        b = wl.make_batch(SHAPE, [40, 0], [30, 17], [0, -1], rng, with_prefix_hidden=True)
        pool = g.new_pool(b.num_pages)
        pb = hp.prefix_only_batch(SHAPE, b)
        dpb = hp.DevBatch(pb, "bf16")
        ab.alora_full_lora_prefill_layer(g.ctx, 0, dpb.hidden, dpb.positions, dpb.ids, dpb.qsl, dpb.seq_lens, pool,
                                         dpb.bt, dpb.max_blocks, b.num_pages, dpb.T, dpb.R, g.empty(pb.T, SHAPE.Nq))
        d = hp.DevBatch(b, "bf16")
        out = g.empty(b.T, SHAPE.Nq)
        ab.alora_prefill_layer(g.ctx, 0, d.hidden, d.positions, d.a_req, d.ids, d.qsl, d.seq_lens, pool, d.bt,
                               d.max_blocks, b.num_pages, b.T, b.R, out)
        assert g.status() == 0
        Ks, Vs = hp.oracle_base_prefix(oracle64, SHAPE, w, b)
        want = hp.oracle_block(oracle64, SHAPE, w, ads, b, Ks, Vs)
        hp.assert_close(hp.to_host(out), want["out"], 2e-2, "layer call after an expired wait", block=SHAPE.head_dim)
    finally:
        g.close()

"""GPU parity: every step of the hot path through the C ABI against the CPU oracle, element by
element, on seeded inputs that span several tiles and ragged tails.  Integer outputs and gated-off
rows must match exactly; floating-point outputs within the tolerance of tests/helpers.tol."""
import numpy as np
import pytest

from paper_2504_12397_b200 import binding as ab
from paper_2504_12397_b200 import workloads as wl

import helpers as hp

pytestmark = pytest.mark.gpu

# reduced 8B-like bf16 shape: same head_dim / group size as the 8B layer, smaller widths
MID = wl.LayerShape(hidden=1024, n_q_heads=8, n_kv_heads=2, head_dim=128, page_size=16, dtype="bf16",
                    intermediate=1536)


def _mid_workload(seed=11, a_req_shift=True):
    """Ragged multi-adapter batch: 6 requests over adapters of ranks 8/16/32/64 and the base model,
    prefixes 0..700, suffixes 1..300, some activation offsets inside the new chunk, shuffled pages."""
    rng = np.random.default_rng(seed)
    w = wl.make_wqkv(MID, rng)
    ads = [wl.make_adapter(MID, r, rng, scale=s) for r, s in ((8, 1.0), (16, 2.0), (32, 1.0), (64, 0.5))]
    for a in ads:  # lift the delta well above bf16 rounding noise so a wrong or missing delta is visible
        for n in ("Bq", "Bk", "Bv"):
            setattr(a, n, wl.bf16_round(getattr(a, n) * 8))
    P = [0, 37, 700, 129, 256, 300]
    S = [150, 300, 1, 131, 128, 17]
    ids = [2, 0, 3, -1, 1, 2]
    a_req = [0, 37 + 130, 700, 0, 256 + 5, 300]
    b = wl.make_batch(MID, P, S, ids, rng, activation_offsets=a_req if a_req_shift else None,
                      shuffle_pages=True, with_prefix_hidden=True)
    return w, ads, b


def _run_base_prefill(g: hp.GpuLayers, shape, b, pool, layer=0):
    pb = hp.prefix_only_batch(shape, b)
    if pb.T == 0:
        return
    d = hp.DevBatch(pb, shape.dtype)
    out = g.empty(pb.T, shape.Nq)
    ab.alora_full_lora_prefill_layer(g.ctx, layer, d.hidden, d.positions, d.ids, d.qsl, d.seq_lens, pool, d.bt,
                                     d.max_blocks, b.num_pages, d.T, d.R, out)


def _gather_pool(orc, shape, pool_np, b):
    return [orc.paged_gather(pool_np, b.block_tables[r], int(b.seq_lens[r]), shape.n_kv_heads, shape.page_size,
                             shape.head_dim) for r in range(b.R)]


@pytest.mark.parametrize("mode", [ab.MODE_ALORA, ab.MODE_FULL_LORA, ab.MODE_BASE])
def test_batch_metadata_is_exact(oracle64, mode):
    w, ads, b = _mid_workload()
    g = hp.GpuLayers(MID, [dict(wqkv=w)], [ads], b.T, b.R)
    try:
        import torch
        d = hp.DevBatch(b, MID.dtype)
        tok = torch.full((b.T,), -9, dtype=torch.int32, device="cuda")
        row = torch.full((b.T,), -9, dtype=torch.int32, device="cuda")
        slot = torch.full((b.T,), -9, dtype=torch.int32, device="cuda")
        ab.alora_batch_metadata(g.ctx, mode, d.positions, d.a_req, d.ids, d.qsl, d.seq_lens, d.bt, d.max_blocks,
                                b.num_pages, d.T, d.R, tok, row, slot)
        assert g.status() == 0
        want_slot = oracle64.slot_mapping(b.positions, b.query_start_loc, b.block_tables, MID.page_size)
        np.testing.assert_array_equal(slot.cpu().numpy().astype(np.int64), want_slot)
        # the oracle's gate, read off a projection with throw-away 4-wide weights
        from oracle import Adapter
        z14, z11 = np.zeros((1, 4)), np.zeros((1, 1))
        _, gate = oracle64.project_qkv(np.zeros((b.T, 4)), np.zeros((3, 4), np.float32), 1, 1, b.positions,
                                       b.query_start_loc, b.activation_offsets, b.adapter_ids,
                                       [Adapter(1, 1.0, z14, z11, z14, z11, z14, z11) for _ in ads],
                                       force_all=(mode == ab.MODE_FULL_LORA))
        req = np.repeat(np.arange(b.R), np.diff(b.query_start_loc))
        np.testing.assert_array_equal(tok.cpu().numpy(), req)
        want_row = np.where(gate.astype(bool), b.adapter_ids[req], -1)
        if mode == ab.MODE_BASE:
            want_row[:] = -1
        np.testing.assert_array_equal(row.cpu().numpy(), want_row)
    finally:
        g.close()


def test_config1_tiny_fp32_layer(oracle64):
    """Config 1 end to end: base prefill builds the cache, the aLoRA suffix prefill reuses it."""
    w = wl.config1()
    shape, b = w.shape, w.batch
    g = hp.GpuLayers(shape, [dict(wqkv=w.wqkv)], [w.adapters], 128, 4)
    try:
        pool = g.new_pool(b.num_pages)
        _run_base_prefill(g, shape, b, pool)
        d = hp.DevBatch(b, shape.dtype)
        out = g.empty(b.T, shape.Nq)
        ab.alora_prefill_layer(g.ctx, 0, d.hidden, d.positions, d.a_req, d.ids, d.qsl, d.seq_lens, pool, d.bt,
                               d.max_blocks, b.num_pages, d.T, d.R, out)
        qkv = g.empty(b.T, shape.N)
        ab.alora_project_qkv(g.ctx, 0, ab.MODE_ALORA, d.hidden, d.positions, d.a_req, d.ids, d.qsl, d.seq_lens,
                             d.T, d.R, qkv)
        assert g.status() == 0
        Ks, Vs = hp.oracle_base_prefix(oracle64, shape, w.wqkv, b)
        want = hp.oracle_block(oracle64, shape, w.wqkv, w.adapters, b, Ks, Vs)
        assert want["gate"].all()
        hp.assert_close(hp.to_host(qkv), want["qkv"], 1e-5, "")
        hp.assert_close(hp.to_host(out), want["out"], 1e-5, "")
        got = _gather_pool(oracle64, shape, hp.to_host(pool), b)
        for r in range(b.R):
            hp.assert_close(got[r][0], want["K"][r], 1e-5, "")
            hp.assert_close(got[r][1], want["V"][r], 1e-5, "")
        # the delta matters in this configuration: the base model's answer is outside the tolerance
        b0 = wl.Batch(**{**b.__dict__, "adapter_ids": np.array([-1], np.int32)})
        base = hp.oracle_block(oracle64, shape, w.wqkv, w.adapters, b0, Ks, Vs)
        assert hp.rel_err(base["qkv"], want["qkv"]) > 1e-3
    finally:
        g.close()


def test_ragged_multi_adapter_layer_bf16(oracle64):
    """Projection, append and attention on a ragged multi-adapter batch with mid-chunk activation."""
    w, ads, b = _mid_workload()
    g = hp.GpuLayers(MID, [dict(wqkv=w)], [ads], 2048, 8)
    try:
        pool = g.new_pool(b.num_pages)
        _run_base_prefill(g, MID, b, pool)
        pool_before = hp.to_host(pool).copy()
        d = hp.DevBatch(b, MID.dtype)
        out = g.empty(b.T, MID.Nq)
        ab.alora_prefill_layer(g.ctx, 0, d.hidden, d.positions, d.a_req, d.ids, d.qsl, d.seq_lens, pool, d.bt,
                               d.max_blocks, b.num_pages, d.T, d.R, out)
        qkv = g.empty(b.T, MID.N)
        ab.alora_project_qkv(g.ctx, 0, ab.MODE_ALORA, d.hidden, d.positions, d.a_req, d.ids, d.qsl, d.seq_lens,
                             d.T, d.R, qkv)
        base = g.empty(b.T, MID.N)
        ab.alora_project_qkv(g.ctx, 0, ab.MODE_BASE, d.hidden, d.positions, d.a_req, d.ids, d.qsl, d.seq_lens,
                             d.T, d.R, base)
        assert g.status() == 0
        Ks, Vs = hp.oracle_base_prefix(oracle64, MID, w, b)
        want = hp.oracle_block(oracle64, MID, w, ads, b, Ks, Vs)
        qkv_h, base_h, out_h = hp.to_host(qkv), hp.to_host(base), hp.to_host(out)
        hp.assert_close(qkv_h, want["qkv"], 2e-2, "")
        hp.assert_close(out_h, want["out"], 2e-2, "")
        # rows whose gate is closed: bit-identical to the GPU base-only projection (Prop. 1)
        off = want["gate"] == 0
        assert off.sum() > 100 and (~off).sum() > 100
        assert np.array_equal(qkv_h[off].view(np.uint32), base_h[off].view(np.uint32))
        # rows whose gate is open really carry the delta
        assert hp.rel_err(base_h[~off], want["qkv"][~off]) > 5e-2
        # KV append: new rows equal the projection's k/v parts bit for bit, every other byte untouched
        pool_after = hp.to_host(pool)
        slots = oracle64.slot_mapping(b.positions, b.query_start_loc, b.block_tables, MID.page_size)
        expect = pool_before.copy()
        oracle64.paged_append(expect, qkv_h[:, MID.Nq:MID.Nq + MID.Nkv], qkv_h[:, MID.Nq + MID.Nkv:], slots,
                              MID.n_kv_heads, MID.page_size, MID.head_dim)
        assert np.array_equal(pool_after.view(np.uint32), expect.view(np.uint32))
        # prefix rows in the cache are the base model's (made by the base prefill) within tolerance
        got = _gather_pool(oracle64, MID, pool_after, b)
        for r in range(b.R):
            hp.assert_close(got[r][0], want["K"][r], 2e-2, "")
            hp.assert_close(got[r][1], want["V"][r], 2e-2, "")
    finally:
        g.close()


def test_sub_steps_compose_to_the_layer_call(oracle64):
    """alora_project_qkv + alora_kv_append + alora_attend == alora_prefill_layer, bit for bit."""
    w, ads, b = _mid_workload(seed=12)
    g = hp.GpuLayers(MID, [dict(wqkv=w)], [ads], 2048, 8)
    try:
        rng = np.random.default_rng(0)
        fill = wl.random_kv_pool(MID, b.num_pages, rng)
        d = hp.DevBatch(b, MID.dtype)
        pool1, pool2 = g.new_pool(b.num_pages, fill), g.new_pool(b.num_pages, fill)
        out1, out2 = g.empty(b.T, MID.Nq), g.empty(b.T, MID.Nq)
        ab.alora_prefill_layer(g.ctx, 0, d.hidden, d.positions, d.a_req, d.ids, d.qsl, d.seq_lens, pool1, d.bt,
                               d.max_blocks, b.num_pages, d.T, d.R, out1)
        qkv = g.empty(b.T, MID.N)
        ab.alora_project_qkv(g.ctx, 0, ab.MODE_ALORA, d.hidden, d.positions, d.a_req, d.ids, d.qsl, d.seq_lens,
                             d.T, d.R, qkv)
        ab.alora_kv_append(g.ctx, qkv, d.positions, d.qsl, d.seq_lens, d.bt, d.max_blocks, b.num_pages, d.T, d.R, pool2)
        ab.alora_attend(g.ctx, qkv, d.positions, d.qsl, d.seq_lens, pool2, d.bt, d.max_blocks, b.num_pages, d.T, d.R, out2)
        assert g.status() == 0
        assert np.array_equal(hp.to_host(pool1).view(np.uint32), hp.to_host(pool2).view(np.uint32))
        assert np.array_equal(hp.to_host(out1).view(np.uint32), hp.to_host(out2).view(np.uint32))
        # attention alone against the oracle on a random (non-projected) cache
        pool_h, qkv_h = hp.to_host(pool2), hp.to_host(qkv)
        kv = _gather_pool(oracle64, MID, pool_h, b)
        kvl = np.concatenate([[0], np.cumsum(b.seq_lens)])
        want, _ = oracle64.attention(qkv_h[:, :MID.Nq], np.concatenate([k for k, _ in kv]),
                                     np.concatenate([v for _, v in kv]), kvl, b.positions, b.query_start_loc,
                                     MID.n_q_heads, MID.n_kv_heads, MID.head_dim)
        hp.assert_close(hp.to_host(out2), want, 2e-2, "")
    finally:
        g.close()


def _boosted_adapters(shape, rng, spec):
    ads = [wl.make_adapter(shape, r, rng, scale=s) for r, s in spec]
    for a in ads:  # lift the delta well above bf16 rounding noise so a wrong or missing delta is visible
        for n in ("Bq", "Bk", "Bv"):
            setattr(a, n, wl.bf16_round(getattr(a, n) * 8))
    return ads


def _check_projection(oracle64, shape, w, ads, b, n_off_expected=None):
    g = hp.GpuLayers(shape, [dict(wqkv=w)], [ads], b.T, b.R)
    try:
        d = hp.DevBatch(b, shape.dtype)
        qkv, base, again = g.empty(b.T, shape.N), g.empty(b.T, shape.N), g.empty(b.T, shape.N)
        for mode, dst in ((ab.MODE_ALORA, qkv), (ab.MODE_BASE, base), (ab.MODE_ALORA, again)):
            ab.alora_project_qkv(g.ctx, 0, mode, d.hidden, d.positions, d.a_req, d.ids, d.qsl, d.seq_lens, d.T, d.R, dst)
        assert g.status() == 0
        want, gate = oracle64.project_qkv(b.hidden, w, shape.Nq, shape.Nkv, b.positions, b.query_start_loc,
                                          b.activation_offsets, b.adapter_ids, hp.oracle_adapters(ads))
        qkv_h, base_h = hp.to_host(qkv), hp.to_host(base)
        hp.assert_close(qkv_h, want, 2e-2, "")
        off = gate == 0
        if n_off_expected is not None:
            assert off.sum() == n_off_expected
        assert off.sum() > 0 and (~off).sum() > 0
        # rows whose gate is closed: bit-identical to the GPU base-only projection (Prop. 1)
        assert np.array_equal(qkv_h[off].view(np.uint32), base_h[off].view(np.uint32))
        # rows whose gate is open really carry the delta
        assert hp.rel_err(base_h[~off], want[~off]) > 5e-2
        # run-to-run determinism
        assert np.array_equal(hp.to_host(again).view(np.uint32), qkv_h.view(np.uint32))
    finally:
        g.close()


def test_projection_row_tile_route_with_fused_shrink(oracle64):
    """Long requests at 256-wide column tiles: row tiles segmented by (adapter, gate), the rank-r shrink
    running as leading work items of the projection kernel."""
    rng = np.random.default_rng(43)
    w = wl.make_wqkv(MID, rng)
    ads = _boosted_adapters(MID, rng, ((8, 1.0), (64, 0.5), (32, 2.0)))
    b = wl.make_batch(MID, [0, 300, 20, 5], [500, 390, 130, 260], [1, 0, -1, 2], rng, activation_offsets=[130, 300, 0, 200])
    _check_projection(oracle64, MID, w, ads, b, n_off_expected=130 + 130 + 195)


def test_projection_of_many_rows_two_row_tiles_per_block(oracle64):
    """Many rows (and enough tiles to fill the blocks): the projection takes 256 x 192 tiles (two row tiles per block).  With this shape's
    blocks of 1024 / 256 / 256 columns the 192-wide column tiles straddle the q | k and k | v boundaries, some
    row tiles are partial, one request runs on the base model and gates open in the middle of requests."""
    rng = np.random.default_rng(45)
    w = wl.make_wqkv(MID, rng)
    ads = _boosted_adapters(MID, rng, ((8, 1.0), (64, 0.5), (32, 2.0)))
    b = wl.make_batch(MID, [0, 300, 20, 5, 0], [1500, 1390, 530, 760, 428], [1, 0, -1, 2, 0], rng,
                      activation_offsets=[130, 300, 0, 200, 77])
    assert b.T == 4608   # 18 row pairs x 8 column tiles = 144 items for 148 blocks: the launcher prefers this tile shape
    _check_projection(oracle64, MID, w, ads, b, n_off_expected=130 + 530 + 195 + 77)


def test_projection_row_wise_route_many_short_requests(oracle64):
    """Many requests of 1..9 new tokens over different adapters and the base model, some gated off: the row
    tiles would hold a few rows each, so the batch takes the row-wise delta route."""
    rng = np.random.default_rng(44)
    w = wl.make_wqkv(MID, rng)
    ads = _boosted_adapters(MID, rng, ((8, 1.0), (64, 0.5), (32, 2.0), (16, 1.0)))
    R = 40
    S = [1 + (i * 7) % 9 for i in range(R)]
    P = [(i * 37) % 200 for i in range(R)]
    ids = [(i % 5) - 1 for i in range(R)]
    a_req = [P[i] + (3 if i % 4 == 0 else 0) for i in range(R)]   # every fourth request opens its gate 3 tokens late
    b = wl.make_batch(MID, P, S, ids, rng, activation_offsets=a_req)
    _check_projection(oracle64, MID, w, ads, b)


@pytest.mark.parametrize("T", [1, 24, 33, 64, 65, 128])
def test_projection_few_row_route_mixed_adapters(oracle64, T):
    """Batches of at most 128 rows (decode steps): the weight-streaming route, K split over the SMs, the shrink of
    every present adapter riding along, slice partials added in fixed order.  One token per request, requests mixing
    the base model and four adapters of different ranks in no particular order, every third adapter request with
    its gate still closed.  Checked: oracle, closed-gate rows bit-identical to the base-only call, determinism."""
    rng = np.random.default_rng(100 + T)
    w = wl.make_wqkv(MID, rng)
    ads = _boosted_adapters(MID, rng, ((8, 1.0), (64, 0.5), (32, 2.0), (16, 1.0)))
    R = T
    ids = [int(x) for x in rng.integers(-1, 4, R)]
    if R >= 24:
        ids[:5] = [3, -1, 0, 2, 1]
    else:
        ids[0] = 2
    P = [int(x) for x in rng.integers(0, 300, R)]
    a_req = [P[i] + (1 if (ids[i] >= 0 and i % 3 == 1) else 0) for i in range(R)]   # gate closed on this step
    if R == 1:
        b2 = wl.make_batch(MID, P + [7], [1, 1], ids + [1], rng, activation_offsets=a_req + [8])   # one open, one closed row
        return _check_projection(oracle64, MID, w, ads, b2)
    b = wl.make_batch(MID, P, [1] * R, ids, rng, activation_offsets=a_req)
    _check_projection(oracle64, MID, w, ads, b)


def test_projection_few_row_route_short_suffixes_one_adapter(oracle64):
    """8 requests x 16 new tokens (128 rows), one adapter, gates opening inside the chunk."""
    rng = np.random.default_rng(49)
    w = wl.make_wqkv(MID, rng)
    ads = _boosted_adapters(MID, rng, ((32, 1.0),))
    P = [100 + 13 * i for i in range(8)]
    a_req = [P[i] + (5 if i % 2 else 0) for i in range(8)]
    b = wl.make_batch(MID, P, [16] * 8, [0] * 8, rng, activation_offsets=a_req)
    _check_projection(oracle64, MID, w, ads, b, n_off_expected=20)


def test_decode_sized_stack_takes_the_few_row_projections(oracle64):
    """Two decoder layers on a batch of 40 rows (requests of 1 .. 6 new tokens on cached prefixes made by a base
    prefill through the same stack): q/k/v, o_proj, gate/up and down all run on the few-row route, the last three
    with the residual added in its second kernel."""
    shape = wl.LayerShape(hidden=512, n_q_heads=4, n_kv_heads=2, head_dim=128, page_size=16, dtype="bf16",
                          intermediate=1024)
    rng = np.random.default_rng(33)
    layers = [wl.make_stack_weights(shape, rng) for _ in range(2)]
    ads = [[wl.make_adapter(shape, 16, rng), wl.make_adapter(shape, 8, rng)] for _ in range(2)]
    for per in ads:
        for a in per:
            for n in ("Bq", "Bk", "Bv"):
                setattr(a, n, wl.bf16_round(getattr(a, n) * 8))
    S = [1, 6, 2, 5, 3, 4, 1, 6, 2, 5, 3, 2]
    assert sum(S) == 40
    ids = [0, 1, -1, 0, 1, -1, 1, 0, -1, 1, 0, 1]
    b = wl.make_batch(shape, [0] * len(S), S, ids, rng, activation_offsets=[2 if i % 4 == 1 else 0 for i in range(len(S))],
                      shuffle_pages=True)
    g = hp.GpuLayers(shape, layers, ads, 128, 16)
    try:
        d = hp.DevBatch(b, shape.dtype)
        pools = [g.new_pool(b.num_pages) for _ in range(2)]
        hout = g.empty(b.T, shape.hidden)
        ab.alora_forward_stack(g.ctx, ab.MODE_ALORA, d.hidden, d.positions, d.a_req, d.ids, d.qsl, d.seq_lens, pools,
                               d.bt, d.max_blocks, b.num_pages, d.T, d.R, hout)
        assert g.status() == 0
        x = b.hidden.astype(np.float64)
        for l in range(2):
            x, blk = oracle64.decoder_layer(x, layers[l], shape.Nq, shape.Nkv, shape.n_q_heads, shape.n_kv_heads,
                                            shape.head_dim, 1e-5, b.positions, b.query_start_loc,
                                            b.activation_offsets, b.adapter_ids, hp.oracle_adapters(ads[l]),
                                            [None] * b.R, [None] * b.R)
            got = _gather_pool(oracle64, shape, hp.to_host(pools[l]), b)
            for r in range(b.R):
                hp.assert_close(got[r][0], blk["K"][r], 2e-2, f"layer {l} K rows of request {r}")
        hp.assert_close(hp.to_host(hout), x, 2e-2, "stack output")
    finally:
        g.close()


def test_projection_with_128_wide_kv_blocks(oracle64):
    """One KV head of 128 columns: the q/k/v block boundaries force 128-wide column tiles, and the rank-r
    shrink then runs as the separate cluster split-K kernel."""
    shape = wl.LayerShape(hidden=1536, n_q_heads=4, n_kv_heads=1, head_dim=128, page_size=16, dtype="bf16")
    rng = np.random.default_rng(41)
    w = wl.make_wqkv(shape, rng)
    ads = _boosted_adapters(shape, rng, ((64, 1.0), (8, 2.0)))
    b = wl.make_batch(shape, [0, 50, 10], [600, 440, 277], [0, 1, 0], rng, activation_offsets=[100, 50, 0])
    _check_projection(oracle64, shape, w, ads, b, n_off_expected=100)


def test_short_suffixes_on_an_empty_or_tiny_cache(oracle64):
    """Requests with 5 .. 40 new tokens and 0 .. 70 cached ones: attention work items of one or two key tiles whose
    rows all fall into one query group of the tensor-core kernel (both groups then share the item, one 64-key half
    of the tile each), including items where one half holds no visible key at all, and the NaN-proofing of V rows
    beyond the causal limit (the pool starts as all-ones bit patterns)."""
    import torch
    rng = np.random.default_rng(47)
    w = wl.make_wqkv(MID, rng)
    ads = _boosted_adapters(MID, rng, ((8, 1.0), (32, 1.0)))
    P = [0, 0, 3, 0, 70, 0, 12]
    S = [5, 9, 20, 40, 6, 32, 33]
    ids = [0, 1, -1, 0, 1, 0, 1]
    b = wl.make_batch(MID, P, S, ids, rng, shuffle_pages=True, with_prefix_hidden=True)
    g = hp.GpuLayers(MID, [dict(wqkv=w)], [ads], 256, 8)
    try:
        pool = g.new_pool(b.num_pages)
        pool.view(torch.int16).fill_(-1)   # bf16 NaN everywhere a kernel does not write
        _run_base_prefill(g, MID, b, pool)
        d = hp.DevBatch(b, MID.dtype)
        out = g.empty(b.T, MID.Nq)
        ab.alora_prefill_layer(g.ctx, 0, d.hidden, d.positions, d.a_req, d.ids, d.qsl, d.seq_lens, pool, d.bt,
                               d.max_blocks, b.num_pages, d.T, d.R, out)
        assert g.status() == 0
        Ks, Vs = hp.oracle_base_prefix(oracle64, MID, w, b)
        want = hp.oracle_block(oracle64, MID, w, ads, b, Ks, Vs)
        out_h = hp.to_host(out)
        assert np.isfinite(out_h).all()
        for r in range(b.R):
            q0, q1 = int(b.query_start_loc[r]), int(b.query_start_loc[r + 1])
            hp.assert_close(out_h[q0:q1], want["out"][q0:q1], 2e-2, f"request {r}")
    finally:
        g.close()


def test_full_lora_recompute_matches_eq4(oracle64):
    w, ads, b = _mid_workload(seed=13)
    fb = hp.full_sequence_batch(MID, b)
    g = hp.GpuLayers(MID, [dict(wqkv=w)], [ads], fb.T, fb.R)
    try:
        d = hp.DevBatch(fb, MID.dtype)
        pool = g.new_pool(b.num_pages)
        out = g.empty(fb.T, MID.Nq)
        ab.alora_full_lora_prefill_layer(g.ctx, 0, d.hidden, d.positions, d.ids, d.qsl, d.seq_lens, pool, d.bt,
                                         d.max_blocks, b.num_pages, d.T, d.R, out)
        assert g.status() == 0
        want = hp.oracle_block(oracle64, MID, w, ads, fb, [None] * fb.R, [None] * fb.R, force_all=True)
        hp.assert_close(hp.to_host(out), want["out"], 2e-2, "")
        got = _gather_pool(oracle64, MID, hp.to_host(pool), fb)
        for r in range(fb.R):
            hp.assert_close(got[r][0], want["K"][r], 2e-2, "")
            hp.assert_close(got[r][1], want["V"][r], 2e-2, "")
    finally:
        g.close()


def test_cache_reuse_identity_on_gpu(oracle64):
    """Prop. 1 on the GPU: masked aLoRA prefill of the whole sequence from scratch leaves the same
    cache as base prefill of the prefix + aLoRA suffix prefill, and the same suffix outputs."""
    w, ads, b = _mid_workload(seed=14, a_req_shift=False)
    fb = hp.full_sequence_batch(MID, b)
    g = hp.GpuLayers(MID, [dict(wqkv=w)], [ads], fb.T, fb.R)
    try:
        pool_a = g.new_pool(b.num_pages)
        _run_base_prefill(g, MID, b, pool_a)
        d = hp.DevBatch(b, MID.dtype)
        out_a = g.empty(b.T, MID.Nq)
        ab.alora_prefill_layer(g.ctx, 0, d.hidden, d.positions, d.a_req, d.ids, d.qsl, d.seq_lens, pool_a, d.bt,
                               d.max_blocks, b.num_pages, d.T, d.R, out_a)
        df = hp.DevBatch(fb, MID.dtype)
        pool_b = g.new_pool(b.num_pages)
        out_b = g.empty(fb.T, MID.Nq)
        ab.alora_prefill_layer(g.ctx, 0, df.hidden, df.positions, df.a_req, df.ids, df.qsl, df.seq_lens, pool_b,
                               df.bt, df.max_blocks, b.num_pages, df.T, df.R, out_b)
        assert g.status() == 0
        pa, pb = hp.to_host(pool_a), hp.to_host(pool_b)
        ka = _gather_pool(oracle64, MID, pa, b); kb = _gather_pool(oracle64, MID, pb, b)
        oa, ob = hp.to_host(out_a), hp.to_host(out_b)
        for r in range(b.R):
            P = int(b.prefix_lens[r])
            # prefix rows: exact (both are base-only arithmetic on the same inputs)
            assert np.array_equal(ka[r][0][:P].view(np.uint32), kb[r][0][:P].view(np.uint32))
            assert np.array_equal(ka[r][1][:P].view(np.uint32), kb[r][1][:P].view(np.uint32))
            hp.assert_close(ka[r][0], kb[r][0], 2e-2, "K")
            hp.assert_close(ka[r][1], kb[r][1], 2e-2, "V")
            lo, hi = b.query_start_loc[r], b.query_start_loc[r + 1]
            tail = slice(fb.query_start_loc[r] + P, fb.query_start_loc[r + 1])
            hp.assert_close(ob[tail], oa[lo:hi], 2e-2, "")
    finally:
        g.close()


def test_decode_steps_match_prefill_rows(oracle64):
    """Prop. 1, second sentence: decoding the suffix token by token reproduces the prefill."""
    rng = np.random.default_rng(21)
    w = wl.make_wqkv(MID, rng)
    ads = [wl.make_adapter(MID, 32, rng), wl.make_adapter(MID, 16, rng)]
    for a in ads:
        for n in ("Bq", "Bk", "Bv"):
            setattr(a, n, wl.bf16_round(getattr(a, n) * 8))
    P, S = [40, 333, 17, 64, 100], [6, 6, 6, 6, 6]
    ids = [0, -1, 1, 0, 1]
    a_req = [42, 0, 17, 0, 103]
    b = wl.make_batch(MID, P, S, ids, rng, activation_offsets=a_req, shuffle_pages=True, with_prefix_hidden=True)
    g = hp.GpuLayers(MID, [dict(wqkv=w)], [ads], 1024, 8)
    try:
        import torch
        pool = g.new_pool(b.num_pages)
        _run_base_prefill(g, MID, b, pool)
        pool_dec = pool.clone()
        d = hp.DevBatch(b, MID.dtype)
        out = g.empty(b.T, MID.Nq)
        ab.alora_prefill_layer(g.ctx, 0, d.hidden, d.positions, d.a_req, d.ids, d.qsl, d.seq_lens, pool, d.bt,
                               d.max_blocks, b.num_pages, d.T, d.R, out)
        out_h = hp.to_host(out)
        dec = np.zeros_like(out_h)
        for i in range(6):
            rows = b.query_start_loc[:-1] + i
            hid = d.hidden[torch.from_numpy(rows).cuda().long()].contiguous()
            pos = hp.idev(b.positions[rows]); sl = hp.idev(b.positions[rows] + 1)
            o = g.empty(b.R, MID.Nq)
            ab.alora_decode_step(g.ctx, 0, hid, pos, d.a_req, d.ids, sl, pool_dec, d.bt, d.max_blocks, b.num_pages,
                                 b.R, o)
            dec[rows] = hp.to_host(o)
        assert g.status() == 0
        Ks, Vs = hp.oracle_base_prefix(oracle64, MID, w, b)
        want = hp.oracle_block(oracle64, MID, w, ads, b, Ks, Vs)
        hp.assert_close(out_h, want["out"], 2e-2, "")
        hp.assert_close(dec, want["out"], 2e-2, "")
        hp.assert_close(hp.to_host(pool_dec), hp.to_host(pool), 2e-2, "")
    finally:
        g.close()


def test_two_layer_stack(oracle64):
    """Reduced decoder stack end to end (RMSNorm, attention block, o_proj, SwiGLU MLP, residuals)."""
    shape = wl.LayerShape(hidden=512, n_q_heads=4, n_kv_heads=2, head_dim=128, page_size=16, dtype="bf16",
                          intermediate=1024)
    rng = np.random.default_rng(31)
    layers = [wl.make_stack_weights(shape, rng) for _ in range(2)]
    ads = [[wl.make_adapter(shape, 16, rng)] for _ in range(2)]
    for per in ads:
        for a in per:
            for n in ("Bq", "Bk", "Bv"):
                setattr(a, n, wl.bf16_round(getattr(a, n) * 8))
    b = wl.make_batch(shape, [0, 0], [200, 77], [0, -1], rng, activation_offsets=[150, 0], shuffle_pages=True)
    g = hp.GpuLayers(shape, layers, ads, 512, 4)
    try:
        d = hp.DevBatch(b, shape.dtype)
        pools = [g.new_pool(b.num_pages) for _ in range(2)]
        hout = g.empty(b.T, shape.hidden)
        ab.alora_forward_stack(g.ctx, ab.MODE_ALORA, d.hidden, d.positions, d.a_req, d.ids, d.qsl, d.seq_lens, pools,
                               d.bt, d.max_blocks, b.num_pages, d.T, d.R, hout)
        assert g.status() == 0
        x = b.hidden.astype(np.float64)
        for l in range(2):
            x, blk = oracle64.decoder_layer(x, layers[l], shape.Nq, shape.Nkv, shape.n_q_heads, shape.n_kv_heads,
                                            shape.head_dim, 1e-5, b.positions, b.query_start_loc,
                                            b.activation_offsets, b.adapter_ids, hp.oracle_adapters(ads[l]),
                                            [None] * b.R, [None] * b.R)
            got = _gather_pool(oracle64, shape, hp.to_host(pools[l]), b)
            for r in range(b.R):
                hp.assert_close(got[r][0], blk["K"][r], 2e-2, "")
        hp.assert_close(hp.to_host(hout), x, 2e-2, "")
    finally:
        g.close()


def test_stack_layer_with_many_rows_takes_the_256_row_gemm(oracle64):
    """One decoder layer on 2048 tokens with a wide MLP: gate/up (2048 x 9472 outputs = 296 tiles of 256 x 256) runs
    on the 256-row GEMM kernel, o_proj and down (one column tile) on the 128-row kernel."""
    shape = wl.LayerShape(hidden=256, n_q_heads=4, n_kv_heads=2, head_dim=64, page_size=16, dtype="bf16",
                          intermediate=4736)
    rng = np.random.default_rng(41)
    layers = [wl.make_stack_weights(shape, rng)]
    ads = [[wl.make_adapter(shape, 8, rng)]]
    b = wl.make_batch(shape, [0] * 8, [256] * 8, [0, -1] * 4, rng, activation_offsets=[100] * 8, shuffle_pages=True)
    g = hp.GpuLayers(shape, layers, ads, 2048, 8)
    try:
        d = hp.DevBatch(b, shape.dtype)
        pools = [g.new_pool(b.num_pages)]
        hout = g.empty(b.T, shape.hidden)
        ab.alora_forward_stack(g.ctx, ab.MODE_ALORA, d.hidden, d.positions, d.a_req, d.ids, d.qsl, d.seq_lens, pools,
                               d.bt, d.max_blocks, b.num_pages, d.T, d.R, hout)
        assert g.status() == 0
        x, _ = oracle64.decoder_layer(b.hidden.astype(np.float64), layers[0], shape.Nq, shape.Nkv, shape.n_q_heads,
                                      shape.n_kv_heads, shape.head_dim, 1e-5, b.positions, b.query_start_loc,
                                      b.activation_offsets, b.adapter_ids, hp.oracle_adapters(ads[0]),
                                      [None] * b.R, [None] * b.R)
        hp.assert_close(hp.to_host(hout), x, 2e-2, "")
    finally:
        g.close()


def test_stack_layer_at_the_8b_shape_with_1024_rows(oracle64):
    """One decoder layer at the 8B layer shape on 4 x 256 new tokens: q/k/v on the 128-row tile route with the fused
    shrink, o_proj, gate / up (28672 columns) and down (K = 14336) on the 256 x 256 dense kernel, the 16-byte norm and
    SwiGLU kernels at their real row lengths.  Every row against the oracle (about 0.23 TFLOP of oracle work)."""
    shape = wl.SHAPE_8B
    rng = np.random.default_rng(48)
    layers = [wl.make_stack_weights(shape, rng)]
    ads = [[wl.make_adapter(shape, 32, rng)]]
    for n in ("Bq", "Bk", "Bv"):
        setattr(ads[0][0], n, wl.bf16_round(getattr(ads[0][0], n) * 8))
    b = wl.make_batch(shape, [0] * 4, [256] * 4, [0, -1, 0, 0], rng, activation_offsets=[100, 0, 0, 255],
                      shuffle_pages=True)
    g = hp.GpuLayers(shape, layers, ads, 1024, 4)
    try:
        d = hp.DevBatch(b, shape.dtype)
        pools = [g.new_pool(b.num_pages)]
        hout = g.empty(b.T, shape.hidden)
        ab.alora_forward_stack(g.ctx, ab.MODE_ALORA, d.hidden, d.positions, d.a_req, d.ids, d.qsl, d.seq_lens, pools,
                               d.bt, d.max_blocks, b.num_pages, d.T, d.R, hout)
        assert g.status() == 0
        x, _ = oracle64.decoder_layer(b.hidden.astype(np.float64), layers[0], shape.Nq, shape.Nkv, shape.n_q_heads,
                                      shape.n_kv_heads, shape.head_dim, 1e-5, b.positions, b.query_start_loc,
                                      b.activation_offsets, b.adapter_ids, hp.oracle_adapters(ads[0]),
                                      [None] * b.R, [None] * b.R)
        hp.assert_close(hp.to_host(hout), x, 2e-2, "8B-shape layer, 1024 rows", block=shape.head_dim)
    finally:
        g.close()


def test_empty_and_degenerate_batches():
    w, ads, b = _mid_workload()
    g = hp.GpuLayers(MID, [dict(wqkv=w)], [ads], 256, 8)
    try:
        import torch
        # T = 0: nothing launched that touches memory, status stays clean
        z = torch.zeros(1, dtype=torch.int32, device="cuda")
        pool = g.new_pool(4)
        out = g.empty(1, MID.Nq)
        ab.alora_prefill_layer(g.ctx, 0, out, z, z, z, z, z, pool, z, 1, 4, 0, 0, out)
        assert g.status() == 0
        # a request with zero new tokens between two non-empty ones
        rng = np.random.default_rng(5)
        b2 = wl.make_batch(MID, [5, 9, 0], [3, 0, 2], [0, 1, -1], rng, shuffle_pages=True)
        d = hp.DevBatch(b2, MID.dtype)
        fill = wl.random_kv_pool(MID, b2.num_pages, rng)
        pool = g.new_pool(b2.num_pages, fill)
        out = g.empty(b2.T, MID.Nq)
        ab.alora_prefill_layer(g.ctx, 0, d.hidden, d.positions, d.a_req, d.ids, d.qsl, d.seq_lens, pool, d.bt,
                               d.max_blocks, b2.num_pages, d.T, d.R, out)
        assert g.status() == 0
        assert np.isfinite(hp.to_host(out)).all()
        # host-side rejections: nothing is launched
        n0 = ab.alora_launch_count(g.ctx)
        for bad in (dict(T=10 ** 6), dict(layer=3), dict(hidden=None)):
            args = dict(layer=0, hidden=d.hidden, T=d.T)
            args.update(bad)
            with pytest.raises(ab.AloraError):
                ab.alora_prefill_layer(g.ctx, args["layer"], args["hidden"], d.positions, d.a_req, d.ids, d.qsl,
                                       d.seq_lens, pool, d.bt, d.max_blocks, b2.num_pages, args["T"], d.R, out)
        assert ab.alora_launch_count(g.ctx) == n0
    finally:
        g.close()


def test_device_side_findings_are_reported_not_trapped():
    """A block-table entry outside the pool and inconsistent positions are recorded in the status
    word; the offending rows are skipped and the context stays usable."""
    w, ads, b = _mid_workload()
    g = hp.GpuLayers(MID, [dict(wqkv=w)], [ads], 2048, 8)
    try:
        rng = np.random.default_rng(6)
        fill = wl.random_kv_pool(MID, b.num_pages, rng)
        d = hp.DevBatch(b, MID.dtype)
        pool = g.new_pool(b.num_pages, fill)
        out = g.empty(b.T, MID.Nq)
        bt = b.block_tables.copy()
        last_blk = (int(b.seq_lens[0]) - 1) // MID.page_size
        bt[0, last_blk] = b.num_pages + 5
        ab.alora_prefill_layer(g.ctx, 0, d.hidden, d.positions, d.a_req, d.ids, d.qsl, d.seq_lens, pool, hp.idev(bt),
                               d.max_blocks, b.num_pages, d.T, d.R, out)
        assert g.status() == 7
        pos = b.positions.copy(); pos[3] += 2
        ab.alora_prefill_layer(g.ctx, 0, d.hidden, hp.idev(pos), d.a_req, d.ids, d.qsl, d.seq_lens, pool, d.bt,
                               d.max_blocks, b.num_pages, d.T, d.R, out)
        assert g.status() == 6
        ab.alora_prefill_layer(g.ctx, 0, d.hidden, d.positions, d.a_req, d.ids, d.qsl, d.seq_lens, pool, d.bt,
                               d.max_blocks, b.num_pages, d.T, d.R, out)
        assert g.status() == 0
    finally:
        g.close()


def test_decode_steps_through_the_stack_match_the_prefill_rows(oracle64):
    """Two decoder layers: a prefill of all but the last three tokens of every request, then three decode steps
    through alora_decode_stack; the rows the steps produce equal the rows of the oracle's stack over the whole
    sequences (Prop. 1, second sentence), for requests on two adapters and on the base model, with gates that open
    before, inside and after the prefilled part."""
    shape = wl.LayerShape(hidden=512, n_q_heads=4, n_kv_heads=2, head_dim=128, page_size=16, dtype="bf16",
                          intermediate=1024)
    rng = np.random.default_rng(37)
    layers = [wl.make_stack_weights(shape, rng) for _ in range(2)]
    ads = [[wl.make_adapter(shape, 16, rng), wl.make_adapter(shape, 8, rng)] for _ in range(2)]
    for per in ads:
        for a in per:
            for n in ("Bq", "Bk", "Bv"):
                setattr(a, n, wl.bf16_round(getattr(a, n) * 8))
    L = [40, 23, 64, 9, 31]
    ids = [0, 1, -1, 0, 1]
    a_req = [10, 22, 0, 0, 100]
    n_dec = 3
    full = wl.make_batch(shape, [0] * len(L), L, ids, rng, activation_offsets=a_req, shuffle_pages=True)
    R = full.R
    g = hp.GpuLayers(shape, layers, ads, 256, 8)
    try:
        pools = [g.new_pool(full.num_pages) for _ in range(2)]
        # prefill part: tokens 0 .. L-4 of every request
        keep = np.concatenate([np.arange(full.query_start_loc[r], full.query_start_loc[r + 1] - n_dec) for r in range(R)])
        pre = wl.Batch(positions=full.positions[keep],
                       query_start_loc=np.concatenate([[0], np.cumsum(np.array(L) - n_dec)]).astype(np.int32),
                       seq_lens=(np.array(L) - n_dec).astype(np.int32), prefix_lens=np.zeros(R, np.int32),
                       activation_offsets=full.activation_offsets, adapter_ids=full.adapter_ids,
                       block_tables=full.block_tables, num_pages=full.num_pages, hidden=full.hidden[keep])
        d = hp.DevBatch(pre, shape.dtype)
        hout = g.empty(pre.T, shape.hidden)
        ab.alora_forward_stack(g.ctx, ab.MODE_ALORA, d.hidden, d.positions, d.a_req, d.ids, d.qsl, d.seq_lens, pools,
                               d.bt, d.max_blocks, full.num_pages, d.T, d.R, hout)
        got = np.zeros((R, n_dec, shape.hidden), np.float32)
        for i in range(n_dec):
            rows = full.query_start_loc[1:] - n_dec + i
            pos = full.positions[rows]
            hid = hp.to_dev(full.hidden[rows], "bf16")
            o = g.empty(R, shape.hidden)
            ab.alora_decode_stack(g.ctx, hid, hp.idev(pos), d.a_req, d.ids, hp.idev(pos + 1), pools, d.bt, d.max_blocks,
                                  full.num_pages, R, o)
            got[:, i] = hp.to_host(o)
        assert g.status() == 0
        x = full.hidden.astype(np.float64)
        for l in range(2):
            x, _ = oracle64.decoder_layer(x, layers[l], shape.Nq, shape.Nkv, shape.n_q_heads, shape.n_kv_heads,
                                          shape.head_dim, 1e-5, full.positions, full.query_start_loc,
                                          full.activation_offsets, full.adapter_ids, hp.oracle_adapters(ads[l]),
                                          [None] * R, [None] * R)
        for i in range(n_dec):
            rows = full.query_start_loc[1:] - n_dec + i
            hp.assert_close(got[:, i], x[rows], 2e-2, f"decode step {i} through the stack")
        hp.assert_close(hp.to_host(hout), x[keep], 2e-2, "prefilled rows")
    finally:
        g.close()

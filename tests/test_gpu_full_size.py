"""GPU parity at the full sizes of the named configurations, in the launch configuration bench.py times:
the whole batch runs on the GPU, and the outputs of a few sampled requests (every row of them) are compared
with the CPU oracle, which computes those requests one by one from the same inputs.  The cached prefix is a
seeded N(0,1) fill of the page pool made on the device (it stands in for the base model's cache; the rows the
oracle needs are copied back from the very pool the kernels read)."""
import numpy as np
import pytest

from paper_2504_12397_b200 import binding as ab
from paper_2504_12397_b200 import workloads as wl

import helpers as hp

pytestmark = pytest.mark.gpu


def _device_pool(shape, num_pages, seed):
    import torch
    g = torch.Generator(device="cuda"); g.manual_seed(seed)
    pool = torch.empty((num_pages, 2, shape.n_kv_heads, shape.page_size, shape.head_dim), device="cuda",
                       dtype=torch.bfloat16)
    for i in range(0, num_pages, 8192):
        n = min(8192, num_pages - i)
        pool[i:i + n] = torch.randn((n,) + tuple(pool.shape[1:]), generator=g, device="cuda",
                                    dtype=torch.float32).to(torch.bfloat16)
    return pool


def _request_kv(pool, b, r, length, shape):
    """Contiguous (K, V) [length, Nkv] float32 of request r, copied from the device pool through its block table."""
    import torch
    nblk = (length + shape.page_size - 1) // shape.page_size
    pages = torch.from_numpy(b.block_tables[r, :nblk].astype(np.int64)).cuda()
    blk = pool[pages].to(torch.float32).cpu().numpy()          # [nblk, 2, Hkv, page, hd]
    kv = blk.transpose(1, 0, 3, 2, 4).reshape(2, nblk * shape.page_size, shape.Nkv)
    return kv[0, :length], kv[1, :length]


def _sub_batch(b, r):
    q0, q1 = int(b.query_start_loc[r]), int(b.query_start_loc[r + 1])
    return q0, q1, wl.Batch(positions=b.positions[q0:q1], query_start_loc=np.array([0, q1 - q0], np.int32),
                            seq_lens=b.seq_lens[r:r + 1], prefix_lens=b.prefix_lens[r:r + 1],
                            activation_offsets=b.activation_offsets[r:r + 1], adapter_ids=b.adapter_ids[r:r + 1],
                            block_tables=b.block_tables[r:r + 1], num_pages=b.num_pages, hidden=b.hidden[q0:q1])


def _check_requests(oracle, shape, w, b, pool_before, pool_after, out_h, sample, qkv_h=None):
    for r in sample:
        P, L = int(b.prefix_lens[r]), int(b.seq_lens[r])
        K0, V0 = _request_kv(pool_before, b, r, P, shape)
        q0, q1, sub = _sub_batch(b, r)
        want = hp.oracle_block(oracle, shape, w.wqkv, w.adapters, sub, [K0 if P else None], [V0 if P else None])
        hd = shape.head_dim
        hp.assert_close(out_h[q0:q1], want["out"], 2e-2, f"attention output of request {r}", block=hd)
        if qkv_h is not None:
            hp.assert_close(qkv_h[q0:q1], want["qkv"], 2e-2, f"projection rows of request {r}", block=hd)
        K1, V1 = _request_kv(pool_after, b, r, L, shape)
        hp.assert_close(K1[P:], want["K"][0][P:], 2e-2, f"appended K rows of request {r}", block=hd)
        hp.assert_close(V1[P:], want["V"][0][P:], 2e-2, f"appended V rows of request {r}", block=hd)
        # the cached prefix of the request is untouched, bit for bit
        assert np.array_equal(K1[:P].view(np.uint32), K0.view(np.uint32))
        assert np.array_equal(V1[:P].view(np.uint32), V0.view(np.uint32))


def _run_layer(w, seed, decode=False, with_qkv=False):
    import torch
    shape, b = w.shape, w.batch
    g = hp.GpuLayers(shape, [dict(wqkv=w.wqkv)], [w.adapters], b.T, b.R)
    try:
        pool = _device_pool(shape, b.num_pages, seed)
        before = pool.clone()
        d = hp.DevBatch(b, "bf16")
        out = g.empty(b.T, shape.Nq)
        if decode:
            ab.alora_decode_step(g.ctx, 0, d.hidden, d.positions, d.a_req, d.ids, d.seq_lens, pool, d.bt, d.max_blocks,
                                 b.num_pages, b.R, out)
        else:
            ab.alora_prefill_layer(g.ctx, 0, d.hidden, d.positions, d.a_req, d.ids, d.qsl, d.seq_lens, pool, d.bt,
                                   d.max_blocks, b.num_pages, b.T, b.R, out)
        qkv_h = None
        if with_qkv:
            qkv = g.empty(b.T, shape.N)
            ab.alora_project_qkv(g.ctx, 0, ab.MODE_ALORA, d.hidden, d.positions, d.a_req, d.ids, d.qsl, d.seq_lens,
                                 b.T, b.R, qkv)
            qkv_h = hp.to_host(qkv)
        assert g.status() == 0
        return before, pool, hp.to_host(out), qkv_h
    finally:
        g.close()


def test_config2_bench_workload_sampled_requests(oracle64):
    """8 requests x (4096 cached + 256 suffix tokens), rank 32: the whole workload, every row of every request."""
    w = wl.config2(seed=2)
    before, after, out_h, qkv_h = _run_layer(w, seed=1002, with_qkv=True)
    _check_requests(oracle64, w.shape, w, w.batch, before, after, out_h, range(w.batch.R), qkv_h)


def test_chunk_straddling_prefill_at_the_bench_shape(oracle64):
    """The headline shape with the activation offset 192 tokens into the 256 new ones (the paper's second regime: an
    uncached tail of the context and the invocation in one call).  Requests 0 and 7 against the oracle; and the
    rows before the offset are BASE-EXACT: their projection rows and their appended K/V have the bits of a call
    with every gate closed, so the base model can later reuse what this call cached for them."""
    w = wl.config2(seed=12, activation_shift=192)
    b, shape = w.batch, w.shape
    before, after, out_h, qkv_h = _run_layer(w, seed=1012, with_qkv=True)
    _check_requests(oracle64, shape, w, b, before, after, out_h, [0, b.R - 1], qkv_h)
    import copy
    wb = copy.copy(w)
    wb.batch = copy.copy(b)
    wb.batch.adapter_ids = np.full(b.R, -1, np.int32)
    _, after_b, _, qkv_b = _run_layer(wb, seed=1012, with_qkv=True)
    S = 256
    closed = np.concatenate([np.arange(r * S, r * S + 192) for r in range(b.R)])
    opened = np.setdiff1d(np.arange(b.T), closed)
    assert np.array_equal(qkv_h[closed].view(np.uint32), qkv_b[closed].view(np.uint32))
    assert hp.rel_err(qkv_h[opened], qkv_b[opened]) > 1e-3
    for r in (0, 3, b.R - 1):
        P = int(b.prefix_lens[r])
        Ka, Va = _request_kv(after, b, r, P + S, shape)
        Kb, Vb = _request_kv(after_b, b, r, P + S, shape)
        assert np.array_equal(Ka[:P + 192].view(np.uint32), Kb[:P + 192].view(np.uint32)), f"base-exact K of request {r}"
        assert np.array_equal(Va[:P + 192].view(np.uint32), Vb[:P + 192].view(np.uint32)), f"base-exact V of request {r}"
        assert not np.array_equal(Ka[P + 192:], Kb[P + 192:])


def test_config3_ragged_multi_adapter_sampled_requests(oracle64):
    """32 requests over adapters of ranks 8/16/32/64, prefixes 512..16384, suffixes 16..512, shuffled pages:
    in full, the request with the most work (longest suffix x context), the request with the most work on the
    rank-64 adapter and on the rank-8 adapter, the two with the least work and the one with the shortest suffix;
    and the projection rows of the whole batch."""
    w = wl.config3(seed=3)
    b = w.batch
    S = (b.seq_lens - b.prefix_lens).astype(np.int64)
    work = S * b.seq_lens.astype(np.int64)
    by_work = np.argsort(work)
    sample = {int(by_work[-1]), int(by_work[0]), int(by_work[1]), int(np.argmin(S))}
    for ad in (0, 3):   # ranks 8 and 64
        on = np.nonzero(b.adapter_ids == ad)[0]
        assert len(on) > 0
        sample.add(int(on[np.argmax(work[on])]))
    before, after, out_h, qkv_h = _run_layer(w, seed=1003, with_qkv=True)
    _check_requests(oracle64, w.shape, w, b, before, after, out_h, sorted(sample), qkv_h)
    want, gate = oracle64.project_qkv(b.hidden, w.wqkv, w.shape.Nq, w.shape.Nkv, b.positions, b.query_start_loc,
                                      b.activation_offsets, b.adapter_ids, hp.oracle_adapters(w.adapters))
    hp.assert_close(qkv_h, want, 2e-2, "projection rows of the whole batch", block=w.shape.head_dim)


def test_long_uniform_batch_whole_items_and_cut_items(oracle64):
    """28 requests x (15400 cached + 1024 suffix tokens) on a small layer shape: 448 attention work items of about
    125 key tiles each, three full rounds over the 148 blocks plus 4 items.  The kernel takes 444 items whole and
    cuts the last 4 into runs of key tiles that many blocks work on, merged afterwards.  Request 27 holds the cut
    items, request 0 only whole ones."""
    shape = wl.LayerShape(hidden=256, n_q_heads=4, n_kv_heads=2, head_dim=64, page_size=16, dtype="bf16")
    w = wl.config2(seed=11, requests=28, prefix=15400, suffix=1024, shape=shape, rank=8)
    before, after, out_h, _ = _run_layer(w, seed=1011)
    _check_requests(oracle64, w.shape, w, w.batch, before, after, out_h, [0, 27])


def test_five_adapters_on_one_shared_prefix_cache(oracle64):
    """Five requests (four different adapters and the base model) whose block tables point at the SAME physical
    pages for their 512 cached positions: every request reads the one base-model prefix cache, writes only its own
    suffix pages, and the shared pages stay bit-identical."""
    shape = wl.LayerShape(hidden=256, n_q_heads=8, n_kv_heads=2, head_dim=128, page_size=16, dtype="bf16")
    rng = np.random.default_rng(77)
    P, S, ids = 512, [40, 24, 17, 33, 64], [0, 1, 2, -1, 3]
    wqkv = wl.make_wqkv(shape, rng)
    ads = [wl.make_adapter(shape, r, rng, scale=4.0) for r in (8, 16, 32, 8)]
    b = wl.make_batch(shape, [P] * 5, S, ids, rng, shuffle_pages=True)
    b.block_tables[1:, :P // shape.page_size] = b.block_tables[0, :P // shape.page_size]
    w = wl.Workload("shared_prefix", shape, wqkv, ads, b, 77)
    before, after, out_h, qkv_h = _run_layer(w, seed=1077, with_qkv=True)
    _check_requests(oracle64, shape, w, b, before, after, out_h, range(5), qkv_h)
    shared = b.block_tables[0, :P // shape.page_size].astype(np.int64)
    import torch
    idx = torch.from_numpy(shared).cuda()
    assert torch.equal(before[idx], after[idx])


def test_short_suffixes_of_many_requests_on_long_prefixes(oracle64):
    """40 requests with 1 .. 64 new tokens on 700 .. 2300 cached ones (6 .. 19 key tiles), base model and two
    adapters.  Up to 16 score rows per KV head (here 4 tokens) a request is on the few-row kernel's list; from 5
    to 32 tokens all its rows fall into the first query group of a tensor-core work item, whose second group then
    skips the item; from 33 tokens on both groups work.  One request of every kind is checked in full."""
    shape = wl.LayerShape(hidden=256, n_q_heads=8, n_kv_heads=2, head_dim=128, page_size=16, dtype="bf16")
    rng = np.random.default_rng(91)
    S = [1, 4, 5, 8, 16, 31, 32, 33, 47, 64] * 4
    P = [int(x) for x in rng.integers(700, 2300, size=len(S))]
    ids = [(-1, 0, 1)[i % 3] for i in range(len(S))]
    wqkv = wl.make_wqkv(shape, rng)
    ads = [wl.make_adapter(shape, r, rng, scale=4.0) for r in (8, 32)]
    b = wl.make_batch(shape, P, S, ids, rng, shuffle_pages=True)
    w = wl.Workload("short_suffixes", shape, wqkv, ads, b, 91)
    before, after, out_h, qkv_h = _run_layer(w, seed=1091, with_qkv=True)
    _check_requests(oracle64, shape, w, b, before, after, out_h, [10, 21, 12, 33, 4, 25, 36, 17, 38, 9], qkv_h)


def test_many_requests_with_two_to_four_new_tokens_take_the_tensor_core_kernel(oracle64):
    """200 requests with 1 .. 4 new tokens (G = 4: at most 16 score rows per KV head) on 300 .. 1500 cached ones.
    160 of them have 2 .. 4 tokens: 320 KV streams for 148 SMs, so the work-list builder sends those to the
    tensor-core kernel (as items shared by its two query groups) and only the one-token requests to the few-row
    kernel.  One request of every length, and the projection rows of all."""
    shape = wl.LayerShape(hidden=256, n_q_heads=8, n_kv_heads=2, head_dim=128, page_size=16, dtype="bf16")
    rng = np.random.default_rng(95)
    S = [2, 3, 4, 1, 4] * 40
    P = [int(x) for x in rng.integers(300, 1500, size=len(S))]
    ids = [(-1, 0, 1)[i % 3] for i in range(len(S))]
    wqkv = wl.make_wqkv(shape, rng)
    ads = [wl.make_adapter(shape, r, rng, scale=4.0) for r in (8, 32)]
    b = wl.make_batch(shape, P, S, ids, rng, shuffle_pages=True)
    w = wl.Workload("many_short", shape, wqkv, ads, b, 95)
    before, after, out_h, qkv_h = _run_layer(w, seed=1095, with_qkv=True)
    _check_requests(oracle64, shape, w, b, before, after, out_h, [0, 51, 102, 153, 199], qkv_h)


def test_few_requests_with_long_contexts_are_spread_over_all_blocks(oracle64):
    """Three requests with 37 000 .. 52 000 cached tokens and 16, 40 and 100 new ones on a small layer shape: 8
    attention work items of 290 .. 407 key tiles for 148 blocks.  The work-list builder cuts them into runs of
    about 19 tiles, one per block; the parts of an item (for the 16-token request: rows shared by the kernel's two
    query groups) are merged afterwards.  All three requests in full."""
    shape = wl.LayerShape(hidden=256, n_q_heads=8, n_kv_heads=2, head_dim=128, page_size=16, dtype="bf16")
    rng = np.random.default_rng(93)
    P, S, ids = [52000, 37000, 41000], [16, 40, 100], [0, -1, 1]
    wqkv = wl.make_wqkv(shape, rng)
    ads = [wl.make_adapter(shape, r, rng, scale=4.0) for r in (8, 32)]
    b = wl.make_batch(shape, P, S, ids, rng, shuffle_pages=True)
    w = wl.Workload("few_long", shape, wqkv, ads, b, 93)
    before, after, out_h, _ = _run_layer(w, seed=1093)
    _check_requests(oracle64, shape, w, b, before, after, out_h, [0, 1, 2])


_SWEEP_SHAPES = (dict(hidden=256, n_q_heads=8, n_kv_heads=2, head_dim=128, page_size=16),
                 dict(hidden=256, n_q_heads=4, n_kv_heads=2, head_dim=64, page_size=32),
                 dict(hidden=256, n_q_heads=8, n_kv_heads=1, head_dim=128, page_size=64))


@pytest.mark.parametrize("seed", range(10))
def test_randomised_batches_over_all_attention_routes(oracle64, seed):
    """Seeded random batches on three layer shapes (group sizes 4, 2, 8; head dims 128, 64; pages of 16, 32, 64):
    many requests with 1 .. 5 new tokens, one to three requests with 20 000 .. 60 000 cached tokens, ragged mixes,
    short suffixes of a medium number of requests, and tiny caches.  Between them they take every route of the
    attention (few-row kernel, whole / shared / cut work items of the tensor-core kernel, merge of the parts).  The
    requests with the least, the median and the most work plus three random ones are checked in full (those the
    oracle finishes in seconds)."""
    rng = np.random.default_rng(1000 + seed)
    shape = wl.LayerShape(dtype="bf16", **_SWEEP_SHAPES[seed % 3])
    kind = seed % 5
    if kind == 0:
        R = int(rng.integers(100, 330)); S = rng.integers(1, 6, size=R); P = rng.integers(0, 900, size=R)
    elif kind == 1:
        R = int(rng.integers(1, 4)); S = rng.integers(5, 200, size=R); P = rng.integers(20000, 60000, size=R)
    elif kind == 2:
        R = int(rng.integers(2, 30)); S = rng.integers(1, 300, size=R); P = rng.integers(0, 3000, size=R)
    elif kind == 3:
        R = int(rng.integers(8, 80)); S = rng.integers(1, 40, size=R); P = rng.integers(100, 5000, size=R)
    else:
        R = int(rng.integers(1, 12)); S = rng.integers(1, 70, size=R); P = rng.integers(0, 80, size=R)
    ids = [int(x) for x in rng.integers(-1, 2, size=R)]
    wqkv = wl.make_wqkv(shape, rng)
    ads = [wl.make_adapter(shape, r, rng, scale=4.0) for r in (8, 32)]
    b = wl.make_batch(shape, [int(x) for x in P], [int(x) for x in S], ids, rng, shuffle_pages=True)
    w = wl.Workload("sweep", shape, wqkv, ads, b, seed)
    before, after, out_h, _ = _run_layer(w, seed=5000 + seed)
    assert np.isfinite(out_h).all()
    work = b.seq_lens.astype(np.int64) * S
    order = np.argsort(work)
    sample = sorted({int(order[0]), int(order[len(order) // 2]), int(order[-1])} | {int(x) for x in rng.integers(0, R, size=3)})
    sample = [r for r in sample if work[r] < 6e6] or [int(order[0])]
    _check_requests(oracle64, shape, w, b, before, after, out_h, sample)


def test_config5_decode_step_sampled_requests(oracle64):
    """64 requests (base model and 4 rank-32 adapters), contexts 1024..32768, one new token each: the shortest,
    the longest and two more requests, and the projection rows of all 64."""
    w = wl.config5(seed=5)
    b = w.batch
    order = np.argsort(b.seq_lens)
    sample = sorted({int(order[0]), int(order[-1]), int(order[len(order) // 2]), 3})
    before, after, out_h, qkv_h = _run_layer(w, seed=1005, decode=True, with_qkv=True)
    _check_requests(oracle64, w.shape, w, b, before, after, out_h, sample, qkv_h)
    want, gate = oracle64.project_qkv(b.hidden, w.wqkv, w.shape.Nq, w.shape.Nkv, b.positions, b.query_start_loc,
                                      b.activation_offsets, b.adapter_ids, hp.oracle_adapters(w.adapters))
    hp.assert_close(qkv_h, want, 2e-2, "")
    assert gate.sum() > 0 and (gate == 0).sum() > 0


def test_config4_size_layer_one_request_and_cache_reuse_identity(oracle64):
    """One 8B-shape layer at the size of the 32-layer stack workload: 4 requests x (32768 cached + 1024 suffix
    tokens).  The base model's cache is made on the GPU by a base prefill of the prefix hidden states (131072
    tokens).  (i) The suffix prefill on that cache takes the long-batch attention route (whole items, then items
    cut into runs and merged) at head dim 128 and group size 4; every row of the last request, which holds the cut
    items, and of the first request is compared with the oracle, which is given the layer's own input and that
    request's cache rows read back from the pool.  (ii) The cache-reuse identity between two GPU runs at this
    size: a masked prefill of all 33792 tokens per request from scratch (gate closed before position 32768) must
    leave bit-identical K/V for the prefix positions and suffix outputs within the tolerance."""
    import torch
    shape = wl.SHAPE_8B
    R, P, S = 4, 32768, 1024
    rng = np.random.default_rng(4)
    wqkv = wl.make_wqkv(shape, rng)
    ads = [wl.make_adapter(shape, 32, rng)]
    b = wl.make_batch(shape, [P] * R, [S] * R, [0] * R, rng, shuffle_pages=True)
    w = wl.Workload("config4_layer", shape, wqkv, ads, b, 4)
    full_T = R * (P + S)
    g = hp.GpuLayers(shape, [dict(wqkv=wqkv)], [ads], full_T, R)
    try:
        gen = torch.Generator(device="cuda"); gen.manual_seed(44)
        # prefix hidden states drawn on the device (bf16-rounded N(0,1)); the suffix rows come from the workload
        hid_full = torch.randn((full_T, shape.hidden), generator=gen, device="cuda", dtype=torch.float32).to(torch.bfloat16)
        d = hp.DevBatch(b, "bf16")
        for r in range(R):
            hid_full[r * (P + S) + P:(r + 1) * (P + S)] = d.hidden[r * S:(r + 1) * S]
        pre_rows = torch.cat([torch.arange(r * (P + S), r * (P + S) + P, device="cuda") for r in range(R)])
        hid_pre = hid_full[pre_rows].contiguous()
        i32 = lambda a: hp.idev(np.ascontiguousarray(a, np.int32))   # noqa: E731
        pos_pre, qsl_pre = i32(np.tile(np.arange(P), R)), i32(np.arange(R + 1) * P)
        pos_full, qsl_full = i32(np.tile(np.arange(P + S), R)), i32(np.arange(R + 1) * (P + S))
        base_ids, len_pre = i32(np.full(R, -1)), i32(np.full(R, P))
        # run A: base prefill of the prefixes, then the aLoRA suffix prefill on that cache
        pool_a = g.new_pool(b.num_pages)
        scratch = g.empty(R * P, shape.Nq)
        ab.alora_full_lora_prefill_layer(g.ctx, 0, hid_pre, pos_pre, base_ids, qsl_pre, len_pre, pool_a, d.bt,
                                         d.max_blocks, b.num_pages, R * P, R, scratch)
        del scratch
        before = pool_a.clone()
        out_a = g.empty(b.T, shape.Nq)
        ab.alora_prefill_layer(g.ctx, 0, d.hidden, d.positions, d.a_req, d.ids, d.qsl, d.seq_lens, pool_a, d.bt,
                               d.max_blocks, b.num_pages, b.T, R, out_a)
        assert g.status() == 0
        out_a_h = hp.to_host(out_a)
        _check_requests(oracle64, shape, w, b, before, pool_a, out_a_h, [0, R - 1])
        # run B: every token new, gate closed before the activation offset
        pool_b = g.new_pool(b.num_pages)
        out_b = g.empty(full_T, shape.Nq)
        ab.alora_prefill_layer(g.ctx, 0, hid_full, pos_full, d.a_req, d.ids, qsl_full, d.seq_lens, pool_b, d.bt,
                               d.max_blocks, b.num_pages, full_T, R, out_b)
        assert g.status() == 0
        for r in range(R):
            Ka, Va = _request_kv(pool_a, b, r, P + S, shape)
            Kb, Vb = _request_kv(pool_b, b, r, P + S, shape)
            assert np.array_equal(Ka[:P].view(np.uint32), Kb[:P].view(np.uint32)), f"prefix K of request {r}"
            assert np.array_equal(Va[:P].view(np.uint32), Vb[:P].view(np.uint32)), f"prefix V of request {r}"
            hp.assert_close(Kb[P:], Ka[P:], 2e-2, f"suffix K of request {r}", block=shape.head_dim)
            hp.assert_close(Vb[P:], Va[P:], 2e-2, f"suffix V of request {r}", block=shape.head_dim)
            tail = hp.to_host(out_b[r * (P + S) + P:(r + 1) * (P + S)])
            hp.assert_close(tail, out_a_h[r * S:(r + 1) * S], 2e-2, f"suffix outputs of request {r}", block=shape.head_dim)
    finally:
        g.close()

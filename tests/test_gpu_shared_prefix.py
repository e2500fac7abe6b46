"""Several adapters on one reused base-model cache (the paper's regime of N adapters invoked on one conversation):
the grouping of decode-sized requests that share leading pages is integer work and compared exactly with a brute-force
restatement of the rule; the grouped attention is compared with the oracle, which knows nothing of groups (the
mathematics does not change); the shared pages stay bit-identical; the copy-on-write helper for a shared partial
tail page."""
import numpy as np
import pytest

from paper_2504_12397_b200 import binding as ab
from paper_2504_12397_b200 import workloads as wl

import helpers as hp

pytestmark = pytest.mark.gpu

SHAPE = wl.LayerShape(hidden=256, n_q_heads=8, n_kv_heads=2, head_dim=128, page_size=16, dtype="bf16")
MIN_SHARED = 256


def brute_force_groups(b: wl.Batch, page, G, small_max):
    """The grouping rule of include/alora.h written out: returns (group_first[R], shared_keys[R])."""
    R = b.R
    n_new = np.diff(b.query_start_loc)
    P = b.seq_lens - n_new
    common = np.zeros(R, np.int64)
    for r in range(1, R):
        if not (0 < n_new[r - 1] <= small_max and 0 < n_new[r] <= small_max):
            continue
        lim = min(P[r - 1] // page, P[r] // page, b.block_tables.shape[1])
        c = 0
        while c < lim and b.block_tables[r - 1, c] == b.block_tables[r, c]:
            c += 1
        common[r] = c * page
    first, shared = np.arange(R), np.zeros(R, np.int64)
    f = 0
    while f < R:
        e = f + 1
        if 0 < n_new[f] <= small_max:
            rows, mn = n_new[f] * G, None
            while e < R and 0 < n_new[e] <= small_max and common[e] >= MIN_SHARED and rows + n_new[e] * G <= 64:
                rows += n_new[e] * G
                mn = common[e] if mn is None else min(mn, common[e])
                e += 1
            s = (mn // 64) * 64 if e - f >= 2 else 0
            if s > 0:
                first[f:e] = f
                shared[f:e] = s
            else:
                e = f + 1
        f = e
    return first, shared


def _conversation_batch(rng, convs, per_conv, new_tokens, base_lens, own_extra, shape=None):
    """`convs` conversations; conversation c has base_lens[c] cached keys on pages of its own; per_conv[c] requests
    point their leading block-table entries at those pages (whole pages only), have own_extra[...] further cached
    keys on private pages, and new_tokens[...] new tokens."""
    shape = shape or SHAPE
    page = shape.page_size
    prefix, new, ids, owners = [], [], [], []
    k = 0
    for c in range(convs):
        for j in range(per_conv[c]):
            prefix.append(base_lens[c] // page * page + own_extra[k])
            new.append(new_tokens[k])
            ids.append((k % 3) - 1)
            owners.append(c)
            k += 1
    b = wl.make_batch(shape, prefix, new, ids, rng, shuffle_pages=True, spare_pages=convs * 300)
    # the conversations' own pages are taken from the spare pages at the end of the shuffled pool
    used = set(int(x) for r in range(b.R) for x in b.block_tables[r, :(b.seq_lens[r] + page - 1) // page])
    free = [p for p in range(b.num_pages) if p not in used]
    for c in range(convs):
        n = base_lens[c] // page
        pages = [free.pop() for _ in range(n)]
        for r in range(b.R):
            if owners[r] == c:
                b.block_tables[r, :n] = pages
    return b, owners


def _run(oracle64, b, check_groups=True, SHAPE=SHAPE):
    import torch
    rng = np.random.default_rng(5)
    wqkv = wl.make_wqkv(SHAPE, rng)
    ads = [wl.make_adapter(SHAPE, r, rng, scale=4.0) for r in (8, 32)]
    g = hp.GpuLayers(SHAPE, [dict(wqkv=wqkv)], [ads], max(b.T, 16), b.R)
    try:
        gen = torch.Generator(device="cuda"); gen.manual_seed(99)
        pool = torch.randn((b.num_pages, 2, SHAPE.n_kv_heads, SHAPE.page_size, SHAPE.head_dim), generator=gen,
                           device="cuda", dtype=torch.float32).to(torch.bfloat16)
        before = pool.clone()
        d = hp.DevBatch(b, "bf16")
        out = g.empty(b.T, SHAPE.Nq)
        ab.alora_prefill_layer(g.ctx, 0, d.hidden, d.positions, d.a_req, d.ids, d.qsl, d.seq_lens, pool, d.bt,
                               d.max_blocks, b.num_pages, b.T, b.R, out)
        gf = torch.full((b.R,), -7, dtype=torch.int32, device="cuda")
        gs = torch.full((b.R,), -7, dtype=torch.int32, device="cuda")
        ab.alora_prefix_groups(g.ctx, b.R, gf, gs)
        assert g.status() == 0
        first, shared = gf.cpu().numpy(), gs.cpu().numpy()
        if check_groups:
            want_first, want_shared = brute_force_groups(b, SHAPE.page_size, SHAPE.group, 16 // SHAPE.group)
            np.testing.assert_array_equal(first, want_first)
            np.testing.assert_array_equal(shared, want_shared)
        out_h = hp.to_host(out)
        pool_h_before, pool_h = hp.to_host(before), hp.to_host(pool)
        for r in range(b.R):
            P, L = int(b.prefix_lens[r]), int(b.seq_lens[r])
            K0, V0 = oracle64.paged_gather(pool_h_before, b.block_tables[r], P, SHAPE.n_kv_heads, SHAPE.page_size, SHAPE.head_dim)
            q0, q1 = int(b.query_start_loc[r]), int(b.query_start_loc[r + 1])
            sub = wl.Batch(positions=b.positions[q0:q1], query_start_loc=np.array([0, q1 - q0], np.int32),
                           seq_lens=b.seq_lens[r:r + 1], prefix_lens=b.prefix_lens[r:r + 1],
                           activation_offsets=b.activation_offsets[r:r + 1], adapter_ids=b.adapter_ids[r:r + 1],
                           block_tables=b.block_tables[r:r + 1], num_pages=b.num_pages, hidden=b.hidden[q0:q1])
            want = hp.oracle_block(oracle64, SHAPE, wqkv, ads, sub, [K0 if P else None], [V0 if P else None])
            hp.assert_close(out_h[q0:q1], want["out"], 2e-2, f"attention output of request {r}", block=SHAPE.head_dim)
            K1, _ = oracle64.paged_gather(pool_h, b.block_tables[r], L, SHAPE.n_kv_heads, SHAPE.page_size, SHAPE.head_dim)
            assert np.array_equal(K1[:P].view(np.uint32), K0.view(np.uint32))    # cached rows untouched, shared or not
        return first, shared
    finally:
        g.close()


def test_five_evaluators_per_conversation_decode_step(oracle64):
    """8 conversations x 5 adapters, one new token each, on 1000 .. 4400 shared keys plus 16 .. 40 keys of their own
    (their invocation and earlier generated tokens): every conversation becomes one group of 5."""
    rng = np.random.default_rng(1)
    convs = 8
    base = [int(x) for x in rng.integers(1000, 4400, convs)]
    own = [int(x) for x in rng.integers(16, 41, convs * 5)]
    b, owners = _conversation_batch(rng, convs, [5] * convs, [1] * (convs * 5), base, own)
    first, shared = _run(oracle64, b)
    assert all(first[r] == (r // 5) * 5 for r in range(b.R))
    assert all(shared[r] == (base[r // 5] // 16 * 16) // 64 * 64 for r in range(b.R))


def test_five_evaluators_per_conversation_at_the_8b_layer_shape(oracle64):
    """The decode step of the evaluator pipeline at full size: the 8B layer shape (8 KV heads, group size 4), 8
    conversations of 4100 .. 4400 cached tokens, each read by 5 requests (two adapters and the base model) with 16 .. 48
    cached tokens of their own and one new token.  Eight prefix groups of five (20 stacked score rows each); every
    request against the oracle, the grouping against the brute-force rule, the shared pages bit-identical."""
    rng = np.random.default_rng(24)
    shape = wl.SHAPE_8B
    convs = 8
    base = [int(x) for x in rng.integers(4100, 4401, convs)]
    n = convs * 5
    b, owners = _conversation_batch(rng, convs, [5] * convs, [1] * n, base, [int(x) for x in rng.integers(16, 49, n)],
                                    shape=shape)
    first, shared = _run(oracle64, b, SHAPE=shape)
    for c in range(convs):
        members = [r for r in range(b.R) if owners[r] == c]
        assert all(first[r] == members[0] for r in members)
        assert all(shared[r] == base[c] // shape.page_size * shape.page_size // 64 * 64 for r in members)


def test_mixed_groups_loners_and_long_requests(oracle64):
    """Groups of different sizes (2, 3, 16: a group of 17 requests is cut after 16 members), requests that share
    fewer than 256 keys (not grouped), a request with too many new tokens for the few-row route between two sharers
    (which splits them), members with 1 .. 4 new tokens (up to the 64 stacked rows), and an unshared request."""
    rng = np.random.default_rng(2)
    per_conv = [2, 3, 17, 2, 3, 1]
    base = [2048, 700, 3000, 200, 1500, 900]
    new = [1, 4,   2, 1, 3,   *([1] * 17),   1, 1,   4, 30, 4,   2]
    own = [int(x) for x in rng.integers(0, 50, sum(per_conv))]
    b, owners = _conversation_batch(rng, len(per_conv), per_conv, new, base, own)
    first, shared = _run(oracle64, b)
    assert shared[0] == 2048 and shared[2] == 640 and shared[5] == 2944 and shared[5 + 16] == 0
    assert shared[22] == 0 and shared[23] == 0          # 200 shared keys: below the minimum
    assert (shared[24:27] == 0).all()                   # the 30-token request in the middle is not on this route


def test_copy_on_write_of_a_shared_partial_tail_page(oracle64):
    """Three requests reuse 1000 cached positions (62 full pages and 8 rows of a 63rd).  Each gets a fresh page for
    block 62 through alora_cow_tail_pages: the 8 reused rows are copied, the table redirected, the shared page is
    not written by the layer call, and every request's result equals the oracle's on its own view of the cache."""
    import torch
    rng = np.random.default_rng(3)
    page, P = SHAPE.page_size, 1000
    b = wl.make_batch(SHAPE, [P] * 3, [1, 3, 2], [0, -1, 1], rng, shuffle_pages=True, spare_pages=8)
    nfull = P // page
    b.block_tables[1:, :nfull + 1] = b.block_tables[0, :nfull + 1]      # all three point at request 0's pages, tail page too
    assert ab.alora_validate_batch(ab.make_config(hidden=256, n_q_heads=8, n_kv_heads=2, head_dim=128, page_size=page,
                                                  max_tokens=16, max_requests=4, max_adapters=2),
                                   b.positions, b.activation_offsets, b.adapter_ids, b.query_start_loc, b.seq_lens,
                                   b.block_tables, b.num_pages) == 6     # two requests would write the same page
    used = set(int(x) for x in b.block_tables[:, :nfull + 1].ravel())
    spare = [p for p in range(b.num_pages) if p not in used and p not in set(int(x) for x in b.block_tables[:, nfull + 1:].ravel())]
    fresh = np.array([-1, spare[0], spare[1]], np.int32)                # request 0 keeps the original tail page
    wqkv = wl.make_wqkv(SHAPE, rng)
    ads = [wl.make_adapter(SHAPE, r, rng, scale=4.0) for r in (8, 32)]
    g = hp.GpuLayers(SHAPE, [dict(wqkv=wqkv)], [ads], 16, 4)
    try:
        gen = torch.Generator(device="cuda"); gen.manual_seed(7)
        pool = torch.randn((b.num_pages, 2, SHAPE.n_kv_heads, page, SHAPE.head_dim), generator=gen, device="cuda",
                           dtype=torch.float32).to(torch.bfloat16)
        before = hp.to_host(pool).copy()
        d = hp.DevBatch(b, "bf16")
        ab.alora_cow_tail_pages(g.ctx, d.qsl, d.seq_lens, d.bt, d.max_blocks, b.num_pages, b.R, hp.idev(fresh), pool)
        bt = d.bt.cpu().numpy()
        assert bt[1, nfull] == fresh[1] and bt[2, nfull] == fresh[2] and bt[0, nfull] == b.block_tables[0, nfull]
        assert ab.alora_validate_batch(g.cfg, b.positions, b.activation_offsets, b.adapter_ids, b.query_start_loc,
                                       b.seq_lens, bt, b.num_pages) == 0
        mid = hp.to_host(pool)
        shared_tail = int(b.block_tables[0, nfull])
        for r in (1, 2):
            assert np.array_equal(mid[fresh[r], :, :, :P % page, :], before[shared_tail, :, :, :P % page, :])
        out = g.empty(b.T, SHAPE.Nq)
        ab.alora_prefill_layer(g.ctx, 0, d.hidden, d.positions, d.a_req, d.ids, d.qsl, d.seq_lens, pool, d.bt,
                               d.max_blocks, b.num_pages, b.T, b.R, out)
        assert g.status() == 0
        after, out_h = hp.to_host(pool), hp.to_host(out)
        assert np.array_equal(after[shared_tail, :, :, :P % page, :], before[shared_tail, :, :, :P % page, :])
        b2 = wl.Batch(**{**b.__dict__, "block_tables": bt})
        for r in range(3):
            K0, V0 = oracle64.paged_gather(before, b.block_tables[0], P, SHAPE.n_kv_heads, page, SHAPE.head_dim)
            q0, q1 = int(b.query_start_loc[r]), int(b.query_start_loc[r + 1])
            sub = wl.Batch(positions=b.positions[q0:q1], query_start_loc=np.array([0, q1 - q0], np.int32),
                           seq_lens=b.seq_lens[r:r + 1], prefix_lens=b.prefix_lens[r:r + 1],
                           activation_offsets=b.activation_offsets[r:r + 1], adapter_ids=b.adapter_ids[r:r + 1],
                           block_tables=bt[r:r + 1], num_pages=b.num_pages, hidden=b.hidden[q0:q1])
            want = hp.oracle_block(oracle64, SHAPE, wqkv, ads, sub, [K0], [V0])
            hp.assert_close(out_h[q0:q1], want["out"], 2e-2, f"request {r}", block=SHAPE.head_dim)
            K1, _ = oracle64.paged_gather(after, bt[r], int(b.seq_lens[r]), SHAPE.n_kv_heads, page, SHAPE.head_dim)
            hp.assert_close(K1[P:], want["K"][0][P:], 2e-2, f"appended keys of request {r}", block=SHAPE.head_dim)
            assert np.array_equal(K1[:P].view(np.uint32), K0.view(np.uint32))
    finally:
        g.close()

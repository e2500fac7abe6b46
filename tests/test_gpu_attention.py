"""GPU parity of the attention step alone (alora_kv_append + alora_attend) against the CPU oracle, on
seeded random caches: short suffixes and decode rows (the few-row split-KV kernel), long suffixes (the
tensor-core kernel), both mixed in one batch, head dims / group sizes / page sizes the kernels are
built for, and a cache whose unused slots hold NaN (nothing outside a row's causal range may leak)."""
import numpy as np
import pytest

from paper_2504_12397_b200 import binding as ab
from paper_2504_12397_b200 import workloads as wl

import helpers as hp

pytestmark = pytest.mark.gpu


def _attend_case(oracle, shape, P, S, seed, nan_canaries=True, scale_q=1.0):
    """Random cache + random new q/k/v rows -> append + attend on the GPU, oracle on the same values."""
    import torch
    rng = np.random.default_rng(seed)
    b = wl.make_batch(shape, P, S, [-1] * len(P), rng, shuffle_pages=True, with_hidden=False)
    T, R = b.T, b.R
    pool_np = wl.random_kv_pool(shape, b.num_pages, rng)
    qkv_np = wl.bf16_round(rng.standard_normal((T, shape.N), dtype=np.float32))
    qkv_np[:, :shape.Nq] *= scale_q
    qkv_np = wl.bf16_round(qkv_np)
    if nan_canaries:
        # every slot that holds no cached position (tails of last pages, spare pages) is NaN
        keep = np.zeros((b.num_pages, shape.page_size), bool)
        for r in range(R):
            for p in range(int(b.prefix_lens[r])):
                keep[b.block_tables[r, p // shape.page_size], p % shape.page_size] = True
        mask = ~keep[:, None, None, :, None]
        pool_np = np.where(np.broadcast_to(mask, pool_np.shape), np.float32(np.nan), pool_np)
    g = hp.GpuLayers(shape, [dict(wqkv=np.zeros((shape.N, shape.hidden), np.float32))], [[]], max(T, 1), max(R, 1))
    try:
        pool = hp.to_dev(pool_np, "bf16")
        qkv = hp.to_dev(qkv_np, "bf16")
        d = hp.DevBatch(b, "bf16")
        out = torch.full((T, shape.Nq), float("nan"), dtype=torch.bfloat16, device="cuda")
        ab.alora_kv_append(g.ctx, qkv, d.positions, d.qsl, d.seq_lens, d.bt, d.max_blocks, b.num_pages, T, R, pool)
        ab.alora_attend(g.ctx, qkv, d.positions, d.qsl, d.seq_lens, pool, d.bt, d.max_blocks, b.num_pages, T, R, out)
        assert g.status() == 0
        got = hp.to_host(out)
    finally:
        g.close()
    # oracle: contiguous K/V per request = cached prefix (from the pool) ++ the new rows
    Ks, Vs, kvl = [], [], [0]
    clean = np.nan_to_num(pool_np, nan=0.0)
    for r in range(R):
        Pr = int(b.prefix_lens[r])
        K0, V0 = oracle.paged_gather(clean, b.block_tables[r], Pr, shape.n_kv_heads, shape.page_size, shape.head_dim)
        rows = slice(b.query_start_loc[r], b.query_start_loc[r + 1])
        Ks.append(np.concatenate([K0, qkv_np[rows, shape.Nq:shape.Nq + shape.Nkv]]))
        Vs.append(np.concatenate([V0, qkv_np[rows, shape.Nq + shape.Nkv:]]))
        kvl.append(kvl[-1] + len(Ks[-1]))
    want, _ = oracle.attention(qkv_np[:, :shape.Nq], np.concatenate(Ks), np.concatenate(Vs), kvl, b.positions,
                               b.query_start_loc, shape.n_q_heads, shape.n_kv_heads, shape.head_dim)
    assert np.isfinite(got).all(), "a value from outside a row's causal range reached an output"
    return hp.rel_err(got, want), got, want


SHAPE_G4 = wl.LayerShape(hidden=256, n_q_heads=8, n_kv_heads=2, head_dim=128, page_size=16, dtype="bf16")


def test_decode_rows_split_kv(oracle64):
    """One new token per request, contexts from 1 key to several key ranges (split-KV and its merge)."""
    P = [0, 1, 15, 16, 63, 64, 65, 255, 256, 257, 1000, 2049, 3333]
    err, _, _ = _attend_case(oracle64, SHAPE_G4, P, [1] * len(P), seed=101)
    assert err <= 2e-2


@pytest.mark.parametrize("S", [2, 3, 4, 5, 8, 13, 16])
def test_short_suffixes_split_kv(oracle64, S):
    """Suffixes of 2..16 tokens (16, 32 or 64 score rows per KV head) with range boundaries that fall
    between the positions of the block's tokens."""
    P = [0, 7, 250, 255, 256, 1021, 2500]
    err, _, _ = _attend_case(oracle64, SHAPE_G4, P, [S] * len(P), seed=200 + S)
    assert err <= 2e-2


def test_mixed_short_and_long_requests(oracle64):
    """Short requests (few-row kernel) and long ones (tensor-core kernel) in one call, ragged."""
    P = [300, 0, 1500, 64, 900, 10, 0]
    S = [1, 16, 17, 200, 4, 129, 1]
    err, got, want = _attend_case(oracle64, SHAPE_G4, P, S, seed=301)
    assert err <= 2e-2


def test_large_scores_do_not_overflow(oracle64):
    """Queries scaled up so that scores reach a few hundred: the running-maximum subtraction must hold."""
    err, _, _ = _attend_case(oracle64, SHAPE_G4, [700, 100, 2100], [1, 16, 3], seed=401, scale_q=24.0)
    assert err <= 2e-2


@pytest.mark.parametrize("hq,hkv,hd,page", [(4, 4, 128, 16), (4, 2, 64, 16), (16, 2, 128, 16), (8, 1, 64, 32),
                                            (4, 1, 128, 8), (8, 2, 128, 64), (8, 2, 128, 128)])
def test_shapes_group_sizes_and_page_sizes(oracle64, hq, hkv, hd, page):
    shape = wl.LayerShape(hidden=256, n_q_heads=hq, n_kv_heads=hkv, head_dim=hd, page_size=page, dtype="bf16")
    P = [0, 130, 777, 31, 1300]
    S = [1, 5, 16, 150, 2]
    err, _, _ = _attend_case(oracle64, shape, P, S, seed=500 + hq + hd + page)
    assert err <= 2e-2

"""The optional rotary position embedding on the GPU against the oracle: rotate-half on the new q and k rows
between projection and append, cached keys post-rotation (the paper's equations carry no rotation: this is a flag,
off by default)."""
import numpy as np
import pytest

from paper_2504_12397_b200 import binding as ab
from paper_2504_12397_b200 import workloads as wl

import helpers as hp

pytestmark = pytest.mark.gpu

THETA = 10000.0


def _run(oracle64, shape, w, ads, b, tol, max_tokens):
    """Base prefill of the prefixes (rotated keys cached), then the aLoRA suffix prefill; the same batch also through
    alora_project_qkv in aLoRA and in base mode.  Returns nothing; asserts."""
    import torch
    g = hp.GpuLayers(shape, [dict(wqkv=w)], [ads], max_tokens, max(b.R, 1), rope_theta=THETA)
    try:
        pool = g.new_pool(b.num_pages)
        pb = hp.prefix_only_batch(shape, b)
        if pb.T:
            dp = hp.DevBatch(pb, shape.dtype)
            ab.alora_full_lora_prefill_layer(g.ctx, 0, dp.hidden, dp.positions, dp.ids, dp.qsl, dp.seq_lens, pool, dp.bt,
                                             dp.max_blocks, b.num_pages, dp.T, dp.R, g.empty(pb.T, shape.Nq))
        d = hp.DevBatch(b, shape.dtype)
        out = g.empty(b.T, shape.Nq)
        ab.alora_prefill_layer(g.ctx, 0, d.hidden, d.positions, d.a_req, d.ids, d.qsl, d.seq_lens, pool, d.bt,
                               d.max_blocks, b.num_pages, d.T, d.R, out)
        qkv, base = g.empty(b.T, shape.N), g.empty(b.T, shape.N)
        ab.alora_project_qkv(g.ctx, 0, ab.MODE_ALORA, d.hidden, d.positions, d.a_req, d.ids, d.qsl, d.seq_lens, d.T, d.R, qkv)
        ab.alora_project_qkv(g.ctx, 0, ab.MODE_BASE, d.hidden, d.positions, d.a_req, d.ids, d.qsl, d.seq_lens, d.T, d.R, base)
        assert g.status() == 0
        Ks, Vs = hp.oracle_base_prefix(oracle64, shape, w, b, rope_theta=THETA)
        want = hp.oracle_block(oracle64, shape, w, ads, b, Ks, Vs, rope_theta=THETA)
        hd = shape.head_dim
        hp.assert_close(hp.to_host(qkv), want["qkv"], tol, "rotated q/k and v rows", block=hd)
        hp.assert_close(hp.to_host(out), want["out"], tol, "attention output", block=hd)
        got = [oracle64.paged_gather(hp.to_host(pool), b.block_tables[r], int(b.seq_lens[r]), shape.n_kv_heads,
                                     shape.page_size, hd) for r in range(b.R)]
        for r in range(b.R):
            hp.assert_close(got[r][0], want["K"][r], tol, f"cached (rotated) keys of request {r}", block=hd)
            hp.assert_close(got[r][1], want["V"][r], tol, f"cached values of request {r}", block=hd)
        # the rotation matters here: without it the keys are far off
        plain = hp.oracle_block(oracle64, shape, w, ads, b, Ks, Vs)
        assert hp.rel_err(plain["qkv"][:, :shape.Nq + shape.Nkv], want["qkv"][:, :shape.Nq + shape.Nkv]) > 0.2
        # Prop. 1 with the flag on: rows whose gate is closed equal the base call's rows bit for bit
        off = torch.from_numpy(want["gate"] == 0).cuda()
        assert int(off.sum()) > 0 and int((~off).sum()) > 0
        assert torch.equal(qkv[off], base[off])
    finally:
        g.close()


def test_rope_ragged_multi_adapter_bf16(oracle64):
    shape = wl.LayerShape(hidden=1024, n_q_heads=8, n_kv_heads=2, head_dim=128, page_size=16, dtype="bf16")
    rng = np.random.default_rng(61)
    w = wl.make_wqkv(shape, rng)
    ads = [wl.make_adapter(shape, r, rng, scale=s) for r, s in ((8, 1.0), (32, 2.0), (64, 0.5))]
    for a in ads:
        for n in ("Bq", "Bk", "Bv"):
            setattr(a, n, wl.bf16_round(getattr(a, n) * 8))
    P, S = [0, 37, 700, 129, 300], [150, 300, 1, 131, 17]
    ids, a_req = [2, 0, 1, -1, 2], [40, 37 + 130, 700, 0, 300]
    b = wl.make_batch(shape, P, S, ids, rng, activation_offsets=a_req, shuffle_pages=True, with_prefix_hidden=True)
    _run(oracle64, shape, w, ads, b, 2e-2, 2048)


def test_rope_few_rows_bf16(oracle64):
    """A decode-sized batch (the few-row projection route, the split-KV attention) with the flag on."""
    shape = wl.LayerShape(hidden=1024, n_q_heads=8, n_kv_heads=2, head_dim=128, page_size=16, dtype="bf16")
    rng = np.random.default_rng(62)
    w = wl.make_wqkv(shape, rng)
    ads = [wl.make_adapter(shape, r, rng, scale=4.0) for r in (16, 32)]
    R = 24
    P = [int(x) for x in rng.integers(10, 900, R)]
    ids = [(i % 3) - 1 for i in range(R)]
    a_req = [P[i] + (1 if i % 4 == 2 else 0) for i in range(R)]
    b = wl.make_batch(shape, P, [1] * R, ids, rng, activation_offsets=a_req, shuffle_pages=True, with_prefix_hidden=True)
    _run(oracle64, shape, w, ads, b, 2e-2, 24 * 900)


def test_rope_tiny_fp32(oracle64):
    w = wl.config1()
    b = w.batch
    b2 = wl.Batch(**{**b.__dict__, "activation_offsets": np.array([70], np.int32)})   # the gate opens 6 tokens in
    _run(oracle64, w.shape, w.wqkv, w.adapters, b2, 1e-5, 128)


def test_rope_config2_sampled_requests(oracle64):
    """The bench workload's shape with the flag on: 8 x (4096 cached + 256 suffix) at the 8B layer shape, cached keys
    a seeded fill of the pool (they stand for already-rotated keys); requests 0 and 5 in full."""
    import torch
    w = wl.config2(seed=2)
    shape, b = w.shape, w.batch
    g = hp.GpuLayers(shape, [dict(wqkv=w.wqkv)], [w.adapters], b.T, b.R, rope_theta=THETA)
    try:
        gen = torch.Generator(device="cuda"); gen.manual_seed(77)
        pool = torch.randn((b.num_pages, 2, shape.n_kv_heads, shape.page_size, shape.head_dim), generator=gen,
                           device="cuda", dtype=torch.float32).to(torch.bfloat16)
        before = pool.clone()
        d = hp.DevBatch(b, "bf16")
        out = g.empty(b.T, shape.Nq)
        ab.alora_prefill_layer(g.ctx, 0, d.hidden, d.positions, d.a_req, d.ids, d.qsl, d.seq_lens, pool, d.bt,
                               d.max_blocks, b.num_pages, b.T, b.R, out)
        assert g.status() == 0
        out_h = hp.to_host(out)
        for r in (0, 5):
            P = int(b.prefix_lens[r])
            nblk = (int(b.seq_lens[r]) + shape.page_size - 1) // shape.page_size
            pages = torch.from_numpy(b.block_tables[r, :nblk].astype(np.int64)).cuda()

            def kv(pl, length):
                blk = pl[pages].to(torch.float32).cpu().numpy()
                x = blk.transpose(1, 0, 3, 2, 4).reshape(2, nblk * shape.page_size, shape.Nkv)
                return x[0, :length], x[1, :length]
            K0, V0 = kv(before, P)
            q0, q1 = int(b.query_start_loc[r]), int(b.query_start_loc[r + 1])
            sub = wl.Batch(positions=b.positions[q0:q1], query_start_loc=np.array([0, q1 - q0], np.int32),
                           seq_lens=b.seq_lens[r:r + 1], prefix_lens=b.prefix_lens[r:r + 1],
                           activation_offsets=b.activation_offsets[r:r + 1], adapter_ids=b.adapter_ids[r:r + 1],
                           block_tables=b.block_tables[r:r + 1], num_pages=b.num_pages, hidden=b.hidden[q0:q1])
            want = hp.oracle_block(oracle64, shape, w.wqkv, w.adapters, sub, [K0], [V0], rope_theta=THETA)
            hp.assert_close(out_h[q0:q1], want["out"], 2e-2, f"attention output of request {r}", block=shape.head_dim)
            K1, V1 = kv(pool, int(b.seq_lens[r]))
            hp.assert_close(K1[P:], want["K"][0][P:], 2e-2, f"appended rotated keys of request {r}", block=shape.head_dim)
            assert np.array_equal(K1[:P].view(np.uint32), K0.view(np.uint32))
    finally:
        g.close()

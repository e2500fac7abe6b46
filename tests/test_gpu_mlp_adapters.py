"""GPU parity of gated adapters on the MLP block (gate, up and down projections adapted under the same per-token gate
as q/k/v, Eq. 5's form per matrix): the decoder stack through the C ABI against the CPU oracle."""
import numpy as np
import pytest

from paper_2504_12397_b200 import binding as ab
from paper_2504_12397_b200 import workloads as wl

import helpers as hp

pytestmark = pytest.mark.gpu

SHAPE = wl.LayerShape(hidden=512, n_q_heads=4, n_kv_heads=2, head_dim=128, page_size=16, dtype="bf16",
                      intermediate=1024)


def _weights(rng, n_layers, ranks=(16, 8), mlp_ranks=(16, 32), mlp_scales=(1.0, 0.5), boost=8):
    layers = [wl.make_stack_weights(SHAPE, rng) for _ in range(n_layers)]
    ads = [[wl.make_adapter(SHAPE, r, rng) for r in ranks] for _ in range(n_layers)]
    mlps = [[wl.make_mlp_adapter(SHAPE, r, rng, scale=s) for r, s in zip(mlp_ranks, mlp_scales)] for _ in range(n_layers)]
    for per in ads:       # deltas well above the bf16 rounding noise, so that a wrong or missing one is visible
        for a in per:
            for n in ("Bq", "Bk", "Bv"):
                setattr(a, n, wl.bf16_round(getattr(a, n) * boost))
    for per in mlps:
        for a in per:
            for n in ("Bg", "Bu", "Bd"):
                setattr(a, n, wl.bf16_round(getattr(a, n) * boost))
    return layers, ads, mlps


def _oracle_stack(orc, layers, ads, mlps, b, with_mlp=True, force_all=False):
    x = b.hidden.astype(np.float64)
    blks = []
    for l in range(len(layers)):
        x, blk = orc.decoder_layer(x, layers[l], SHAPE.Nq, SHAPE.Nkv, SHAPE.n_q_heads, SHAPE.n_kv_heads,
                                   SHAPE.head_dim, 1e-5, b.positions, b.query_start_loc, b.activation_offsets,
                                   b.adapter_ids, hp.oracle_adapters(ads[l]), [None] * b.R, [None] * b.R,
                                   force_all=force_all,
                                   mlp_adapters=hp.oracle_mlp_adapters(mlps[l]) if with_mlp else None)
        blks.append(blk)
    return x, blks


def _run_stack(g, b, mode=ab.MODE_ALORA):
    d = hp.DevBatch(b, SHAPE.dtype)
    pools = [g.new_pool(b.num_pages) for _ in range(g.n_layers)]
    hout = g.empty(b.T, SHAPE.hidden)
    ab.alora_forward_stack(g.ctx, mode, d.hidden, d.positions, d.a_req, d.ids, d.qsl, d.seq_lens, pools, d.bt,
                           d.max_blocks, b.num_pages, d.T, d.R, hout)
    assert g.status() == 0
    return hp.to_host(hout), pools


def test_two_layer_stack_with_mlp_adapters(oracle64):
    """Two decoder layers, four requests on two adapters (ranks 16 / 8 on q/k/v, 16 / 32 with scales 1 / 0.5 on the
    MLP) and the base model; one gate opens in the middle of its request's new tokens, and the 64-row tiles of the
    expand step hold rows of several requests.  Hidden states out of the stack and both layers' caches against the
    oracle; the oracle WITHOUT the MLP adapters is far outside the tolerance, so the comparison sees them."""
    rng = np.random.default_rng(41)
    layers, ads, mlps = _weights(rng, 2)
    S, ids, a_req = [70, 33, 20, 45], [0, -1, 1, 0], [41, 0, 0, 0]
    b = wl.make_batch(SHAPE, [0] * 4, S, ids, rng, activation_offsets=a_req, shuffle_pages=True)
    g = hp.GpuLayers(SHAPE, layers, ads, 512, 8, mlp_adapters_per_layer=mlps)
    try:
        got, pools = _run_stack(g, b)
        want, blks = _oracle_stack(oracle64, layers, ads, mlps, b)
        hp.assert_close(got, want, 2e-2, "stack output with MLP adapters", block=SHAPE.head_dim)
        for l in range(2):
            kv = [oracle64.paged_gather(hp.to_host(pools[l]), b.block_tables[r], int(b.seq_lens[r]), SHAPE.n_kv_heads,
                                        SHAPE.page_size, SHAPE.head_dim) for r in range(b.R)]
            for r in range(b.R):
                hp.assert_close(kv[r][0], blks[l]["K"][r], 2e-2, f"layer {l} keys of request {r}", block=SHAPE.head_dim)
                hp.assert_close(kv[r][1], blks[l]["V"][r], 2e-2, f"layer {l} values of request {r}", block=SHAPE.head_dim)
        plain, _ = _oracle_stack(oracle64, layers, ads, mlps, b, with_mlp=False)
        open_rows = np.concatenate([np.arange(41, 70), np.arange(103, 123), np.arange(123, 168)])
        assert hp.rel_err(got[open_rows], plain[open_rows]) > 0.1
    finally:
        g.close()


def test_closed_gate_rows_keep_the_bits_of_the_base_mlp(oracle64):
    """One layer: the rows before the activation offset, and the rows of a base-model request, come out of the stack
    with exactly the bits of an ALORA_MODE_BASE call on the same inputs (the expand step neither reads nor writes
    them); the open rows differ."""
    rng = np.random.default_rng(42)
    layers, ads, mlps = _weights(rng, 1)
    S, ids, a_req = [90, 50, 40], [0, -1, 1], [37, 0, 40]          # request 2's gate never opens
    b = wl.make_batch(SHAPE, [0] * 3, S, ids, rng, activation_offsets=a_req, shuffle_pages=True)
    g = hp.GpuLayers(SHAPE, layers, ads, 512, 8, mlp_adapters_per_layer=mlps)
    try:
        got, _ = _run_stack(g, b)
        base, _ = _run_stack(g, b, mode=ab.MODE_BASE)
        closed = np.concatenate([np.arange(0, 37), np.arange(90, 180)])
        assert np.array_equal(got[closed].view(np.uint32), base[closed].view(np.uint32))
        assert hp.rel_err(got[37:90], base[37:90]) > 0.05
        want, _ = _oracle_stack(oracle64, layers, ads, mlps, b)
        hp.assert_close(got, want, 2e-2, "one layer with MLP adapters", block=SHAPE.head_dim)
    finally:
        g.close()


def test_full_lora_mode_opens_the_mlp_gate_everywhere(oracle64):
    """The recompute path (Eq. 4): every row of an adapter request is adapted, in the MLP too."""
    rng = np.random.default_rng(43)
    layers, ads, mlps = _weights(rng, 1)
    b = wl.make_batch(SHAPE, [0, 0], [80, 30], [1, -1], rng, activation_offsets=[60, 0], shuffle_pages=True)
    g = hp.GpuLayers(SHAPE, layers, ads, 256, 4, mlp_adapters_per_layer=mlps)
    try:
        got, _ = _run_stack(g, b, mode=ab.MODE_FULL_LORA)
        want, _ = _oracle_stack(oracle64, layers, ads, mlps, b, force_all=True)
        hp.assert_close(got, want, 2e-2, "full-LoRA stack with MLP adapters", block=SHAPE.head_dim)
    finally:
        g.close()


def test_decode_steps_with_mlp_adapters_match_the_prefill_rows(oracle64):
    """Two layers: a prefill of all but the last two tokens, then two decode steps through alora_decode_stack (few
    rows: the shrink runs on the weight-streaming GEMM pair); the produced rows equal the oracle's rows of the whole
    sequences.  Adapter 1 has no MLP part on layer 1: its rows there get the q/k/v deltas only."""
    rng = np.random.default_rng(44)
    layers, ads, mlps = _weights(rng, 2)
    mlps[1][1] = None
    L, ids, a_req, n_dec = [40, 23, 64, 31], [0, 1, -1, 1], [10, 22, 0, 0], 2
    full = wl.make_batch(SHAPE, [0] * len(L), L, ids, rng, activation_offsets=a_req, shuffle_pages=True)
    R = full.R
    g = hp.GpuLayers(SHAPE, layers, ads, 256, 8, mlp_adapters_per_layer=mlps)
    try:
        pools = [g.new_pool(full.num_pages) for _ in range(2)]
        keep = np.concatenate([np.arange(full.query_start_loc[r], full.query_start_loc[r + 1] - n_dec) for r in range(R)])
        pre = wl.Batch(positions=full.positions[keep],
                       query_start_loc=np.concatenate([[0], np.cumsum(np.array(L) - n_dec)]).astype(np.int32),
                       seq_lens=(np.array(L) - n_dec).astype(np.int32), prefix_lens=np.zeros(R, np.int32),
                       activation_offsets=full.activation_offsets, adapter_ids=full.adapter_ids,
                       block_tables=full.block_tables, num_pages=full.num_pages, hidden=full.hidden[keep])
        d = hp.DevBatch(pre, SHAPE.dtype)
        hout = g.empty(pre.T, SHAPE.hidden)
        ab.alora_forward_stack(g.ctx, ab.MODE_ALORA, d.hidden, d.positions, d.a_req, d.ids, d.qsl, d.seq_lens, pools,
                               d.bt, d.max_blocks, full.num_pages, d.T, d.R, hout)
        got = np.zeros((R, n_dec, SHAPE.hidden), np.float32)
        for i in range(n_dec):
            rows = full.query_start_loc[1:] - n_dec + i
            pos = full.positions[rows]
            o = g.empty(R, SHAPE.hidden)
            ab.alora_decode_stack(g.ctx, hp.to_dev(full.hidden[rows], "bf16"), hp.idev(pos), d.a_req, d.ids,
                                  hp.idev(pos + 1), pools, d.bt, d.max_blocks, full.num_pages, R, o)
            got[:, i] = hp.to_host(o)
        assert g.status() == 0
        # the oracle's adapter 1 on layer 1 has a zero MLP part
        zero = wl.make_mlp_adapter(SHAPE, 8, np.random.default_rng(0), zero_b=True)
        o_mlps = [mlps[0], [mlps[1][0], zero]]
        want, _ = _oracle_stack(oracle64, layers, ads, o_mlps, full)
        for i in range(n_dec):
            rows = full.query_start_loc[1:] - n_dec + i
            hp.assert_close(got[:, i], want[rows], 2e-2, f"decode step {i} with MLP adapters", block=SHAPE.head_dim)
        hp.assert_close(hp.to_host(hout), want[keep], 2e-2, "prefilled rows", block=SHAPE.head_dim)
    finally:
        g.close()


def test_mlp_adapters_across_token_chunks_of_the_mlp(oracle64):
    """A batch longer than one MLP pass of the stack entry (8192 tokens): 18 requests of 470 tokens on two adapters
    and the base model, one layer; the rows around the pass boundary and a sample of the others against the oracle."""
    rng = np.random.default_rng(45)
    layers, ads, mlps = _weights(rng, 1)
    R, S = 18, 470
    ids = [(r % 3) - 1 for r in range(R)]
    a_req = [0 if r % 2 else 200 for r in range(R)]
    b = wl.make_batch(SHAPE, [0] * R, [S] * R, ids, rng, activation_offsets=a_req, shuffle_pages=True)
    assert b.T > 8192
    g = hp.GpuLayers(SHAPE, layers, ads, b.T, R, mlp_adapters_per_layer=mlps)
    try:
        got, _ = _run_stack(g, b)
        want, _ = _oracle_stack(oracle64, layers, ads, mlps, b)
        r_b = 8192 // S                                    # the request that holds row 8192
        rows = np.unique(np.concatenate([np.arange(r_b * S, (r_b + 1) * S), np.arange(0, 300), np.arange(b.T - 300, b.T),
                                         rng.choice(b.T, 600, replace=False)]))
        hp.assert_close(got[rows], want[rows], 2e-2, "rows around the MLP pass boundary", block=SHAPE.head_dim)
    finally:
        g.close()


def test_one_layer_at_the_8b_shape(oracle64):
    """One decoder layer at the 8B layer shape (hidden 4096, intermediate 14336: gate / up rows of 57 KB, a down
    projection with K = 14336) with adapters on q/k/v and on the MLP: three requests (rank 32 and rank 8 adapters and
    the base model), 160 new tokens, one gate opening inside its chunk; every row against the oracle, closed rows
    bit-equal to the base-mode call."""
    shape = wl.SHAPE_8B
    rng = np.random.default_rng(47)
    layers = [wl.make_stack_weights(shape, rng)]
    ads = [[wl.make_adapter(shape, r, rng) for r in (32, 8)]]
    mlps = [[wl.make_mlp_adapter(shape, r, rng, scale=s) for r, s in ((32, 1.0), (8, 2.0))]]
    for a in ads[0]:
        for n in ("Bq", "Bk", "Bv"):
            setattr(a, n, wl.bf16_round(getattr(a, n) * 8))
    for a in mlps[0]:
        for n in ("Bg", "Bu", "Bd"):
            setattr(a, n, wl.bf16_round(getattr(a, n) * 8))
    S, ids, a_req = [70, 50, 40], [0, -1, 1], [33, 0, 0]
    b = wl.make_batch(shape, [0] * 3, S, ids, rng, activation_offsets=a_req, shuffle_pages=True)
    g = hp.GpuLayers(shape, layers, ads, 256, 4, mlp_adapters_per_layer=mlps)
    try:
        d = hp.DevBatch(b, shape.dtype)

        def run(mode):
            pools = [g.new_pool(b.num_pages)]
            hout = g.empty(b.T, shape.hidden)
            ab.alora_forward_stack(g.ctx, mode, d.hidden, d.positions, d.a_req, d.ids, d.qsl, d.seq_lens, pools, d.bt,
                                   d.max_blocks, b.num_pages, d.T, d.R, hout)
            assert g.status() == 0
            return hp.to_host(hout)

        got, base = run(ab.MODE_ALORA), run(ab.MODE_BASE)
        x, _ = oracle64.decoder_layer(b.hidden.astype(np.float64), layers[0], shape.Nq, shape.Nkv, shape.n_q_heads,
                                      shape.n_kv_heads, shape.head_dim, 1e-5, b.positions, b.query_start_loc,
                                      b.activation_offsets, b.adapter_ids, hp.oracle_adapters(ads[0]), [None] * 3,
                                      [None] * 3, mlp_adapters=hp.oracle_mlp_adapters(mlps[0]))
        hp.assert_close(got, x, 2e-2, "8B-shape layer with MLP adapters", block=shape.head_dim)
        closed = np.concatenate([np.arange(0, 33), np.arange(70, 120)])
        assert np.array_equal(got[closed].view(np.uint32), base[closed].view(np.uint32))
        opened = np.concatenate([np.arange(33, 70), np.arange(120, 160)])
        assert hp.rel_err(got[opened], base[opened]) > 0.02
    finally:
        g.close()


def test_registering_again_replaces_the_mlp_part(oracle64):
    """Registering an adapter's MLP part a second time replaces it: with a smaller rank (the padding of the first
    registration must not leak) and then with B = 0 (the stack then equals the one with q/k/v adapters only)."""
    rng = np.random.default_rng(49)
    layers, ads, mlps = _weights(rng, 1, mlp_ranks=(32, 16))
    b = wl.make_batch(SHAPE, [0, 0], [75, 30], [0, 1], rng, activation_offsets=[20, 0], shuffle_pages=True)
    g = hp.GpuLayers(SHAPE, layers, ads, 256, 4, mlp_adapters_per_layer=mlps)
    try:
        def register(i, m):
            mats = [hp.to_dev(getattr(m, n), "bf16") for n in ("Ag", "Bg", "Au", "Bu", "Ad", "Bd")]
            ab.alora_register_mlp_adapter(g.ctx, i, 0, m.rank, m.scale, *mats)
            return mats
        small = wl.make_mlp_adapter(SHAPE, 8, rng, scale=2.0)
        for n in ("Bg", "Bu", "Bd"):
            setattr(small, n, wl.bf16_round(getattr(small, n) * 8))
        keep = register(0, small)
        got, _ = _run_stack(g, b)
        want, _ = _oracle_stack(oracle64, layers, ads, [[small, mlps[0][1]]], b)
        hp.assert_close(got, want, 2e-2, "after replacing adapter 0's MLP part by a rank-8 one", block=SHAPE.head_dim)
        zero = wl.make_mlp_adapter(SHAPE, 16, rng, zero_b=True)
        keep += register(0, zero) + register(1, zero)
        got, _ = _run_stack(g, b)
        want, _ = _oracle_stack(oracle64, layers, ads, mlps, b, with_mlp=False)
        hp.assert_close(got, want, 2e-2, "after replacing both MLP parts by B = 0", block=SHAPE.head_dim)
    finally:
        g.close()


def test_mlp_adapter_registration_errors():
    rng = np.random.default_rng(46)
    layers, ads, mlps = _weights(rng, 1)
    g = hp.GpuLayers(SHAPE, layers, [[ads[0][0]]], 64, 2, n_adapters=2)
    try:
        m = mlps[0][0]
        mats = [hp.to_dev(getattr(m, n), "bf16") for n in ("Ag", "Bg", "Au", "Bu", "Ad", "Bd")]
        lib = ab.load_library()

        def reg(ctx, adapter_id, layer, rank):
            return lib.alora_register_mlp_adapter(ctx, adapter_id, layer, rank, 1.0, *[x.data_ptr() for x in mats], None)

        # status codes of include/alora.h: 1 invalid argument, 3 capacity, 4 no weights
        assert reg(g.ctx, 1, 0, m.rank) == 4       # adapter 1 has no q/k/v part on this layer
        assert reg(g.ctx, 2, 0, m.rank) == 3         # id beyond max_adapters
        assert reg(g.ctx, 0, 1, m.rank) == 1      # no such layer
        assert reg(g.ctx, 0, 0, 4096) == 3           # rank beyond max_rank
        assert reg(g.ctx, 0, 0, m.rank) == 0
    finally:
        g.close()

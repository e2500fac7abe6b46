"""Pins for the CPU oracle: each check ties it to something other than itself.

What fixes the values: the paper's identities (Prop. 1: rows before activation are the base
model's, cache reuse; Eq. 5 with a zero delta; Eq. 4 as a merged dense weight; Prop. 2's counts),
library routines used as references only inside this file (numpy matmul, torch
scaled_dot_product_attention), closed forms (one key, uniform scores, two-key logistic weight,
constant V), brute force in pure Python on tiny inputs, and a hand-computed example
(tests/golden/eq5_hand_example.txt).
"""
import os

import numpy as np
import pytest
import torch

from oracle import Adapter, MlpAdapter
from paper_2504_12397_b200 import workloads as wl

SMALL = wl.LayerShape(hidden=32, n_q_heads=4, n_kv_heads=2, head_dim=8, page_size=4, dtype="fp32")


def _ad(a: wl.AdapterWeights) -> Adapter:
    return Adapter(a.rank, a.scale, a.Aq, a.Bq, a.Ak, a.Bk, a.Av, a.Bv)


def _setup(seed=0, prefix=(7, 12), new=(5, 3), ids=(0, 1), ranks=(3, 5), a_req=None, scale=(1.0, 0.5)):
    rng = np.random.default_rng(seed)
    W = wl.make_wqkv(SMALL, rng) * 10
    ads = [wl.make_adapter(SMALL, r, rng, scale=s) for r, s in zip(ranks, scale)]
    for a in ads:  # make the delta comparable to the base term so a dropped term is visible
        for n in ("Aq", "Bq", "Ak", "Bk", "Av", "Bv"):
            setattr(a, n, getattr(a, n) * 20)
    b = wl.make_batch(SMALL, prefix, new, ids, rng, activation_offsets=a_req, shuffle_pages=True,
                      with_prefix_hidden=True)
    return W, ads, b


def _full_sequence_batch(b: wl.Batch, rng):
    """The same requests presented as one uncached sequence each (prefix hidden ++ new hidden)."""
    xs, pos, qsl = [], [], [0]
    for r in range(b.R):
        lo, hi = b.query_start_loc[r], b.query_start_loc[r + 1]
        xs.append(np.concatenate([b.prefix_hidden[r], b.hidden[lo:hi]]))
        pos.append(np.arange(b.seq_lens[r], dtype=np.int32))
        qsl.append(qsl[-1] + int(b.seq_lens[r]))
    return np.concatenate(xs), np.concatenate(pos), np.asarray(qsl, np.int32)


# ---- projection -----------------------------------------------------------------------------------

def test_projection_matches_library_matmul(oracle64):
    """Eq. 5 against numpy: y = x W^T + gate * s * (x A^T) B^T per block, gate = [p >= a_req]."""
    W, ads, b = _setup(a_req=(9, 12))  # request 0 activates two tokens into its new chunk
    qkv, gate = oracle64.project_qkv(b.hidden, W, SMALL.Nq, SMALL.Nkv, b.positions, b.query_start_loc,
                                     b.activation_offsets, b.adapter_ids, [_ad(a) for a in ads])
    x = b.hidden.astype(np.float64)
    ref = x @ W.astype(np.float64).T
    exp_gate = np.zeros(b.T, np.uint8)
    for r in range(b.R):
        a = ads[b.adapter_ids[r]]
        for t in range(b.query_start_loc[r], b.query_start_loc[r + 1]):
            if b.positions[t] >= b.activation_offsets[r]:
                exp_gate[t] = 1
                d = np.concatenate([(a.Bq.astype(np.float64) @ (a.Aq.astype(np.float64) @ x[t])),
                                    (a.Bk.astype(np.float64) @ (a.Ak.astype(np.float64) @ x[t])),
                                    (a.Bv.astype(np.float64) @ (a.Av.astype(np.float64) @ x[t]))])
                ref[t] += a.scale * d
    assert np.array_equal(gate, exp_gate)
    assert gate.sum() == 3 + 3 and gate[0] == 0 and gate[1] == 0 and gate[2] == 1
    np.testing.assert_allclose(qkv, ref, rtol=1e-12, atol=1e-13)
    # the delta is not negligible in this fixture: dropping it would be seen
    assert np.abs(qkv - x @ W.astype(np.float64).T).max() > 1e-2


def test_hand_example_eq5(oracle64):
    """A 2-dimensional example worked by hand from Eq. 5 (tests/golden/eq5_hand_example.txt)."""
    path = os.path.join(os.path.dirname(__file__), "golden", "eq5_hand_example.txt")
    vals = {}
    for line in open(path):
        line = line.split("#")[0].strip()
        if not line:
            continue
        k, v = line.split("=")
        vals[k.strip()] = np.array([float(z) for z in v.split()], np.float64)
    H, Nq, Nkv = 2, 2, 1
    W = vals["W"].reshape(4, 2).astype(np.float32)
    ad = Adapter(1, float(vals["scale"][0]), vals["Aq"].reshape(1, 2), vals["Bq"].reshape(2, 1),
                 vals["Ak"].reshape(1, 2), vals["Bk"].reshape(1, 1), vals["Av"].reshape(1, 2),
                 vals["Bv"].reshape(1, 1))
    x = vals["x"].reshape(3, 2)
    qkv, gate = oracle64.project_qkv(x, W, Nq, Nkv, [0, 1, 2], [0, 3], [1], [0], [ad])
    np.testing.assert_array_equal(gate, [0, 1, 1])
    np.testing.assert_allclose(qkv, vals["qkv"].reshape(3, 4), rtol=0, atol=1e-12)
    out, pairs = oracle64.attention(qkv[:, :2], qkv[:, 2:3], qkv[:, 3:4], [0, 3], [0, 1, 2], [0, 3],
                                    Hq=2, Hkv=1, hd=1, softmax_scale=1.0)
    assert pairs == 6
    np.testing.assert_allclose(out, vals["attn"].reshape(3, 2), rtol=0, atol=1e-9)


def test_prop1_rows_before_activation_are_bit_equal_to_base(oracle64, oracle32):
    """Prop. 1: for p < a_req the adapter model's q/k/v rows are the base model's, bit for bit."""
    for orc in (oracle64, oracle32):
        for a_req in [(0, 0), (9, 13), (7, 12), (100, 100)]:
            W, ads, b = _setup(a_req=a_req)
            A = [_ad(a) for a in ads]
            qkv, gate = orc.project_qkv(b.hidden, W, SMALL.Nq, SMALL.Nkv, b.positions,
                                        b.query_start_loc, b.activation_offsets, b.adapter_ids, A)
            base, g0 = orc.project_qkv(b.hidden, W, SMALL.Nq, SMALL.Nkv, b.positions,
                                       b.query_start_loc, b.activation_offsets, [-1] * b.R, A)
            assert g0.sum() == 0
            off = gate == 0
            assert np.array_equal(qkv[off].view(np.uint64), base[off].view(np.uint64))
            if (~off).any():
                assert np.abs(qkv[~off] - base[~off]).min(axis=1).max() > 0
            exp = np.concatenate([b.positions[b.query_start_loc[r]:b.query_start_loc[r + 1]] >= a_req[r]
                                  for r in range(b.R)])
            assert np.array_equal(gate.astype(bool), exp)


def test_zero_B_reproduces_base(oracle64):
    """Eq. 5 with Delta = 0 (B = 0): every output equals the base model's."""
    W, ads, b = _setup(a_req=(0, 0))
    for a in ads:
        a.Bq[:] = 0; a.Bk[:] = 0; a.Bv[:] = 0
    A = [_ad(a) for a in ads]
    P = [None] * b.R
    kw = dict(Nq=SMALL.Nq, Nkv=SMALL.Nkv, Hq=4, Hkv=2, hd=8)
    xs, pos, qsl = _full_sequence_batch(b, None)
    on = oracle64.attention_block(xs, W, positions=pos, query_start_loc=qsl, activation_offsets=[0, 0],
                                  adapter_ids=b.adapter_ids, adapters=A, prefix_K=P, prefix_V=P, **kw)
    off = oracle64.attention_block(xs, W, positions=pos, query_start_loc=qsl, activation_offsets=[0, 0],
                                   adapter_ids=[-1, -1], adapters=A, prefix_K=P, prefix_V=P, **kw)
    assert on["gate"].all() and not off["gate"].any()
    np.testing.assert_array_equal(on["qkv"], off["qkv"])
    np.testing.assert_array_equal(on["out"], off["out"])


def test_full_activation_is_merged_weight_lora(oracle64):
    """Eq. 4: a_req = 0 (or force_all) equals a dense projection with W + s B A, built with numpy."""
    W, ads, b = _setup(ids=(1, 1), a_req=(0, 0))
    a = ads[1]
    merged = W.astype(np.float64).copy()
    merged[:SMALL.Nq] += a.scale * a.Bq.astype(np.float64) @ a.Aq.astype(np.float64)
    merged[SMALL.Nq:SMALL.Nq + SMALL.Nkv] += a.scale * a.Bk.astype(np.float64) @ a.Ak.astype(np.float64)
    merged[SMALL.Nq + SMALL.Nkv:] += a.scale * a.Bv.astype(np.float64) @ a.Av.astype(np.float64)
    ref = b.hidden.astype(np.float64) @ merged.T
    A = [_ad(x) for x in ads]
    q1, _ = oracle64.project_qkv(b.hidden, W, SMALL.Nq, SMALL.Nkv, b.positions, b.query_start_loc,
                                 b.activation_offsets, b.adapter_ids, A)
    q2, _ = oracle64.project_qkv(b.hidden, W, SMALL.Nq, SMALL.Nkv, b.positions, b.query_start_loc,
                                 [50, 50], b.adapter_ids, A, force_all=True)
    np.testing.assert_allclose(q1, ref, rtol=1e-11, atol=1e-12)
    np.testing.assert_array_equal(q1, q2)


# ---- attention --------------------------------------------------------------------------------------

def _sdpa_reference(q, K, V, positions, Hq, Hkv, hd, scale):
    """torch's library attention with an explicit boolean mask, one request."""
    G = Hq // Hkv
    T, L = q.shape[0], K.shape[0]
    qt = torch.from_numpy(q.reshape(T, Hq, hd)).permute(1, 0, 2)[None]
    kt = torch.from_numpy(K.reshape(L, Hkv, hd)).permute(1, 0, 2).repeat_interleave(G, dim=0)[None]
    vt = torch.from_numpy(V.reshape(L, Hkv, hd)).permute(1, 0, 2).repeat_interleave(G, dim=0)[None]
    mask = torch.from_numpy(np.arange(L)[None, :] <= np.asarray(positions)[:, None])
    o = torch.nn.functional.scaled_dot_product_attention(qt, kt, vt, attn_mask=mask, scale=scale)
    return o[0].permute(1, 0, 2).reshape(T, Hq * hd).numpy()


@pytest.mark.parametrize("Hq,Hkv", [(4, 2), (4, 4), (6, 1)])
def test_attention_matches_library_sdpa(oracle64, Hq, Hkv):
    """Eq. 1 with a causal mask and grouped heads against torch SDPA (fp64, explicit mask)."""
    rng = np.random.default_rng(5)
    hd = 8
    lens, news = [11, 6], [4, 6]  # second request has no cached prefix
    qsl = np.array([0, 4, 10], np.int32)
    kvl = np.array([0, 11, 17], np.int32)
    pos = np.concatenate([np.arange(7, 11), np.arange(0, 6)]).astype(np.int32)
    q = rng.standard_normal((10, Hq * hd)) * 2
    K = rng.standard_normal((17, Hkv * hd)) * 2
    V = rng.standard_normal((17, Hkv * hd))
    out, pairs = oracle64.attention(q, K, V, kvl, pos, qsl, Hq, Hkv, hd)
    for r in range(2):
        ref = _sdpa_reference(q[qsl[r]:qsl[r + 1]], K[kvl[r]:kvl[r + 1]], V[kvl[r]:kvl[r + 1]],
                              pos[qsl[r]:qsl[r + 1]], Hq, Hkv, hd, 1 / np.sqrt(hd))
        np.testing.assert_allclose(out[qsl[r]:qsl[r + 1]], ref, rtol=1e-10, atol=1e-12)
    assert pairs == sum(p + 1 for p in pos)


def test_attention_closed_forms(oracle64):
    hd, Hq, Hkv = 4, 2, 1
    # one visible key: output is that key's value row, whatever the scores
    q = np.array([[1., 2, 3, 4, -1, 0, 2, 5]])
    K = np.array([[0.3, -2, 1, 7.]]); V = np.array([[9., 8, 7, 6]])
    out, _ = oracle64.attention(q, K, V, [0, 1], [0], [0, 1], Hq, Hkv, hd)
    np.testing.assert_allclose(out, [[9, 8, 7, 6, 9, 8, 7, 6]], atol=1e-14)
    # q = 0: uniform weights over exactly the p+1 visible keys (catches a mask that is off by one)
    V = np.arange(20, dtype=np.float64).reshape(5, 4)
    K = np.random.default_rng(0).standard_normal((5, 4))
    out, pairs = oracle64.attention(np.zeros((2, 8)), K, V, [0, 5], [2, 4], [0, 2], Hq, Hkv, hd)
    np.testing.assert_allclose(out[0, :4], V[:3].mean(0), atol=1e-13)
    np.testing.assert_allclose(out[1, 4:], V[:5].mean(0), atol=1e-13)
    assert pairs == 3 + 5
    # two keys, scores a*b/sqrt(hd) and 0: weight of key 0 is the logistic of the scaled score
    a, bb = 3.0, 0.7
    q = np.zeros((1, 8)); q[0, 0] = a; q[0, 4] = -a
    K = np.zeros((2, 4)); K[0, 0] = bb
    V = np.array([[1., 0, 0, 0], [0, 1., 0, 0]])
    out, _ = oracle64.attention(q, K, V, [0, 2], [1], [0, 1], Hq, Hkv, hd)
    w = 1 / (1 + np.exp(-a * bb / np.sqrt(hd)))
    np.testing.assert_allclose(out[0, :2], [w, 1 - w], atol=1e-14)
    np.testing.assert_allclose(out[0, 4:6], [1 - w, w], atol=1e-14)
    # constant V rows: output equals the constant; softmax weights sum to one
    rng = np.random.default_rng(1)
    q = rng.standard_normal((3, 8)) * 30  # large scores: needs the max subtraction to stay finite
    K = rng.standard_normal((6, 4)) * 30
    V = np.tile(np.array([[2., -1, 0.5, 4]]), (6, 1))
    out, _ = oracle64.attention(q, K, V, [0, 6], [3, 4, 5], [0, 3], Hq, Hkv, hd)
    np.testing.assert_allclose(out, np.tile(V[0], (3, 2)), atol=1e-12)
    assert np.isfinite(out).all()


def test_group_head_mapping_brute_force(oracle64):
    """Query head h must read KV head h // G: brute force in Python on a tiny case."""
    rng = np.random.default_rng(2)
    Hq, Hkv, hd, L = 6, 3, 2, 4
    q = rng.standard_normal((1, Hq * hd)); K = rng.standard_normal((L, Hkv * hd))
    V = rng.standard_normal((L, Hkv * hd))
    out, _ = oracle64.attention(q, K, V, [0, L], [L - 1], [0, 1], Hq, Hkv, hd)
    for h in range(Hq):
        g = h // 2
        s = [sum(q[0, h * hd + d] * K[j, g * hd + d] for d in range(hd)) / np.sqrt(hd) for j in range(L)]
        e = [np.exp(v - max(s)) for v in s]
        for d in range(hd):
            ref = sum(e[j] * V[j, g * hd + d] for j in range(L)) / sum(e)
            assert abs(out[0, h * hd + d] - ref) < 1e-13


# ---- cache reuse, decode, paging, counts ----------------------------------------------------------------

def _base_prefix_cache(orc, W, b, A):
    Ks, Vs = [], []
    for r in range(b.R):
        P = int(b.prefix_lens[r])
        qkv, _ = orc.project_qkv(b.prefix_hidden[r], W, SMALL.Nq, SMALL.Nkv, np.arange(P), [0, P],
                                 [0], [-1], A)
        Ks.append(qkv[:, SMALL.Nq:SMALL.Nq + SMALL.Nkv]); Vs.append(qkv[:, SMALL.Nq + SMALL.Nkv:])
    return Ks, Vs


def test_cache_reuse_identity(oracle64):
    """Prop. 1: aLoRA over the whole sequence from scratch == base prefix cache + aLoRA suffix."""
    W, ads, b = _setup()
    A = [_ad(a) for a in ads]
    kw = dict(Nq=SMALL.Nq, Nkv=SMALL.Nkv, Hq=4, Hkv=2, hd=8)
    Ks, Vs = _base_prefix_cache(oracle64, W, b, A)
    reuse = oracle64.attention_block(b.hidden, W, positions=b.positions, query_start_loc=b.query_start_loc,
                                     activation_offsets=b.activation_offsets, adapter_ids=b.adapter_ids,
                                     adapters=A, prefix_K=Ks, prefix_V=Vs, **kw)
    xs, pos, qsl = _full_sequence_batch(b, None)
    scratch = oracle64.attention_block(xs, W, positions=pos, query_start_loc=qsl,
                                       activation_offsets=b.activation_offsets, adapter_ids=b.adapter_ids,
                                       adapters=A, prefix_K=[None] * b.R, prefix_V=[None] * b.R, **kw)
    for r in range(b.R):
        np.testing.assert_array_equal(scratch["K"][r], reuse["K"][r])
        np.testing.assert_array_equal(scratch["V"][r], reuse["V"][r])
        lo, hi = b.query_start_loc[r], b.query_start_loc[r + 1]
        tail = slice(qsl[r] + b.prefix_lens[r], qsl[r + 1])
        np.testing.assert_array_equal(scratch["out"][tail], reuse["out"][lo:hi])
    # and the ordinary LoRA of Eq. 4 does NOT have this property (its prefix rows differ)
    lora = oracle64.attention_block(xs, W, positions=pos, query_start_loc=qsl,
                                    activation_offsets=b.activation_offsets, adapter_ids=b.adapter_ids,
                                    adapters=A, prefix_K=[None] * b.R, prefix_V=[None] * b.R,
                                    force_all=True, **kw)
    assert np.abs(lora["K"][0][:b.prefix_lens[0]] - Ks[0]).max() > 1e-3


def test_decode_step_equals_prefill_row(oracle64):
    """Prop. 1, second sentence: feeding the suffix one token at a time gives the prefill's rows."""
    W, ads, b = _setup()
    A = [_ad(a) for a in ads]
    kw = dict(Nq=SMALL.Nq, Nkv=SMALL.Nkv, Hq=4, Hkv=2, hd=8)
    Ks, Vs = _base_prefix_cache(oracle64, W, b, A)
    pre = oracle64.attention_block(b.hidden, W, positions=b.positions, query_start_loc=b.query_start_loc,
                                   activation_offsets=b.activation_offsets, adapter_ids=b.adapter_ids,
                                   adapters=A, prefix_K=Ks, prefix_V=Vs, **kw)
    for r in range(b.R):
        K, V = Ks[r], Vs[r]
        for i, t in enumerate(range(b.query_start_loc[r], b.query_start_loc[r + 1])):
            step = oracle64.attention_block(b.hidden[t:t + 1], W, positions=[b.positions[t]],
                                            query_start_loc=[0, 1],
                                            activation_offsets=[b.activation_offsets[r]],
                                            adapter_ids=[b.adapter_ids[r]], adapters=A,
                                            prefix_K=[K], prefix_V=[V], **kw)
            np.testing.assert_allclose(step["out"][0], pre["out"][t], rtol=0, atol=1e-14)
            K, V = step["K"][0], step["V"][0]
        np.testing.assert_array_equal(K, pre["K"][r])


def test_slot_mapping_brute_force_and_page_permutation(oracle64):
    W, ads, b = _setup(prefix=(7, 12, 0), new=(5, 3, 9), ids=(0, 1, -1), a_req=None)
    ps = SMALL.page_size
    slots = oracle64.slot_mapping(b.positions, b.query_start_loc, b.block_tables, ps)
    t = 0
    for r in range(b.R):
        for p in range(b.prefix_lens[r], b.seq_lens[r]):
            assert slots[t] == b.block_tables[r][p // ps] * ps + p % ps
            t += 1
    assert len(set(slots.tolist())) == b.T
    # append + gather round trip through two different physical page assignments
    rng = np.random.default_rng(3)
    krows = rng.standard_normal((b.T, SMALL.Nkv)).astype(np.float32)
    vrows = rng.standard_normal((b.T, SMALL.Nkv)).astype(np.float32)
    results = []
    for perm_seed in (0, 1):
        perm = np.random.default_rng(perm_seed).permutation(b.num_pages).astype(np.int32)
        bt = perm[b.block_tables]
        pool = np.full((b.num_pages, 2, SMALL.n_kv_heads, ps, SMALL.head_dim), -7.0, np.float32)
        before = pool.copy()
        s = oracle64.slot_mapping(b.positions, b.query_start_loc, bt, ps)
        oracle64.paged_append(pool, krows, vrows, s, SMALL.n_kv_heads, ps, SMALL.head_dim)
        # exactly T * Hkv * hd * 2 elements changed, all inside the new tokens' slots
        changed = pool != before
        assert changed.sum() == b.T * SMALL.Nkv * 2
        per = []
        for r in range(b.R):
            K, V = oracle64.paged_gather(pool, bt[r], int(b.seq_lens[r]), SMALL.n_kv_heads, ps, SMALL.head_dim)
            lo, hi = b.query_start_loc[r], b.query_start_loc[r + 1]
            np.testing.assert_array_equal(K[b.prefix_lens[r]:], krows[lo:hi])
            np.testing.assert_array_equal(V[b.prefix_lens[r]:], vrows[lo:hi])
            assert (K[:b.prefix_lens[r]] == -7).all()
            per.append((K, V))
        results.append(per)
    for (K0, V0), (K1, V1) in zip(*results):
        np.testing.assert_array_equal(K0, K1)
        np.testing.assert_array_equal(V0, V1)


def test_prop2_operation_and_row_counts(oracle64):
    """Prop. 2: score pairs S*P + S(S+1)/2 with cache reuse vs (P+S)(P+S+1)/2 without; rows S vs P+S."""
    W, ads, b = _setup()
    A = [_ad(a) for a in ads]
    kw = dict(Nq=SMALL.Nq, Nkv=SMALL.Nkv, Hq=4, Hkv=2, hd=8)
    Ks, Vs = _base_prefix_cache(oracle64, W, b, A)
    reuse = oracle64.attention_block(b.hidden, W, positions=b.positions, query_start_loc=b.query_start_loc,
                                     activation_offsets=b.activation_offsets, adapter_ids=b.adapter_ids,
                                     adapters=A, prefix_K=Ks, prefix_V=Vs, **kw)
    xs, pos, qsl = _full_sequence_batch(b, None)
    full = oracle64.attention_block(xs, W, positions=pos, query_start_loc=qsl,
                                    activation_offsets=b.activation_offsets, adapter_ids=b.adapter_ids,
                                    adapters=A, prefix_K=[None] * b.R, prefix_V=[None] * b.R,
                                    force_all=True, **kw)
    P, S = b.prefix_lens.astype(int), (b.seq_lens - b.prefix_lens).astype(int)
    assert reuse["pairs"] == int((S * P + S * (S + 1) // 2).sum())
    assert full["pairs"] == int(((P + S) * (P + S + 1) // 2).sum())
    assert reuse["qkv"].shape[0] == S.sum() and full["qkv"].shape[0] == (P + S).sum()


def test_f32_build_agrees_with_f64(oracle64, oracle32):
    W, ads, b = _setup()
    A = [_ad(a) for a in ads]
    kw = dict(Nq=SMALL.Nq, Nkv=SMALL.Nkv, Hq=4, Hkv=2, hd=8)
    Ks, Vs = _base_prefix_cache(oracle64, W, b, A)
    r64 = oracle64.attention_block(b.hidden, W, positions=b.positions, query_start_loc=b.query_start_loc,
                                   activation_offsets=b.activation_offsets, adapter_ids=b.adapter_ids,
                                   adapters=A, prefix_K=Ks, prefix_V=Vs, **kw)
    r32 = oracle32.attention_block(b.hidden, W, positions=b.positions, query_start_loc=b.query_start_loc,
                                   activation_offsets=b.activation_offsets, adapter_ids=b.adapter_ids,
                                   adapters=A, prefix_K=Ks, prefix_V=Vs, **kw)
    assert np.abs(r64["qkv"] - r32["qkv"]).max() < 1e-5 * np.abs(r64["qkv"]).max()
    assert np.abs(r64["out"] - r32["out"]).max() < 1e-5 * np.abs(r64["out"]).max()
    assert np.abs(r64["out"] - r32["out"]).max() > 0  # the two builds really differ in precision


# ---- decoder-layer glue -----------------------------------------------------------------------------

def test_rmsnorm_swiglu_linear_against_library(oracle64):
    rng = np.random.default_rng(4)
    x = rng.standard_normal((5, 32)); w = rng.standard_normal(32).astype(np.float32)
    ref = torch.nn.functional.rms_norm(torch.from_numpy(x), (32,), torch.from_numpy(w.astype(np.float64)), 1e-5)
    np.testing.assert_allclose(oracle64.rmsnorm(x, w, 1e-5), ref.numpy(), rtol=1e-12)
    gu = rng.standard_normal((5, 12))
    ref = torch.nn.functional.silu(torch.from_numpy(gu[:, :6])) * torch.from_numpy(gu[:, 6:])
    np.testing.assert_allclose(oracle64.swiglu(gu), ref.numpy(), rtol=1e-12)
    Wm = rng.standard_normal((7, 32)).astype(np.float32)
    np.testing.assert_allclose(oracle64.linear(x, Wm), x @ Wm.astype(np.float64).T, rtol=1e-12, atol=1e-13)


def test_prop1_holds_through_a_two_layer_stack(oracle64):
    """Prop. 1's induction over depth: with the gate, every state of every prefix token agrees with
    the base model's after two full decoder layers."""
    shape = wl.LayerShape(hidden=32, n_q_heads=4, n_kv_heads=2, head_dim=8, page_size=4, dtype="fp32",
                          intermediate=48)
    rng = np.random.default_rng(6)
    layers = [wl.make_stack_weights(shape, rng) for _ in range(2)]
    for lw in layers:
        for k in ("wqkv", "wo", "wgate_up", "wdown"):
            lw[k] = lw[k] * 10
    ads = [[wl.make_adapter(shape, 4, rng) for _ in range(1)] for _ in range(2)]
    for per_layer in ads:
        for a in per_layer:
            for n in ("Aq", "Bq", "Ak", "Bk", "Av", "Bv"):
                setattr(a, n, getattr(a, n) * 20)
    L, a_req = 12, 7
    h = rng.standard_normal((L, 32))
    pos, qsl = np.arange(L), [0, L]
    kw = dict(Nq=shape.Nq, Nkv=shape.Nkv, Hq=4, Hkv=2, hd=8, eps=1e-5)

    def run(ids):
        x = h
        states = []
        for l in range(2):
            x, blk = oracle64.decoder_layer(x, layers[l], positions=pos, query_start_loc=qsl,
                                            activation_offsets=[a_req], adapter_ids=ids,
                                            adapters=[_ad(a) for a in ads[l]], prefix_K=[None],
                                            prefix_V=[None], **kw)
            states.append((x, blk["K"][0], blk["V"][0]))
        return states

    for (xa, Ka, Va), (xb, Kb, Vb) in zip(run([0]), run([-1])):
        np.testing.assert_array_equal(xa[:a_req], xb[:a_req])
        np.testing.assert_array_equal(Ka[:a_req], Kb[:a_req])
        np.testing.assert_array_equal(Va[:a_req], Vb[:a_req])
        assert np.abs(xa[a_req:] - xb[a_req:]).max() > 1e-6


# ---- decoder layer against an independent restatement; pool layout by plain indexing ----------------

STACK_SHAPE = wl.LayerShape(hidden=32, n_q_heads=4, n_kv_heads=2, head_dim=8, page_size=4, dtype="fp32",
                            intermediate=48)


def _torch_decoder_layer(h, lw, ad, shape, eps, positions, qsl, a_req, ids, prefix_K, prefix_V):
    """Pre-norm residual decoder layer written with library ops only (fp64): rms_norm, matmul,
    scaled_dot_product_attention under an explicit visibility mask, silu.  One request at a time."""
    F = torch.nn.functional
    t64 = lambda a: torch.from_numpy(np.asarray(a, np.float64))
    H, Nq, Nkv, Hq, Hkv, hd, I = (shape.hidden, shape.Nq, shape.Nkv, shape.n_q_heads, shape.n_kv_heads,
                                  shape.head_dim, shape.intermediate)
    out = torch.empty((len(positions), H), dtype=torch.float64)
    for r in range(len(qsl) - 1):
        lo, hi = int(qsl[r]), int(qsl[r + 1])
        x, pos = t64(h[lo:hi]), torch.as_tensor(np.asarray(positions[lo:hi], np.int64))
        xn = F.rms_norm(x, (H,), t64(lw["norm_attn"]), eps)
        qkv = xn @ t64(lw["wqkv"]).T
        if ids[r] >= 0:
            a = ad[ids[r]]
            delta = torch.cat([(xn @ t64(a.Aq).T) @ t64(a.Bq).T, (xn @ t64(a.Ak).T) @ t64(a.Bk).T,
                               (xn @ t64(a.Av).T) @ t64(a.Bv).T], dim=1) * a.scale
            qkv = torch.where((pos >= int(a_req[r]))[:, None], qkv + delta, qkv)
        K = torch.cat([t64(prefix_K[r]), qkv[:, Nq:Nq + Nkv]]) if prefix_K[r] is not None else qkv[:, Nq:Nq + Nkv]
        V = torch.cat([t64(prefix_V[r]), qkv[:, Nq + Nkv:]]) if prefix_V[r] is not None else qkv[:, Nq + Nkv:]
        L = K.shape[0]
        q = qkv[:, :Nq].reshape(hi - lo, Hq, hd).transpose(0, 1)
        Kh = K.reshape(L, Hkv, hd).transpose(0, 1).repeat_interleave(Hq // Hkv, dim=0)
        Vh = V.reshape(L, Hkv, hd).transpose(0, 1).repeat_interleave(Hq // Hkv, dim=0)
        visible = torch.arange(L)[None, :] <= pos[:, None]
        o = F.scaled_dot_product_attention(q, Kh, Vh, attn_mask=visible)
        h1 = x + o.transpose(0, 1).reshape(hi - lo, Nq) @ t64(lw["wo"]).T
        xm = F.rms_norm(h1, (H,), t64(lw["norm_mlp"]), eps)
        gu = xm @ t64(lw["wgate_up"]).T
        out[lo:hi] = h1 + (F.silu(gu[:, :I]) * gu[:, I:]) @ t64(lw["wdown"]).T
    return out.numpy()


def test_decoder_layer_against_library_restatement(oracle64):
    """The layer composition (norm, gated q/k/v, attention over cached ++ new rows, o_proj and its
    residual, norm, SwiGLU MLP and its residual) against the same layer written with torch ops:
    two requests, one with an adapter whose gate opens in the middle of its new tokens, both on
    cached prefixes.  Weights are scaled up so that either residual branch, either norm gain and
    the delta each move the result by far more than the tolerance."""
    shape, eps = STACK_SHAPE, 1e-5
    rng = np.random.default_rng(11)
    lw = wl.make_stack_weights(shape, rng)
    for k in ("wqkv", "wo", "wgate_up", "wdown"):
        lw[k] = lw[k] * 10
    ad = [wl.make_adapter(shape, 4, rng)]
    for n in ("Aq", "Bq", "Ak", "Bk", "Av", "Bv"):
        setattr(ad[0], n, getattr(ad[0], n) * 20)
    prefix, new, ids, a_req = (6, 9), (7, 5), (0, -1), (9, 0)
    T = sum(new)
    h = rng.standard_normal((T, shape.hidden))
    qsl = np.asarray([0, new[0], T], np.int32)
    pos = np.concatenate([np.arange(p, p + n) for p, n in zip(prefix, new)]).astype(np.int32)
    pK = [rng.standard_normal((p, shape.Nkv)) for p in prefix]
    pV = [rng.standard_normal((p, shape.Nkv)) for p in prefix]
    got, blk = oracle64.decoder_layer(h, lw, shape.Nq, shape.Nkv, shape.n_q_heads, shape.n_kv_heads,
                                      shape.head_dim, eps, pos, qsl, a_req, ids, [_ad(ad[0])], pK, pV)
    want = _torch_decoder_layer(h, lw, ad, shape, eps, pos, qsl, a_req, ids, pK, pV)
    np.testing.assert_allclose(got, want, rtol=1e-10, atol=1e-11)
    assert blk["gate"].tolist() == [0, 0, 0, 1, 1, 1, 1] + [0] * 5
    # each part of the composition carries weight here: leaving it out is far outside the tolerance
    assert np.abs(got - h).max() > 0.1


# ---- gated adapters on the MLP block (Eq. 5's form applied to gate, up, down) ---------------------------

def _mlp_ad(a: wl.MlpAdapterWeights) -> MlpAdapter:
    return MlpAdapter(a.rank, a.scale, a.Ag, a.Bg, a.Au, a.Bu, a.Ad, a.Bd)


def _mlp_linear_case(seed=21):
    rng = np.random.default_rng(seed)
    K, N = 24, 40
    W = (rng.standard_normal((N, K)) * 0.3).astype(np.float32)
    ranks, scales = [3, 5], [1.0, 0.5]
    As = [(rng.standard_normal((r, K)) * 0.4).astype(np.float32) for r in ranks]
    Bs = [(rng.standard_normal((N, r)) * 0.4).astype(np.float32) for r in ranks]
    prefix, new, ids = (4, 9, 2), (6, 5, 3), (1, -1, 0)
    qsl = np.concatenate([[0], np.cumsum(new)]).astype(np.int32)
    pos = np.concatenate([np.arange(p, p + n) for p, n in zip(prefix, new)]).astype(np.int32)
    x = rng.standard_normal((sum(new), K))
    return x, W, pos, qsl, ids, ranks, scales, As, Bs, prefix, new


def test_mlp_gated_linear_special_cases(oracle64):
    """One adapted MLP matrix: rows before the activation offset are bit-equal to the plain product, B = 0 gives the
    plain product everywhere, an offset of 0 gives the merged matrix W + s B A (library matmul), and a mid-chunk
    offset gives the row-wise mix of the two; adapters 0 and 1 have different ranks and scales."""
    x, W, pos, qsl, ids, ranks, scales, As, Bs, prefix, new = _mlp_linear_case()
    base = oracle64.linear(x, W)
    a_req = [prefix[0] + 2, 0, prefix[2] + 1]            # opens inside request 0 and request 2
    y = oracle64.gated_linear(x, W, pos, qsl, a_req, ids, ranks, scales, As, Bs)
    W64 = W.astype(np.float64)
    for r in range(3):
        lo, hi = qsl[r], qsl[r + 1]
        if ids[r] < 0:
            np.testing.assert_array_equal(y[lo:hi], base[lo:hi])
            continue
        k = ids[r]
        merged = W64 + scales[k] * Bs[k].astype(np.float64) @ As[k].astype(np.float64)
        open_ = pos[lo:hi] >= a_req[r]
        assert open_.any() and not open_.all()
        np.testing.assert_array_equal(y[lo:hi][~open_], base[lo:hi][~open_])
        np.testing.assert_allclose(y[lo:hi][open_], x[lo:hi][open_] @ merged.T, rtol=1e-11, atol=1e-12)
        assert np.abs(y[lo:hi][open_] - base[lo:hi][open_]).max() > 1e-2
    zero = oracle64.gated_linear(x, W, pos, qsl, [0, 0, 0], ids, ranks, scales, As, [b * 0 for b in Bs])
    np.testing.assert_array_equal(zero, base)
    late = oracle64.gated_linear(x, W, pos, qsl, [10 ** 6] * 3, ids, ranks, scales, As, Bs)
    np.testing.assert_array_equal(late, base)
    forced = oracle64.gated_linear(x, W, pos, qsl, [10 ** 6] * 3, ids, ranks, scales, As, Bs, force_all=True)
    lo, hi = qsl[0], qsl[1]
    np.testing.assert_allclose(forced[lo:hi], x[lo:hi] @ (W64 + scales[1] * Bs[1].astype(np.float64) @ As[1].astype(np.float64)).T,
                               rtol=1e-11, atol=1e-12)


def _torch_adapted_mlp(h1, lw, mlp, shape, eps, pos, a_req, adapter):
    """norm, adapted gate / up, SwiGLU, adapted down and the residual of ONE request in torch fp64 ops."""
    F = torch.nn.functional
    t64 = lambda a: torch.from_numpy(np.asarray(a, np.float64))
    H, I = shape.hidden, shape.intermediate
    h1 = t64(h1)
    xm = F.rms_norm(h1, (H,), t64(lw["norm_mlp"]), eps)
    open_ = (torch.as_tensor(np.asarray(pos, np.int64)) >= int(a_req))[:, None] if adapter is not None else None
    wg, wu = t64(lw["wgate_up"][:I]), t64(lw["wgate_up"][I:])

    def lin(x, W, A, B):
        y = x @ W.T
        if adapter is None:
            return y
        return torch.where(open_, y + adapter.scale * ((x @ t64(A).T) @ t64(B).T), y)

    m = adapter
    gate = lin(xm, wg, m.Ag if m else None, m.Bg if m else None)
    up = lin(xm, wu, m.Au if m else None, m.Bu if m else None)
    act = F.silu(gate) * up
    return (h1 + lin(act, t64(lw["wdown"]), m.Ad if m else None, m.Bd if m else None)).numpy()


def test_decoder_layer_with_mlp_adapters_against_library_restatement(oracle64):
    """The layer with adapters on q/k/v AND on gate, up and down: the attention half is taken from the oracle's own
    layer without MLP adapters (pinned above), the MLP half is restated in torch ops.  The gate opens in the middle
    of request 0's new tokens; request 1 runs the base model.  Every adapted matrix carries weight: zeroing any one
    of Bg, Bu, Bd moves the result by far more than the tolerance."""
    shape, eps = STACK_SHAPE, 1e-5
    rng = np.random.default_rng(12)
    lw = wl.make_stack_weights(shape, rng)
    for k in ("wqkv", "wo", "wgate_up", "wdown"):
        lw[k] = lw[k] * 10
    ad = [wl.make_adapter(shape, 4, rng)]
    mlp = [wl.make_mlp_adapter(shape, 4, rng, scale=0.5)]
    for n in ("Ag", "Bg", "Au", "Bu", "Ad", "Bd"):
        setattr(mlp[0], n, getattr(mlp[0], n) * 20)
    prefix, new, ids, a_req = (6, 9), (7, 5), (0, -1), (9, 0)
    T = sum(new)
    h = rng.standard_normal((T, shape.hidden))
    qsl = np.asarray([0, new[0], T], np.int32)
    pos = np.concatenate([np.arange(p, p + n) for p, n in zip(prefix, new)]).astype(np.int32)
    pK = [rng.standard_normal((p, shape.Nkv)) for p in prefix]
    pV = [rng.standard_normal((p, shape.Nkv)) for p in prefix]
    args = (h, lw, shape.Nq, shape.Nkv, shape.n_q_heads, shape.n_kv_heads, shape.head_dim, eps, pos, qsl, a_req, ids,
            [_ad(ad[0])], pK, pV)
    got, blk = oracle64.decoder_layer(*args, mlp_adapters=[_mlp_ad(mlp[0])])
    # h1 = the state after the attention half, from the composition pinned by the test above
    h1 = h + oracle64.linear(blk["out"], lw["wo"])
    want = np.concatenate([_torch_adapted_mlp(h1[:7], lw, mlp, shape, eps, pos[:7], a_req[0], mlp[0]),
                           _torch_adapted_mlp(h1[7:], lw, mlp, shape, eps, pos[7:], a_req[1], None)])
    np.testing.assert_allclose(got, want, rtol=1e-10, atol=1e-11)
    plain, _ = oracle64.decoder_layer(*args)
    np.testing.assert_array_equal(got[:3], plain[:3])       # rows before the offset: the layer without MLP adapters
    np.testing.assert_array_equal(got[7:], plain[7:])       # the base-model request
    assert np.abs(got[3:7] - plain[3:7]).max() > 0.1
    for name in ("Bg", "Bu", "Bd"):
        z = _mlp_ad(mlp[0])
        setattr(z, name, getattr(z, name) * 0)
        other, _ = oracle64.decoder_layer(*args, mlp_adapters=[z])
        assert np.abs(other[3:7] - got[3:7]).max() > 1e-2, name


def test_cache_reuse_identity_through_two_layers_with_mlp_adapters(oracle64):
    """Prop. 1 with adapted MLP blocks: because the MLP adapters are gated like q/k/v, a whole sequence run from
    scratch leaves, in BOTH layers, prefix K/V bit-equal to the base model's, and the suffix computed on the base
    model's caches equals the suffix rows of the from-scratch run.  With the MLP gate left open on the prefix
    (ordinary LoRA on the MLP) the second layer's prefix K/V differ: the identity needs the gate."""
    shape, eps = STACK_SHAPE, 1e-5
    rng = np.random.default_rng(13)
    layers = [wl.make_stack_weights(shape, rng) for _ in range(2)]
    for lw in layers:
        for k in ("wqkv", "wo", "wgate_up", "wdown"):
            lw[k] = lw[k] * 10
    ads = [[wl.make_adapter(shape, 4, rng)] for _ in range(2)]
    mlps = [[wl.make_mlp_adapter(shape, 4, rng)] for _ in range(2)]
    for per in mlps:
        for n in ("Ag", "Bg", "Au", "Bu", "Ad", "Bd"):
            setattr(per[0], n, getattr(per[0], n) * 20)
    P, S = 9, 5
    L = P + S
    h = rng.standard_normal((L, shape.hidden))
    kw = dict(Nq=shape.Nq, Nkv=shape.Nkv, Hq=shape.n_q_heads, Hkv=shape.n_kv_heads, hd=shape.head_dim, eps=eps)

    def run(x, pos, a_req, ids, caches, mlp_gate_open=False):
        out = []
        for l in range(2):
            m = [_mlp_ad(mlps[l][0])]
            if mlp_gate_open:   # ordinary LoRA on the MLP only: a separate call with offset 0 for the MLP half
                x1, blk = oracle64.decoder_layer(x, layers[l], positions=pos, query_start_loc=[0, len(pos)],
                                                 activation_offsets=[a_req], adapter_ids=ids,
                                                 adapters=[_ad(ads[l][0])], prefix_K=[caches[l][0]],
                                                 prefix_V=[caches[l][1]], **kw)
                h1 = x + oracle64.linear(blk["out"], layers[l]["wo"])
                x = _torch_adapted_mlp(h1, layers[l], None, shape, eps, pos, 0, mlps[l][0])
            else:
                x, blk = oracle64.decoder_layer(x, layers[l], positions=pos, query_start_loc=[0, len(pos)],
                                                activation_offsets=[a_req], adapter_ids=ids,
                                                adapters=[_ad(ads[l][0])], prefix_K=[caches[l][0]],
                                                prefix_V=[caches[l][1]], mlp_adapters=m, **kw)
            out.append((x, blk["K"][0], blk["V"][0]))
        return out

    none = [(None, None)] * 2
    base = run(h[:P], np.arange(P), 0, [-1], none)                       # base model prefills the prefix
    scratch = run(h, np.arange(L), P, [0], none)                         # aLoRA on the whole sequence
    reuse = run(h[P:], np.arange(P, L), P, [0], [(K, V) for _, K, V in base])
    # hidden states entering layer 2 on the reuse path are the suffix rows of layer 1's output
    for l in range(2):
        np.testing.assert_array_equal(scratch[l][1][:P], base[l][1])
        np.testing.assert_array_equal(scratch[l][2][:P], base[l][2])
        np.testing.assert_allclose(reuse[l][0], scratch[l][0][P:], rtol=1e-11, atol=1e-12)
        np.testing.assert_allclose(reuse[l][1][P:], scratch[l][1][P:], rtol=1e-11, atol=1e-12)
    assert np.abs(scratch[1][0][P:] - run(h, np.arange(L), P, [-1], none)[1][0][P:]).max() > 1e-2
    lora_mlp = run(h, np.arange(L), P, [0], none, mlp_gate_open=True)
    np.testing.assert_array_equal(lora_mlp[0][1][:P], base[0][1])        # layer 1's keys see no MLP yet
    assert np.abs(lora_mlp[1][1][:P] - base[1][1]).max() > 1e-3          # layer 2's prefix keys are no longer the base's


def test_pool_layout_by_plain_indexing(oracle64):
    """The cache layout pool[page][plane][kv head][row][hd] (plane 0 = K, 1 = V), read back with
    numpy indexing after an append: row p of a request sits in page block_table[p // page] at row
    p % page, K in plane 0, V in plane 1, head g in pool[..., g, row, :].  Heads, planes, rows and
    head-dim extents all differ, so a layout with any two of them exchanged cannot pass."""
    Hkv, ps, hd = 3, 4, 5
    rng = np.random.default_rng(12)
    bt = np.asarray([[5, 2, 7], [1, 6, 0]], np.int32)
    prefix, new = (3, 0), (6, 5)
    qsl = np.asarray([0, 6, 11], np.int32)
    pos = np.concatenate([np.arange(p, p + n) for p, n in zip(prefix, new)]).astype(np.int32)
    T = 11
    k = rng.standard_normal((T, Hkv * hd)).astype(np.float32)
    v = rng.standard_normal((T, Hkv * hd)).astype(np.float32)
    pool = np.full((9, 2, Hkv, ps, hd), -7.0, np.float32)
    slots = oracle64.slot_mapping(pos, qsl, bt, ps)
    oracle64.paged_append(pool, k, v, slots, Hkv, ps, hd)
    untouched = np.ones(pool.shape, bool)
    for r in range(2):
        for t in range(qsl[r], qsl[r + 1]):
            page, row = bt[r, pos[t] // ps], pos[t] % ps
            assert slots[t] == page * ps + row
            for g in range(Hkv):
                np.testing.assert_array_equal(pool[page, 0, g, row, :], k[t, g * hd:(g + 1) * hd])
                np.testing.assert_array_equal(pool[page, 1, g, row, :], v[t, g * hd:(g + 1) * hd])
            untouched[page, :, :, row, :] = False
    assert (pool[untouched] == -7).all()
    # the gather reads the same layout: fill a pool by indexing, gather it, compare
    pool2 = rng.standard_normal(pool.shape).astype(np.float32)
    K, V = oracle64.paged_gather(pool2, bt[0], 9, Hkv, ps, hd)
    for p in range(9):
        for g in range(Hkv):
            np.testing.assert_array_equal(K[p, g * hd:(g + 1) * hd], pool2[bt[0, p // ps], 0, g, p % ps, :])
            np.testing.assert_array_equal(V[p, g * hd:(g + 1) * hd], pool2[bt[0, p // ps], 1, g, p % ps, :])


# ---- optional rotary position embedding -----------------------------------------------------------------

def _rope_complex(x, positions, n_heads, hd, theta):
    """Independent restatement: the pair (x[i], x[i + hd/2]) as the complex number x[i] + j x[i + hd/2], multiplied
    by exp(j p theta^(-2i/hd))."""
    T = x.shape[0]
    v = np.asarray(x, np.float64).reshape(T, n_heads, 2, hd // 2)
    z = v[:, :, 0, :] + 1j * v[:, :, 1, :]
    freq = theta ** (-2.0 * np.arange(hd // 2) / hd)
    z = z * np.exp(1j * np.asarray(positions, np.float64)[:, None, None] * freq[None, None, :])
    return np.stack([z.real, z.imag], axis=2).reshape(T, n_heads * hd)


def test_rope_against_complex_multiplication_and_hand_example(oracle64):
    rng = np.random.default_rng(21)
    x = rng.standard_normal((9, 3 * 16))
    pos = np.array([0, 1, 2, 3, 17, 100, 1000, 4095, 32767], np.int32)
    got = oracle64.rope(x, pos, 3, 16, 10000.0)
    np.testing.assert_allclose(got, _rope_complex(x, pos, 3, 16, 10000.0), rtol=1e-12, atol=1e-12)
    # position 0 is the identity; every head keeps its norm
    np.testing.assert_array_equal(got[0], x[0])
    np.testing.assert_allclose(np.linalg.norm(got.reshape(9, 3, 16), axis=2), np.linalg.norm(x.reshape(9, 3, 16), axis=2),
                               rtol=1e-12)
    assert np.abs(got[1:] - x[1:]).max() > 0.1
    # hand-worked values (tests/golden/rope_hand_example.txt)
    vals = {}
    for line in open(os.path.join(os.path.dirname(__file__), "golden", "rope_hand_example.txt")):
        line = line.split("#")[0].strip()
        if "=" in line:
            k, v = line.split("=")
            vals[k.strip()] = [float(t) for t in v.split()]
    y = oracle64.rope(np.array([vals["x"]]), [int(vals["p"][0])], 1, int(vals["hd"][0]), vals["theta"][0])
    np.testing.assert_allclose(y[0], vals["y"], rtol=1e-13)


def test_rope_scores_depend_on_the_position_difference_only(oracle64):
    """<R_m q, R_n k> = <R_(m+s) q, R_(n+s) k> for any shift s: what makes cached post-rotation keys reusable."""
    rng = np.random.default_rng(22)
    q, k = rng.standard_normal((1, 32)), rng.standard_normal((1, 32))
    base = None
    for s in (0, 5, 900):
        qm = oracle64.rope(q, [7 + s], 1, 32, 500.0)
        kn = oracle64.rope(k, [3 + s], 1, 32, 500.0)
        dot = float(qm[0] @ kn[0])
        base = dot if base is None else base
        assert abs(dot - base) < 1e-10
    # ... and it does depend on the difference
    assert abs(float(oracle64.rope(q, [8], 1, 32, 500.0)[0] @ oracle64.rope(k, [3], 1, 32, 500.0)[0]) - base) > 1e-3


def test_rope_in_the_attention_block_is_rotation_then_plain_attention(oracle64):
    """With rope_theta set the block equals: project, rotate q and k rows by hand (complex restatement), then the
    plain block's attention on cached rotated keys.  Rows before the activation offset still equal the base
    model's (Prop. 1 does not care about the rotation: it is the same function of the row on both sides)."""
    W, ads, b = _setup(a_req=(9, 12))
    A = [_ad(a) for a in ads]
    kw = dict(Nq=SMALL.Nq, Nkv=SMALL.Nkv, Hq=4, Hkv=2, hd=8)
    theta = 100.0
    rng = np.random.default_rng(5)
    Ks = [rng.standard_normal((int(p), SMALL.Nkv)) for p in b.prefix_lens]
    Vs = [rng.standard_normal((int(p), SMALL.Nkv)) for p in b.prefix_lens]
    got = oracle64.attention_block(b.hidden, W, positions=b.positions, query_start_loc=b.query_start_loc,
                                   activation_offsets=b.activation_offsets, adapter_ids=b.adapter_ids, adapters=A,
                                   prefix_K=Ks, prefix_V=Vs, rope_theta=theta, **kw)
    qkv, _ = oracle64.project_qkv(b.hidden, W, SMALL.Nq, SMALL.Nkv, b.positions, b.query_start_loc,
                                  b.activation_offsets, b.adapter_ids, A)
    q = _rope_complex(qkv[:, :SMALL.Nq], b.positions, 4, 8, theta)
    k = _rope_complex(qkv[:, SMALL.Nq:SMALL.Nq + SMALL.Nkv], b.positions, 2, 8, theta)
    np.testing.assert_allclose(got["qkv"][:, :SMALL.Nq], q, rtol=1e-11, atol=1e-12)
    np.testing.assert_allclose(got["qkv"][:, SMALL.Nq:SMALL.Nq + SMALL.Nkv], k, rtol=1e-11, atol=1e-12)
    np.testing.assert_array_equal(got["qkv"][:, SMALL.Nq + SMALL.Nkv:], qkv[:, SMALL.Nq + SMALL.Nkv:])   # v is not rotated
    Kc = np.concatenate([np.concatenate([Ks[r], k[b.query_start_loc[r]:b.query_start_loc[r + 1]]]) for r in range(b.R)])
    Vc = np.concatenate([np.concatenate([Vs[r], qkv[b.query_start_loc[r]:b.query_start_loc[r + 1], SMALL.Nq + SMALL.Nkv:]])
                         for r in range(b.R)])
    kvl = np.concatenate([[0], np.cumsum(b.seq_lens)])
    want, _ = oracle64.attention(q, Kc, Vc, kvl, b.positions, b.query_start_loc, 4, 2, 8)
    np.testing.assert_allclose(got["out"], want, rtol=1e-11, atol=1e-12)
    base = oracle64.attention_block(b.hidden, W, positions=b.positions, query_start_loc=b.query_start_loc,
                                    activation_offsets=b.activation_offsets, adapter_ids=[-1, -1], adapters=A,
                                    prefix_K=Ks, prefix_V=Vs, rope_theta=theta, **kw)
    off = got["gate"] == 0
    assert off.sum() == 2 and np.array_equal(got["qkv"][off], base["qkv"][off])

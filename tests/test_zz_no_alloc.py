"""The allocation-free projection entry point against the regular one.

alora_project_qkv_static exists for callers that may not allocate device memory (a plug-in inside an
engine that owns all of it, a loop that cannot afford cudaMalloc's synchronisation).  It keeps its
scratch in a fixed array of the library, shared by all calls and never cleared, so the check is made
twice in a row with different batch shapes and gates: the second call must not see the first one's
leftovers.  Collected last on purpose (file name), and self-contained so that it also passes alone."""
import numpy as np
import pytest

from paper_2504_12397_b200 import binding as ab
from paper_2504_12397_b200 import workloads as wl

import helpers as hp

pytestmark = pytest.mark.gpu

SHAPE = wl.LayerShape(hidden=512, n_q_heads=4, n_kv_heads=2, head_dim=128, page_size=16, dtype="bf16")


def _case(seed, P, S, on, a_req, rank):
    rng = np.random.default_rng(seed)
    w = wl.make_wqkv(SHAPE, rng)
    ad = wl.make_adapter(SHAPE, rank, rng, scale=1.5)
    for n in ("Bq", "Bk", "Bv"):
        setattr(ad, n, wl.bf16_round(getattr(ad, n) * 8))
    ids = [0 if o else -1 for o in on]
    b = wl.make_batch(SHAPE, P, S, ids, rng, activation_offsets=a_req)
    return w, ad, b, np.asarray(on, np.int32)


def _oracle_qkv(orc, shape, w, ad, b, on):
    ids = np.where(np.asarray(on) != 0, 0, -1).astype(np.int32)
    want, gate = orc.project_qkv(b.hidden, w, shape.Nq, shape.Nkv, b.positions, b.query_start_loc,
                                 b.activation_offsets, ids, hp.oracle_adapters([ad]))
    return want, gate.astype(bool)


def _static_call(g, shape, dtype, d, w_dev, ad, mats, on, out):
    rc = ab.alora_project_qkv_static(g.cfg.dtype, shape.hidden, shape.Nq, shape.Nkv, d.hidden, w_dev, d.positions,
                                     d.qsl, d.a_req, None if on is None else hp.idev(on), ad.rank, ad.scale, *mats,
                                     d.T, d.R, out)
    assert rc == 0


@pytest.mark.parametrize("dtype", ["bf16", "fp32"])
def test_static_scratch_projection_matches_regular_entry_twice(oracle64, dtype):
    """Two calls in a row with different batch shapes and gates.  Each is compared with the regular entry point,
    with the CPU oracle directly, and -- for the rows whose gate is closed -- bit for bit with a call of the same
    entry in which no request has the adapter on (the base projection, Prop. 1)."""
    import torch
    shape = wl.LayerShape(**{**SHAPE.__dict__, "dtype": dtype})
    tol = 2e-2 if dtype == "bf16" else 1e-5
    cases = [_case(1, [10, 0, 300], [200, 90, 33], [1, 1, 1], [10, 0, 300], 32),      # every row gated on
             _case(2, [5, 64], [70, 41], [1, 0], [40, 64], 8)]                          # fewer rows, some gated off
    for w, ad, b, on in cases:
        g = hp.GpuLayers(shape, [dict(wqkv=w)], [[ad]], b.T, b.R)
        try:
            d = hp.DevBatch(b, dtype)
            want = g.empty(b.T, shape.N)
            ab.alora_project_qkv(g.ctx, 0, ab.MODE_ALORA, d.hidden, d.positions, d.a_req, d.ids, d.qsl, d.seq_lens,
                                 d.T, d.R, want)
            mats = [hp.to_dev(getattr(ad, n), dtype) for n in ("Aq", "Bq", "Ak", "Bk", "Av", "Bv")]
            got = torch.full_like(want, float("nan"))
            _static_call(g, shape, dtype, d, g.keep[0]["wqkv"], ad, mats, on, got)
            base = torch.full_like(want, float("nan"))
            _static_call(g, shape, dtype, d, g.keep[0]["wqkv"], ad, mats, np.zeros_like(on), base)
            torch.cuda.synchronize()
            assert g.status() == 0
            hp.assert_close(hp.to_host(got), hp.to_host(want), tol, "static entry against the regular entry")
            want_o, gate = _oracle_qkv(oracle64, shape, w, ad, b, on)
            hp.assert_close(hp.to_host(got), want_o, tol, "static entry against the oracle", block=shape.head_dim)
            base_o, _ = _oracle_qkv(oracle64, shape, w, ad, b, np.zeros_like(on))
            hp.assert_close(hp.to_host(base), base_o, tol, "static entry, adapter off, against the oracle")
            assert torch.equal(got[torch.from_numpy(~gate).cuda()], base[torch.from_numpy(~gate).cuda()]), \
                "rows with a closed gate must equal the base projection bit for bit"
            if gate.any():   # the delta is well above the tolerance in these fixtures
                assert hp.rel_err(hp.to_host(base)[gate], want_o[gate]) > 5 * tol
        finally:
            g.close()


def test_static_scratch_at_its_limits_allocates_nothing(oracle64):
    """The largest call the fixed array admits (ALORA_STATIC_MAX_TOKENS tokens, rank ALORA_STATIC_MAX_RANK: the
    only shape that reaches the array's last bytes), with adapter_on = NULL (every request has the adapter on),
    against the oracle; the device's free memory is the same before and after the second such call."""
    import torch
    T, rank = ab.STATIC_MAX_TOKENS, ab.STATIC_MAX_RANK
    P, S = [100, 0, 7], [T - 1500, 1000, 500]
    w, ad, b, _ = _case(5, P, S, [1, 1, 1], [100 + 50, 0, 7 + 499], rank)
    g = hp.GpuLayers(SHAPE, [dict(wqkv=w)], [[ad]], 16, 4)    # only holds the weights; the entry takes no context
    try:
        d = hp.DevBatch(b, "bf16")
        assert d.T == T
        mats = [hp.to_dev(getattr(ad, n), "bf16") for n in ("Aq", "Bq", "Ak", "Bk", "Av", "Bv")]
        got = torch.full((T, SHAPE.N), float("nan"), dtype=torch.bfloat16, device="cuda")
        _static_call(g, SHAPE, "bf16", d, g.keep[0]["wqkv"], ad, mats, None, got)
        torch.cuda.synchronize()
        free0 = torch.cuda.mem_get_info()[0]
        got.fill_(float("nan"))
        _static_call(g, SHAPE, "bf16", d, g.keep[0]["wqkv"], ad, mats, None, got)
        torch.cuda.synchronize()
        assert torch.cuda.mem_get_info()[0] == free0, "the call changed the amount of free device memory"
        want_o, gate = _oracle_qkv(oracle64, SHAPE, w, ad, b, [1, 1, 1])
        assert gate.sum() == T - 50 - 499
        hp.assert_close(hp.to_host(got), want_o, 2e-2, "largest admitted call against the oracle", block=SHAPE.head_dim)
    finally:
        g.close()


def test_static_scratch_limits_are_enforced():
    import torch
    z = torch.zeros(16, dtype=torch.int32, device="cuda")
    x = torch.zeros(16, dtype=torch.bfloat16, device="cuda")
    args = dict(dtype=ab.DTYPE_BF16, hidden=64, n_q=64, n_kv=32, d_hidden=x, d_wqkv=x, positions=z,
                query_start_loc=z, activation_offsets=z, adapter_on=None, rank=8, scale=1.0, Aq=x, Bq=x, Ak=x, Bk=x,
                Av=x, Bv=x, T=1, R=1, qkv=x)
    assert ab.alora_project_qkv_static(**{**args, "T": ab.STATIC_MAX_TOKENS + 1}) == 3   # ALORA_ERR_CAPACITY
    assert ab.alora_project_qkv_static(**{**args, "rank": ab.STATIC_MAX_RANK + 1}) == 3
    assert ab.alora_project_qkv_static(**{**args, "d_hidden": None}) == 1                 # ALORA_ERR_INVALID_ARG
    assert ab.alora_project_qkv_static(**{**args, "T": 0}) == 0

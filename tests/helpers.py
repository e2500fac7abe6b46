"""Shared plumbing of the GPU parity tests: upload a seeded workload, run the C-ABI entry points,
bring results back as numpy, and build the oracle's expectation from the same inputs."""
from __future__ import annotations

import numpy as np

from paper_2504_12397_b200 import binding as ab  # noqa: F401
from paper_2504_12397_b200 import workloads as wl
from paper_2504_12397_b200.device import DevBatch, GpuLayers, idev, to_dev, to_host  # noqa: F401


def rel_err(got: np.ndarray, want: np.ndarray) -> float:
    """Tensor-max-normalised error: max|got - want| / max|want|."""
    want = np.asarray(want, np.float64)
    got = np.asarray(got, np.float64)
    denom = np.abs(want).max() if want.size else 0.0
    return float(np.abs(got - want).max() / (denom if denom > 0 else 1.0)) if want.size else 0.0


def rel_err_elementwise(got: np.ndarray, want: np.ndarray) -> float:
    """Second measure: max over elements of |got - want| / (|want| + 1e-2 * rms(want)).  Every element is
    judged against its own magnitude, with a floor of one percent of the tensor's rms so that elements
    near zero do not divide by nothing."""
    want = np.asarray(want, np.float64)
    got = np.asarray(got, np.float64)
    if not want.size:
        return 0.0
    rms = float(np.sqrt(np.mean(want * want)))
    return float((np.abs(got - want) / (np.abs(want) + 1e-2 * (rms if rms > 0 else 1.0))).max())


def rel_err_blocks(got: np.ndarray, want: np.ndarray, block: int) -> float:
    """Third measure: the tensor-max-normalised error taken separately for every (row, block of `block`
    columns) -- one head of one token -- so that a head or a token of small magnitude cannot hide behind a
    large one elsewhere in the tensor.  Blocks whose expected values are all below 1e-3 of the tensor's
    maximum are normalised by that floor instead."""
    want = np.asarray(want, np.float64)
    got = np.asarray(got, np.float64)
    if not want.size:
        return 0.0
    T, N = want.shape
    assert N % block == 0
    w = np.abs(want).reshape(T, N // block, block).max(axis=2)
    d = np.abs(got - want).reshape(T, N // block, block).max(axis=2)
    floor = 1e-3 * np.abs(want).max()
    return float((d / np.maximum(w, floor if floor > 0 else 1.0)).max())


# Bounds of the three measures for bf16 results against the fp64 oracle.
# (1) Tensor-wide: the method's stated bound, 2e-2.
# (2) Elementwise, |d| / (|want| + 1e-2 rms): decided by the elements near zero, whose error does not shrink with
#     them.  Each bf16 rounding on the way (q/k/v rows, softmax probabilities, outputs; through a decoder layer
#     about ten of them) leaves noise of about 2^-9 / sqrt(3) of the tensor's rms, so a 5-sigma element of ten
#     stages is off by ~0.02 .. 0.04 rms and reads 2 .. 4 here (measured: up to 3.1 through a two-layer stack, 0.5
#     .. 1.7 for single kernels).  The stated bound (1) itself admits 2e-2 * max|want| ~ 0.1 rms, i.e. ~10 here.  The
#     bound sits between the two.  A wrong element (missing delta, wrong head or row) is off by O(rms): ~100.
# (3) Per (row, head): the same absolute error against a head's own maximum, which is 2 .. 3 sigma where the
#     tensor's is ~5 sigma: three times the stated bound.  Measured: up to 1.7e-2.
TOL_ELEMENTWISE_BF16 = 8.0
TOL_BLOCKS_BF16 = 6e-2


WORST = {}   # largest value of each measure seen in this session, per data type (printed by conftest at the end)


def assert_close(got, want, shape_or_tol, what: str = "", block: int = 0):
    """All parity assertions go through here: the stated tensor-wide bound, plus the elementwise and (when a
    block width is given) per-(row, head) measures.  Returns the three figures for reporting."""
    tol_ = shape_or_tol if isinstance(shape_or_tol, float) else tol(shape_or_tol)
    bf16 = tol_ > 1e-3
    e1 = rel_err(got, want)
    e2 = rel_err_elementwise(got, want)
    e3 = rel_err_blocks(got, want, block) if block else 0.0
    rec = WORST.setdefault("bf16" if bf16 else "fp32", [0.0, 0.0, 0.0])
    rec[0], rec[1], rec[2] = max(rec[0], e1), max(rec[1], e2), max(rec[2], e3)
    assert e1 <= tol_, f"{what}: max|d|/max|want| = {e1:.3e} > {tol_:g}"
    assert e2 <= (TOL_ELEMENTWISE_BF16 if bf16 else 1e-3), f"{what}: elementwise measure {e2:.3e}"
    if block:
        assert e3 <= (TOL_BLOCKS_BF16 if bf16 else 1e-4), f"{what}: per-(row, head) measure {e3:.3e}"
    return e1, e2, e3


def tol(shape: wl.LayerShape) -> float:
    # bf16: the method's stated bound; fp32: H-length fp32 dot products err by about sqrt(H) * 2^-24 ~ 1e-6
    # relative, taken with a tenfold margin
    return 2e-2 if shape.dtype == "bf16" else 1e-5


def full_sequence_batch(shape: wl.LayerShape, b: wl.Batch) -> wl.Batch:
    """The same requests with prefix ++ new tokens all presented as new tokens (positions from 0),
    same block tables: what a base prefill or a full-LoRA recompute is given."""
    R = b.R
    qsl = np.zeros(R + 1, np.int32)
    qsl[1:] = np.cumsum(b.seq_lens)
    pos = np.concatenate([np.arange(n, dtype=np.int32) for n in b.seq_lens])
    hid = np.concatenate([np.concatenate([b.prefix_hidden[r], b.hidden[b.query_start_loc[r]:b.query_start_loc[r + 1]]])
                          for r in range(R)])
    return wl.Batch(positions=pos, query_start_loc=qsl, seq_lens=b.seq_lens.copy(),
                    prefix_lens=np.zeros(R, np.int32), activation_offsets=b.activation_offsets.copy(),
                    adapter_ids=b.adapter_ids.copy(), block_tables=b.block_tables, num_pages=b.num_pages,
                    hidden=hid)


def prefix_only_batch(shape: wl.LayerShape, b: wl.Batch) -> wl.Batch:
    """Only the cached prefixes as new tokens of a base-model prefill (same block tables)."""
    R = b.R
    qsl = np.zeros(R + 1, np.int32)
    qsl[1:] = np.cumsum(b.prefix_lens)
    pos = np.concatenate([np.arange(n, dtype=np.int32) for n in b.prefix_lens] or [np.zeros(0, np.int32)])
    hid = np.concatenate(b.prefix_hidden) if R else np.zeros((0, shape.hidden), np.float32)
    return wl.Batch(positions=pos, query_start_loc=qsl, seq_lens=b.prefix_lens.copy(),
                    prefix_lens=np.zeros(R, np.int32), activation_offsets=np.zeros(R, np.int32),
                    adapter_ids=np.full(R, -1, np.int32), block_tables=b.block_tables, num_pages=b.num_pages,
                    hidden=hid)


def oracle_adapters(ads):
    from oracle import Adapter
    return [Adapter(a.rank, a.scale, a.Aq, a.Bq, a.Ak, a.Bk, a.Av, a.Bv) for a in ads]


def oracle_mlp_adapters(ads):
    from oracle import MlpAdapter
    return [MlpAdapter(a.rank, a.scale, a.Ag, a.Bg, a.Au, a.Bu, a.Ad, a.Bd) for a in ads]


def oracle_base_prefix(orc, shape, wqkv, b: wl.Batch, rope_theta: float = 0.0):
    """Base-model K/V of every request's prefix, from the prefix hidden states (Eq. 2); with a rotary base, keys as
    they would be cached (rotated by their positions)."""
    Ks, Vs = [], []
    for r in range(b.R):
        P = int(b.prefix_lens[r])
        if P == 0:
            Ks.append(None); Vs.append(None)
            continue
        qkv, _ = orc.project_qkv(b.prefix_hidden[r], wqkv, shape.Nq, shape.Nkv, np.arange(P), [0, P], [0], [-1], [])
        k = qkv[:, shape.Nq:shape.Nq + shape.Nkv]
        if rope_theta:
            k = orc.rope(k, np.arange(P), shape.n_kv_heads, shape.head_dim, rope_theta)
        Ks.append(k); Vs.append(qkv[:, shape.Nq + shape.Nkv:])
    return Ks, Vs


def oracle_block(orc, shape, wqkv, ads, b: wl.Batch, Ks, Vs, force_all=False, rope_theta: float = 0.0):
    return orc.attention_block(b.hidden, wqkv, shape.Nq, shape.Nkv, shape.n_q_heads, shape.n_kv_heads, shape.head_dim,
                               b.positions, b.query_start_loc, b.activation_offsets, b.adapter_ids,
                               oracle_adapters(ads), Ks, Vs, force_all=force_all, rope_theta=rope_theta)

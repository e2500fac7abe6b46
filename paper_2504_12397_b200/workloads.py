"""Seeded synthetic workloads shaped like the paper's multi-turn serving settings.

This module only *draws inputs*: weights, adapters, hidden states, request lengths, activation
offsets, block tables.  It contains none of the method's arithmetic and imports neither the CUDA
binding nor the CPU oracle, so both sides can be fed the same bits from it.

Distributions: W, A, B ~ N(0, 0.02^2), hidden states ~ N(0, 1), KV pages of 16 tokens handed out
from a pool either in order or through a seeded random permutation.  bf16 workloads round every
tensor to bf16 once here (round to nearest even) and hand out the rounded values as float32, so a
consumer that narrows them to bf16 loses nothing.
"""
from __future__ import annotations

from dataclasses import dataclass, field
from typing import List, Optional, Sequence

import numpy as np


def bf16_round(a: np.ndarray) -> np.ndarray:
    """Round float32 values to the nearest bf16 (ties to even); result is float32."""
    a = np.ascontiguousarray(a, dtype=np.float32)
    u = a.view(np.uint32).astype(np.uint64)
    u = (u + 0x7FFF + ((u >> 16) & 1)) & 0xFFFF0000
    return u.astype(np.uint32).view(np.float32).reshape(a.shape)


def bf16_bits(a: np.ndarray) -> np.ndarray:
    """uint16 bit patterns of float32 values that are exactly representable in bf16."""
    a = np.ascontiguousarray(a, dtype=np.float32)
    return (a.view(np.uint32) >> 16).astype(np.uint16).reshape(a.shape)


def bf16_from_bits(b: np.ndarray) -> np.ndarray:
    """float32 values of bf16 bit patterns."""
    b = np.ascontiguousarray(b, dtype=np.uint16)
    return (b.astype(np.uint32) << 16).view(np.float32).reshape(b.shape)


@dataclass(frozen=True)
class LayerShape:
    hidden: int
    n_q_heads: int
    n_kv_heads: int
    head_dim: int
    page_size: int = 16
    dtype: str = "bf16"  # "bf16" | "fp32"
    intermediate: int = 0

    @property
    def Nq(self):
        return self.n_q_heads * self.head_dim

    @property
    def Nkv(self):
        return self.n_kv_heads * self.head_dim

    @property
    def N(self):
        return self.Nq + 2 * self.Nkv

    @property
    def group(self):
        return self.n_q_heads // self.n_kv_heads


TINY = LayerShape(hidden=256, n_q_heads=4, n_kv_heads=2, head_dim=64, dtype="fp32", intermediate=512)
SHAPE_8B = LayerShape(hidden=4096, n_q_heads=32, n_kv_heads=8, head_dim=128, dtype="bf16",
                      intermediate=14336)


@dataclass
class AdapterWeights:
    rank: int
    scale: float
    Aq: np.ndarray
    Bq: np.ndarray
    Ak: np.ndarray
    Bk: np.ndarray
    Av: np.ndarray
    Bv: np.ndarray


@dataclass
class MlpAdapterWeights:
    """The low-rank pairs of one adapter on the MLP block: gate, up ([r, H] / [I, r]) and down ([r, I] / [H, r])."""
    rank: int
    scale: float
    Ag: np.ndarray
    Bg: np.ndarray
    Au: np.ndarray
    Bu: np.ndarray
    Ad: np.ndarray
    Bd: np.ndarray


@dataclass
class Batch:
    """A ragged batch of new tokens on top of per-request cached prefixes."""
    positions: np.ndarray            # [T] int32, position of each new token in its sequence
    query_start_loc: np.ndarray      # [R+1] int32
    seq_lens: np.ndarray             # [R] int32, prefix + new tokens
    prefix_lens: np.ndarray          # [R] int32
    activation_offsets: np.ndarray   # [R] int32
    adapter_ids: np.ndarray          # [R] int32, -1 = base model
    block_tables: np.ndarray         # [R, max_blocks] int32 (unused entries 0)
    num_pages: int
    hidden: Optional[np.ndarray] = None          # [T, H] float32 (already rounded for bf16)
    prefix_hidden: Optional[List[np.ndarray]] = None  # per request [P_r, H], or None

    @property
    def T(self):
        return int(self.query_start_loc[-1])

    @property
    def R(self):
        return len(self.seq_lens)


def _round(a, dtype):
    a = a.astype(np.float32)
    return bf16_round(a) if dtype == "bf16" else a


def make_wqkv(shape: LayerShape, rng: np.random.Generator) -> np.ndarray:
    return _round(rng.normal(0.0, 0.02, (shape.N, shape.hidden)), shape.dtype)


def make_adapter(shape: LayerShape, rank: int, rng: np.random.Generator, scale: float = 1.0,
                 zero_b: bool = False) -> AdapterWeights:
    def A():
        return _round(rng.normal(0.0, 0.02, (rank, shape.hidden)), shape.dtype)

    def B(n):
        m = rng.normal(0.0, 0.02, (n, rank))
        return _round(np.zeros_like(m) if zero_b else m, shape.dtype)

    return AdapterWeights(rank, scale, A(), B(shape.Nq), A(), B(shape.Nkv), A(), B(shape.Nkv))


def make_mlp_adapter(shape: LayerShape, rank: int, rng: np.random.Generator, scale: float = 1.0,
                     zero_b: bool = False) -> MlpAdapterWeights:
    """Random-weight MLP adapter with the distribution of the q/k/v ones (N(0, 0.02^2), rounded to the layer dtype)."""
    H, I = shape.hidden, shape.intermediate

    def A(k):
        return _round(rng.normal(0.0, 0.02, (rank, k)), shape.dtype)

    def B(n):
        m = rng.normal(0.0, 0.02, (n, rank))
        return _round(np.zeros_like(m) if zero_b else m, shape.dtype)

    return MlpAdapterWeights(rank, scale, A(H), B(I), A(H), B(I), A(I), B(H))


def make_stack_weights(shape: LayerShape, rng: np.random.Generator) -> dict:
    """One decoder layer's base weights: fused qkv, o_proj, fused gate/up, down, two norm gains."""
    H, I = shape.hidden, shape.intermediate
    return dict(
        wqkv=make_wqkv(shape, rng),
        wo=_round(rng.normal(0.0, 0.02, (H, shape.Nq)), shape.dtype),
        wgate_up=_round(rng.normal(0.0, 0.02, (2 * I, H)), shape.dtype),
        wdown=_round(rng.normal(0.0, 0.02, (H, I)), shape.dtype),
        norm_attn=_round(1.0 + 0.1 * rng.normal(0.0, 1.0, H), shape.dtype),
        norm_mlp=_round(1.0 + 0.1 * rng.normal(0.0, 1.0, H), shape.dtype),
    )


def make_batch(shape: LayerShape, prefix_lens: Sequence[int], new_lens: Sequence[int],
               adapter_ids: Sequence[int], rng: np.random.Generator,
               activation_offsets: Optional[Sequence[int]] = None, shuffle_pages: bool = False,
               spare_pages: int = 3, with_hidden: bool = True, with_prefix_hidden: bool = False) -> Batch:
    """Lay out R requests: request r has prefix_lens[r] cached positions and new_lens[r] new tokens.

    Every request gets ceil((prefix+new)/page) private pages out of a pool that also holds
    `spare_pages` pages owned by nobody (canaries).  activation_offsets defaults to the prefix length.
    """
    prefix_lens = np.asarray(prefix_lens, np.int32)
    new_lens = np.asarray(new_lens, np.int32)
    R = len(prefix_lens)
    seq_lens = prefix_lens + new_lens
    qsl = np.zeros(R + 1, np.int32)
    qsl[1:] = np.cumsum(new_lens)
    T = int(qsl[-1])
    positions = np.concatenate(
        [np.arange(prefix_lens[r], seq_lens[r], dtype=np.int32) for r in range(R)]
        or [np.zeros(0, np.int32)])
    ps = shape.page_size
    blocks = (seq_lens + ps - 1) // ps
    max_blocks = max(1, int(blocks.max()) if R else 1)
    num_pages = int(blocks.sum()) + spare_pages
    order = rng.permutation(num_pages) if shuffle_pages else np.arange(num_pages)
    bt = np.zeros((R, max_blocks), np.int32)
    nxt = 0
    for r in range(R):
        bt[r, :blocks[r]] = order[nxt:nxt + blocks[r]]
        nxt += int(blocks[r])
    a_req = prefix_lens.copy() if activation_offsets is None else np.asarray(activation_offsets, np.int32)
    hidden = _round(rng.normal(0.0, 1.0, (T, shape.hidden)), shape.dtype) if with_hidden else None
    ph = None
    if with_prefix_hidden:
        ph = [_round(rng.normal(0.0, 1.0, (int(p), shape.hidden)), shape.dtype) for p in prefix_lens]
    return Batch(positions=positions, query_start_loc=qsl, seq_lens=seq_lens.astype(np.int32),
                 prefix_lens=prefix_lens, activation_offsets=a_req.astype(np.int32),
                 adapter_ids=np.asarray(adapter_ids, np.int32), block_tables=bt, num_pages=num_pages,
                 hidden=hidden, prefix_hidden=ph)


def random_kv_pool(shape: LayerShape, num_pages: int, rng: np.random.Generator) -> np.ndarray:
    """A pool [pages, 2, Hkv, page, hd] filled with N(0,1) values (rounded for bf16): stands in for a
    base-model cache when the base prefill itself is not the thing under test."""
    a = rng.standard_normal((num_pages, 2, shape.n_kv_heads, shape.page_size, shape.head_dim),
                            dtype=np.float32)
    return _round(a, shape.dtype)


# ---- the five named configurations --------------------------------------------------------------

@dataclass
class Workload:
    name: str
    shape: LayerShape
    wqkv: np.ndarray
    adapters: List[AdapterWeights]
    batch: Batch
    seed: int
    notes: str = ""
    extra: dict = field(default_factory=dict)


def config1(seed: int = 0) -> Workload:
    """Tiny fp32 layer: 1 request, 64 cached positions, activation at 64, 16 new tokens, rank 8."""
    rng = np.random.default_rng(seed)
    w = make_wqkv(TINY, rng)
    ad = [make_adapter(TINY, 8, rng)]
    b = make_batch(TINY, [64], [16], [0], rng, with_prefix_hidden=True)
    return Workload("config1_tiny_fp32", TINY, w, ad, b, seed)


def config2(seed: int = 2, requests: int = 8, prefix: int = 4096, suffix: int = 256,
            shape: LayerShape = SHAPE_8B, rank: int = 32, activation_shift: int = 0,
            shuffle_pages: bool = False) -> Workload:
    """One 8B-shape bf16 layer: 8 requests x (4096 cached + 256 new at the activation offset).  With
    `activation_shift` > 0 the adapter activates that many tokens INTO the new chunk: the call prefills an
    uncached tail of the context with the base weights and the invocation with the adapter (the paper's second
    regime: the context is not all cached yet when the adapter is invoked)."""
    rng = np.random.default_rng(seed)
    w = make_wqkv(shape, rng)
    ad = [make_adapter(shape, rank, rng)]
    b = make_batch(shape, [prefix] * requests, [suffix] * requests, [0] * requests, rng,
                   activation_offsets=[prefix + activation_shift] * requests, shuffle_pages=shuffle_pages)
    return Workload("config2_8b_layer", shape, w, ad, b, seed)


def config3(seed: int = 3, requests: int = 32, shape: LayerShape = SHAPE_8B,
            prefix_range=(512, 16384), suffix_range=(16, 512), ranks=(8, 16, 32, 64)) -> Workload:
    """Ragged multi-adapter batch: requests drawn over four adapters of different ranks, prefix and
    suffix lengths uniform in the given ranges, shuffled pages."""
    rng = np.random.default_rng(seed)
    w = make_wqkv(shape, rng)
    ad = [make_adapter(shape, r, rng) for r in ranks]
    P = rng.integers(prefix_range[0], prefix_range[1] + 1, requests)
    S = rng.integers(suffix_range[0], suffix_range[1] + 1, requests)
    ids = rng.integers(0, len(ranks), requests)
    b = make_batch(shape, P, S, ids, rng, shuffle_pages=True)
    return Workload("config3_ragged_multi_adapter", shape, w, ad, b, seed)


def config5(seed: int = 5, requests: int = 64, shape: LayerShape = SHAPE_8B,
            ctx_range=(1024, 32768), n_adapters: int = 4, rank: int = 32) -> Workload:
    """Decode batch: one new token per request, context lengths uniform in ctx_range, requests mixing
    the base model (-1) and n_adapters rank-32 adapters, every adapter already active."""
    rng = np.random.default_rng(seed)
    w = make_wqkv(shape, rng)
    ad = [make_adapter(shape, rank, rng) for _ in range(n_adapters)]
    ctx = rng.integers(ctx_range[0], ctx_range[1] + 1, requests)
    ids = rng.integers(-1, n_adapters, requests)
    # the cache holds ctx-1 positions and the step adds the token at position ctx-1
    b = make_batch(shape, ctx - 1, [1] * requests, ids, rng, shuffle_pages=True,
                   activation_offsets=np.maximum(ctx - 1 - rng.integers(0, 64, requests), 0))
    return Workload("config5_decode", shape, w, ad, b, seed)

"""Shared plumbing of the GPU parity tests: upload a seeded workload, run the C-ABI entry points,
bring results back as numpy, and build the oracle's expectation from the same inputs."""
from __future__ import annotations

import numpy as np

from paper_2504_12397_b200 import binding as ab
from paper_2504_12397_b200 import workloads as wl


def rel_err(got: np.ndarray, want: np.ndarray) -> float:
    """Tensor-max-normalised error: max|got - want| / max|want|."""
    want = np.asarray(want, np.float64)
    got = np.asarray(got, np.float64)
    denom = np.abs(want).max()
    return float(np.abs(got - want).max() / (denom if denom > 0 else 1.0))


def tol(shape: wl.LayerShape) -> float:
    # bf16: the method's stated bound; fp32: H-length fp32 dot products err by about sqrt(H) * 2^-24 ~ 1e-6
    # relative, taken with a tenfold margin
    return 2e-2 if shape.dtype == "bf16" else 1e-5


def to_dev(a: np.ndarray, dtype: str):
    import torch
    t = torch.from_numpy(np.ascontiguousarray(a, dtype=np.float32)).cuda()
    return t.to(torch.bfloat16).contiguous() if dtype == "bf16" else t.contiguous()


def to_host(t) -> np.ndarray:
    import torch
    return t.detach().to(torch.float32).cpu().numpy()


def idev(a):
    import torch
    return torch.from_numpy(np.ascontiguousarray(a, dtype=np.int32)).cuda()


class GpuLayers:
    """A context plus device copies of weights/adapters for `n_layers` layers of one shape."""

    def __init__(self, shape: wl.LayerShape, layer_weights, adapters_per_layer, max_tokens, max_requests,
                 n_adapters=None):
        import torch
        self.shape = shape
        self.n_layers = len(layer_weights)
        n_ad = n_adapters if n_adapters is not None else max([len(a) for a in adapters_per_layer] + [1])
        max_rank = max([a.rank for per in adapters_per_layer for a in per] + [8])
        self.cfg = ab.make_config(
            hidden=shape.hidden, n_q_heads=shape.n_q_heads, n_kv_heads=shape.n_kv_heads, head_dim=shape.head_dim,
            page_size=shape.page_size, n_layers=self.n_layers, intermediate=shape.intermediate if "wo" in layer_weights[0] else 0,
            max_adapters=n_ad, max_rank=max_rank, dtype=ab.DTYPE_BF16 if shape.dtype == "bf16" else ab.DTYPE_FP32,
            max_tokens=max_tokens, max_requests=max_requests)
        self.ctx = ab.alora_create(self.cfg)
        self.keep = []
        for l, lw in enumerate(layer_weights):
            dev = {k: to_dev(v, shape.dtype) for k, v in lw.items()}
            self.keep.append(dev)
            ab.alora_set_layer_weights(self.ctx, l, dev["wqkv"], dev.get("wo"), dev.get("wgate_up"), dev.get("wdown"),
                                       dev.get("norm_attn"), dev.get("norm_mlp"))
            for i, a in enumerate(adapters_per_layer[l]):
                mats = [to_dev(getattr(a, n), shape.dtype) for n in ("Aq", "Bq", "Ak", "Bk", "Av", "Bv")]
                ab.alora_register_adapter(self.ctx, i, l, a.rank, a.scale, *mats)
        torch.cuda.synchronize()
        self.torch_dtype = torch.bfloat16 if shape.dtype == "bf16" else torch.float32

    def close(self):
        if self.ctx:
            ab.alora_destroy(self.ctx)
            self.ctx = None

    def new_pool(self, num_pages, fill=None):
        import torch
        s = self.shape
        if fill is None:
            return torch.zeros((num_pages, 2, s.n_kv_heads, s.page_size, s.head_dim), dtype=self.torch_dtype, device="cuda")
        return to_dev(fill, s.dtype)

    def empty(self, *shape):
        import torch
        return torch.empty(shape, dtype=self.torch_dtype, device="cuda")

    def status(self) -> int:
        return ab.alora_get_status(self.ctx)


class DevBatch:
    def __init__(self, b: wl.Batch, dtype: str):
        self.b = b
        self.positions = idev(b.positions)
        self.qsl = idev(b.query_start_loc)
        self.seq_lens = idev(b.seq_lens)
        self.a_req = idev(b.activation_offsets)
        self.ids = idev(b.adapter_ids)
        self.bt = idev(b.block_tables)
        self.max_blocks = b.block_tables.shape[1]
        self.hidden = to_dev(b.hidden, dtype) if b.hidden is not None else None
        self.T, self.R = b.T, b.R


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


def oracle_base_prefix(orc, shape, wqkv, b: wl.Batch):
    """Base-model K/V of every request's prefix, from the prefix hidden states (Eq. 2)."""
    Ks, Vs = [], []
    for r in range(b.R):
        P = int(b.prefix_lens[r])
        if P == 0:
            Ks.append(None); Vs.append(None)
            continue
        qkv, _ = orc.project_qkv(b.prefix_hidden[r], wqkv, shape.Nq, shape.Nkv, np.arange(P), [0, P], [0], [-1], [])
        Ks.append(qkv[:, shape.Nq:shape.Nq + shape.Nkv]); Vs.append(qkv[:, shape.Nq + shape.Nkv:])
    return Ks, Vs


def oracle_block(orc, shape, wqkv, ads, b: wl.Batch, Ks, Vs, force_all=False):
    return orc.attention_block(b.hidden, wqkv, shape.Nq, shape.Nkv, shape.n_q_heads, shape.n_kv_heads, shape.head_dim,
                               b.positions, b.query_start_loc, b.activation_offsets, b.adapter_ids,
                               oracle_adapters(ads), Ks, Vs, force_all=force_all)

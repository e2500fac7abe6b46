"""Device-memory plumbing around the C-ABI binding: a context with device copies of one or more layers'
weights and adapters, and a ragged batch uploaded to the device.  PyTorch is used for allocation and
host <-> device copies only; no arithmetic of the method happens here."""
from __future__ import annotations

import numpy as np

from . import binding as ab
from . import workloads as wl


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
                 n_adapters=None, rope_theta: float = 0.0, mlp_adapters_per_layer=None):
        import torch
        self.shape = shape
        self.n_layers = len(layer_weights)
        n_ad = n_adapters if n_adapters is not None else max([len(a) for a in adapters_per_layer] + [1])
        max_rank = max([a.rank for per in adapters_per_layer for a in per] + [8])
        if mlp_adapters_per_layer:
            max_rank = max([max_rank] + [a.rank for per in mlp_adapters_per_layer for a in per if a is not None])
        self.cfg = ab.make_config(
            hidden=shape.hidden, n_q_heads=shape.n_q_heads, n_kv_heads=shape.n_kv_heads, head_dim=shape.head_dim,
            page_size=shape.page_size, n_layers=self.n_layers, intermediate=shape.intermediate if "wo" in layer_weights[0] else 0,
            max_adapters=n_ad, max_rank=max_rank, dtype=ab.DTYPE_BF16 if shape.dtype == "bf16" else ab.DTYPE_FP32,
            max_tokens=max_tokens, max_requests=max_requests, rope_theta=rope_theta)
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
            # MLP parts (optional; None = this adapter has none on this layer), after the q/k/v parts they extend
            for i, a in enumerate(mlp_adapters_per_layer[l] if mlp_adapters_per_layer else []):
                if a is None:
                    continue
                mats = [to_dev(getattr(a, n), shape.dtype) for n in ("Ag", "Bg", "Au", "Bu", "Ad", "Bd")]
                ab.alora_register_mlp_adapter(self.ctx, i, l, a.rank, a.scale, *mats)
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
    """Device copies of one ragged batch's integer arrays and hidden states."""

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

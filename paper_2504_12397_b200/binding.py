"""ctypes binding of libalora_b200.so: the same entry points as include/alora.h, argument marshalling only.

Tensors are torch CUDA tensors (used purely as device-memory handles: `data_ptr()`), streams are
torch streams or raw integers.  Nothing here computes; without the compiled library every call
fails with AloraLibraryMissing, and without a CUDA device alora_create fails.  There is no fallback.
"""
from __future__ import annotations

import ctypes as C
import os
from typing import Optional, Sequence

_HERE = os.path.dirname(os.path.abspath(__file__))
LIB_PATH = os.path.join(_HERE, "libalora_b200.so")

ALORA_OK = 0
DTYPE_BF16, DTYPE_FP32 = 0, 1
MODE_ALORA, MODE_FULL_LORA, MODE_BASE = 0, 1, 2


class AloraLibraryMissing(RuntimeError):
    pass


class AloraError(RuntimeError):
    def __init__(self, status: int, where: str, detail: str = ""):
        self.status = status
        super().__init__(f"{where}: status {status} ({status_string(status)}) {detail}".strip())


class alora_config(C.Structure):
    _fields_ = [(n, C.c_int32) for n in (
        "hidden", "n_q_heads", "n_kv_heads", "head_dim", "page_size", "n_layers", "intermediate",
        "max_adapters", "max_rank", "dtype", "device", "max_tokens", "max_requests")] + [
        ("rms_eps", C.c_float), ("rope_theta", C.c_float), ("softmax_scale", C.c_float)]


_lib = None
_VP, _IP, _I = C.c_void_p, C.c_void_p, C.c_int


def _signatures(lib):
    lib.alora_create.argtypes = [C.POINTER(alora_config), C.POINTER(_VP)]
    lib.alora_destroy.argtypes = [_VP]
    lib.alora_set_layer_weights.argtypes = [_VP, _I] + [_VP] * 6
    lib.alora_register_adapter.argtypes = [_VP, _I, _I, _I, C.c_float] + [_VP] * 6 + [_VP]
    lib.alora_register_mlp_adapter.argtypes = [_VP, _I, _I, _I, C.c_float] + [_VP] * 6 + [_VP]
    lib.alora_register_mlp_adapter.restype = C.c_int
    lib.alora_validate_batch.argtypes = [C.POINTER(alora_config)] + [_IP] * 6 + [_I] * 4
    lib.alora_batch_metadata.argtypes = [_VP, _I] + [_IP] * 6 + [_I] * 4 + [_IP] * 3 + [_VP]
    lib.alora_project_qkv.argtypes = [_VP, _I, _I, _VP] + [_IP] * 5 + [_I, _I, _VP, _VP]
    lib.alora_kv_append.argtypes = [_VP, _VP] + [_IP] * 4 + [_I] * 4 + [_VP, _VP]
    lib.alora_attend.argtypes = [_VP, _VP] + [_IP] * 3 + [_VP, _IP] + [_I] * 4 + [_VP, _VP]
    lib.alora_prefill_layer.argtypes = [_VP, _I, _VP] + [_IP] * 5 + [_VP, _IP] + [_I] * 4 + [_VP, _VP]
    lib.alora_decode_step.argtypes = [_VP, _I, _VP] + [_IP] * 4 + [_VP, _IP] + [_I] * 3 + [_VP, _VP]
    lib.alora_full_lora_prefill_layer.argtypes = [_VP, _I, _VP] + [_IP] * 4 + [_VP, _IP] + [_I] * 4 + [_VP, _VP]
    lib.alora_forward_stack.argtypes = [_VP, _I, _VP] + [_IP] * 5 + [C.POINTER(_VP), _IP] + [_I] * 4 + [_VP, _VP]
    lib.alora_get_status.argtypes = [_VP, _VP, C.POINTER(C.c_int32)]
    lib.alora_status_string.argtypes = [_I]
    lib.alora_status_string.restype = C.c_char_p
    lib.alora_last_cuda_error.argtypes = [_VP]
    lib.alora_last_cuda_error.restype = C.c_char_p
    lib.alora_launch_count.argtypes = [_VP]
    lib.alora_launch_count.restype = C.c_int64
    lib.alora_profile_enable.argtypes = [_VP, _I]
    lib.alora_profile_read.argtypes = [_VP, C.POINTER(C.c_double), C.POINTER(C.c_int64)]
    for name in ("alora_profile_enable", "alora_profile_read", "alora_create", "alora_destroy", "alora_set_layer_weights", "alora_register_adapter",
                 "alora_validate_batch", "alora_batch_metadata", "alora_project_qkv", "alora_kv_append",
                 "alora_attend", "alora_prefill_layer", "alora_decode_step",
                 "alora_full_lora_prefill_layer", "alora_forward_stack", "alora_get_status"):
        getattr(lib, name).restype = C.c_int


def load_library():
    """Load libalora_b200.so (built by paper_2504_12397_b200.build); raises if it is not there."""
    global _lib
    if _lib is None:
        if not os.path.exists(LIB_PATH):
            raise AloraLibraryMissing(
                f"{LIB_PATH} not found: run `python -m paper_2504_12397_b200.build` (needs nvcc). "
                "There is no CPU fallback.")
        lib = C.CDLL(LIB_PATH)
        _signatures(lib)
        _lib = lib
    return _lib


def status_string(status: int) -> str:
    return load_library().alora_status_string(int(status)).decode()


def _ptr(t) -> Optional[int]:
    if t is None:
        return None
    if isinstance(t, int):
        return t
    return t.data_ptr()


def _stream(s) -> Optional[int]:
    if s is None:
        import torch
        return torch.cuda.current_stream().cuda_stream
    if isinstance(s, int):
        return s
    return s.cuda_stream


def _check(ctx, rc: int, where: str):
    if rc != ALORA_OK:
        detail = ""
        if ctx is not None and rc == 5:
            detail = load_library().alora_last_cuda_error(ctx).decode()
        raise AloraError(rc, where, detail)


def make_config(**kw) -> alora_config:
    cfg = alora_config()
    defaults = dict(page_size=16, n_layers=1, intermediate=0, max_adapters=1, max_rank=64, dtype=DTYPE_BF16,
                    device=0, max_tokens=1, max_requests=1, rms_eps=1e-5, rope_theta=0.0, softmax_scale=0.0)
    defaults.update(kw)
    for k, v in defaults.items():
        setattr(cfg, k, v)
    return cfg


def alora_create(cfg: alora_config) -> int:
    lib = load_library()
    out = _VP()
    _check(None, lib.alora_create(C.byref(cfg), C.byref(out)), "alora_create")
    return out.value


def alora_destroy(ctx: int) -> None:
    _check(None, load_library().alora_destroy(ctx), "alora_destroy")


def alora_set_layer_weights(ctx, layer, wqkv, wo=None, wgate_up=None, wdown=None, norm_attn=None, norm_mlp=None):
    rc = load_library().alora_set_layer_weights(ctx, layer, _ptr(wqkv), _ptr(wo), _ptr(wgate_up), _ptr(wdown),
                                                _ptr(norm_attn), _ptr(norm_mlp))
    _check(ctx, rc, "alora_set_layer_weights")


def alora_register_adapter(ctx, adapter_id, layer, rank, scale, Aq, Bq, Ak, Bk, Av, Bv, stream=None):
    rc = load_library().alora_register_adapter(ctx, adapter_id, layer, rank, scale, _ptr(Aq), _ptr(Bq), _ptr(Ak),
                                               _ptr(Bk), _ptr(Av), _ptr(Bv), _stream(stream))
    _check(ctx, rc, "alora_register_adapter")


def alora_register_mlp_adapter(ctx, adapter_id, layer, rank, scale, Ag, Bg, Au, Bu, Ad, Bd, stream=None):
    rc = load_library().alora_register_mlp_adapter(ctx, adapter_id, layer, rank, scale, _ptr(Ag), _ptr(Bg), _ptr(Au),
                                                   _ptr(Bu), _ptr(Ad), _ptr(Bd), _stream(stream))
    _check(ctx, rc, "alora_register_mlp_adapter")


def alora_selftest_claim_order(grid, n_shrink, n_row_tiles, n_col_tiles, resident_slots, high_blocks_first=True,
                               static_order=False) -> bool:
    """Host-only model of the projection launch's item order; True when every item completes."""
    lib = load_library()
    lib.alora_selftest_claim_order.argtypes = [_I] * 7 + [C.POINTER(C.c_int)]
    lib.alora_selftest_claim_order.restype = C.c_int
    done = C.c_int(-1)
    rc = lib.alora_selftest_claim_order(grid, n_shrink, n_row_tiles, n_col_tiles, resident_slots,
                                        int(bool(high_blocks_first)), int(bool(static_order)), C.byref(done))
    if rc != 0:
        raise AloraError(rc, "alora_selftest_claim_order", "")
    return done.value == 1


def alora_validate_batch(cfg: alora_config, positions, activation_offsets, adapter_ids, query_start_loc,
                         seq_lens, block_tables, num_pages: int) -> int:
    """Host-side check; arguments are numpy int32 arrays (block_tables 2-D).  Returns the status code."""
    import numpy as np

    def hp(a):
        if a is None:
            return None, None
        a = np.ascontiguousarray(a, dtype=np.int32)
        return a, a.ctypes.data

    pos, p0 = hp(positions); ar, p1 = hp(activation_offsets); ids, p2 = hp(adapter_ids)
    qsl, p3 = hp(query_start_loc); sl, p4 = hp(seq_lens); bt, p5 = hp(block_tables)
    max_blocks = 0 if bt is None else bt.shape[1]
    return load_library().alora_validate_batch(C.byref(cfg), p0, p1, p2, p3, p4, p5, max_blocks, num_pages,
                                               len(pos), len(sl))


def alora_batch_metadata(ctx, mode, positions, activation_offsets, adapter_ids, query_start_loc, seq_lens,
                         block_tables, max_blocks, num_pages, T, R, token_request=None, row_adapter=None,
                         slot_mapping=None, stream=None):
    rc = load_library().alora_batch_metadata(ctx, mode, _ptr(positions), _ptr(activation_offsets), _ptr(adapter_ids),
                                             _ptr(query_start_loc), _ptr(seq_lens), _ptr(block_tables), max_blocks,
                                             num_pages, T, R, _ptr(token_request), _ptr(row_adapter),
                                             _ptr(slot_mapping), _stream(stream))
    _check(ctx, rc, "alora_batch_metadata")


def alora_project_qkv(ctx, layer, mode, hidden, positions, activation_offsets, adapter_ids, query_start_loc,
                      seq_lens, T, R, qkv, stream=None):
    rc = load_library().alora_project_qkv(ctx, layer, mode, _ptr(hidden), _ptr(positions), _ptr(activation_offsets),
                                          _ptr(adapter_ids), _ptr(query_start_loc), _ptr(seq_lens), T, R, _ptr(qkv),
                                          _stream(stream))
    _check(ctx, rc, "alora_project_qkv")


def alora_kv_append(ctx, qkv, positions, query_start_loc, seq_lens, block_tables, max_blocks, num_pages, T, R,
                    paged_kv, stream=None):
    rc = load_library().alora_kv_append(ctx, _ptr(qkv), _ptr(positions), _ptr(query_start_loc), _ptr(seq_lens),
                                        _ptr(block_tables), max_blocks, num_pages, T, R, _ptr(paged_kv),
                                        _stream(stream))
    _check(ctx, rc, "alora_kv_append")


def alora_attend(ctx, qkv, positions, query_start_loc, seq_lens, paged_kv, block_tables, max_blocks, num_pages,
                 T, R, attn_out, stream=None):
    rc = load_library().alora_attend(ctx, _ptr(qkv), _ptr(positions), _ptr(query_start_loc), _ptr(seq_lens),
                                     _ptr(paged_kv), _ptr(block_tables), max_blocks, num_pages, T, R,
                                     _ptr(attn_out), _stream(stream))
    _check(ctx, rc, "alora_attend")


def alora_prefill_layer(ctx, layer, hidden, positions, activation_offsets, adapter_ids, query_start_loc, seq_lens,
                        paged_kv, block_tables, max_blocks, num_pages, T, R, attn_out, stream=None):
    rc = load_library().alora_prefill_layer(ctx, layer, _ptr(hidden), _ptr(positions), _ptr(activation_offsets),
                                            _ptr(adapter_ids), _ptr(query_start_loc), _ptr(seq_lens),
                                            _ptr(paged_kv), _ptr(block_tables), max_blocks, num_pages, T, R,
                                            _ptr(attn_out), _stream(stream))
    _check(ctx, rc, "alora_prefill_layer")


def alora_decode_step(ctx, layer, hidden, positions, activation_offsets, adapter_ids, seq_lens, paged_kv,
                      block_tables, max_blocks, num_pages, R, attn_out, stream=None):
    rc = load_library().alora_decode_step(ctx, layer, _ptr(hidden), _ptr(positions), _ptr(activation_offsets),
                                          _ptr(adapter_ids), _ptr(seq_lens), _ptr(paged_kv), _ptr(block_tables),
                                          max_blocks, num_pages, R, _ptr(attn_out), _stream(stream))
    _check(ctx, rc, "alora_decode_step")


def alora_full_lora_prefill_layer(ctx, layer, hidden, positions, adapter_ids, query_start_loc, seq_lens, paged_kv,
                                  block_tables, max_blocks, num_pages, T, R, attn_out, stream=None):
    rc = load_library().alora_full_lora_prefill_layer(ctx, layer, _ptr(hidden), _ptr(positions), _ptr(adapter_ids),
                                                      _ptr(query_start_loc), _ptr(seq_lens), _ptr(paged_kv),
                                                      _ptr(block_tables), max_blocks, num_pages, T, R,
                                                      _ptr(attn_out), _stream(stream))
    _check(ctx, rc, "alora_full_lora_prefill_layer")


def alora_forward_stack(ctx, mode, hidden_in, positions, activation_offsets, adapter_ids, query_start_loc,
                        seq_lens, paged_kv_layers: Sequence, block_tables, max_blocks, num_pages, T, R, hidden_out,
                        stream=None):
    arr = (_VP * len(paged_kv_layers))(*[_ptr(p) for p in paged_kv_layers])
    rc = load_library().alora_forward_stack(ctx, mode, _ptr(hidden_in), _ptr(positions), _ptr(activation_offsets),
                                            _ptr(adapter_ids), _ptr(query_start_loc), _ptr(seq_lens), arr,
                                            _ptr(block_tables), max_blocks, num_pages, T, R, _ptr(hidden_out),
                                            _stream(stream))
    _check(ctx, rc, "alora_forward_stack")


def alora_decode_stack(ctx, hidden_in, positions, activation_offsets, adapter_ids, seq_lens, paged_kv_layers: Sequence,
                       block_tables, max_blocks, num_pages, R, hidden_out, stream=None):
    arr = (_VP * len(paged_kv_layers))(*[_ptr(p) for p in paged_kv_layers])
    f = load_library().alora_decode_stack
    f.argtypes = [C.c_void_p] + [_VP] * 5 + [C.POINTER(_VP), _VP, _I, _I, _I, _VP, _VP]
    f.restype = C.c_int
    _check(ctx, f(ctx, _ptr(hidden_in), _ptr(positions), _ptr(activation_offsets), _ptr(adapter_ids), _ptr(seq_lens), arr,
                  _ptr(block_tables), max_blocks, num_pages, R, _ptr(hidden_out), _stream(stream)), "alora_decode_stack")


def alora_get_status(ctx, stream=None) -> int:
    out = C.c_int32(0)
    _check(ctx, load_library().alora_get_status(ctx, _stream(stream), C.byref(out)), "alora_get_status")
    return int(out.value)


def alora_prefix_groups(ctx, R, group_first, shared_keys, stream=None) -> None:
    f = load_library().alora_prefix_groups
    f.argtypes = [C.c_void_p, _I, _VP, _VP, _VP]
    f.restype = C.c_int
    _check(ctx, f(ctx, R, _ptr(group_first), _ptr(shared_keys), _stream(stream)), "alora_prefix_groups")


def alora_cow_tail_pages(ctx, query_start_loc, seq_lens, block_tables, max_blocks, num_pages, R, fresh_pages, paged_kv,
                         stream=None) -> None:
    f = load_library().alora_cow_tail_pages
    f.argtypes = [C.c_void_p, _VP, _VP, _VP, _I, _I, _I, _VP, _VP, _VP]
    f.restype = C.c_int
    _check(ctx, f(ctx, _ptr(query_start_loc), _ptr(seq_lens), _ptr(block_tables), max_blocks, num_pages, R,
                  _ptr(fresh_pages), _ptr(paged_kv), _stream(stream)), "alora_cow_tail_pages")


def alora_selftest_wait_timeout(ctx, limit_cycles: int, stream=None) -> None:
    f = load_library().alora_selftest_wait_timeout
    f.argtypes = [C.c_void_p, C.c_int64, _VP]
    f.restype = C.c_int
    _check(ctx, f(ctx, int(limit_cycles), _stream(stream)), "alora_selftest_wait_timeout")


def alora_launch_count(ctx) -> int:
    return int(load_library().alora_launch_count(ctx))


PROFILE_KINDS = ("metadata", "shrink", "project_qkv", "kv_append", "attention", "attention_few_row", "linear", "glue")


def alora_profile_enable(ctx, on: bool) -> None:
    _check(ctx, load_library().alora_profile_enable(ctx, int(bool(on))), "alora_profile_enable")


def alora_profile_read(ctx) -> dict:
    """{family: (milliseconds, launch groups)} accumulated since profiling was enabled."""
    ms = (C.c_double * len(PROFILE_KINDS))()
    n = (C.c_int64 * len(PROFILE_KINDS))()
    _check(ctx, load_library().alora_profile_read(ctx, ms, n), "alora_profile_read")
    return {k: (float(ms[i]), int(n[i])) for i, k in enumerate(PROFILE_KINDS)}


STATIC_MAX_TOKENS, STATIC_MAX_RANK = 4096, 64


def alora_project_qkv_static(dtype, hidden, n_q, n_kv, d_hidden, d_wqkv, positions, query_start_loc,
                             activation_offsets, adapter_on, rank, scale, Aq, Bq, Ak, Bk, Av, Bv, T, R, qkv,
                             stream=None) -> int:
    """Context-free gated projection that allocates nothing (scratch is a fixed array in the library).
    For callers that may not call cudaMalloc.  Returns the status code instead of raising, so that the
    capacity errors can be inspected."""
    lib = load_library()
    f = lib.alora_project_qkv_static
    f.argtypes = [_I] * 4 + [_VP] * 6 + [_I, C.c_float] + [_VP] * 6 + [_I, _I, _VP, _VP]
    f.restype = C.c_int
    return f(dtype, hidden, n_q, n_kv, _ptr(d_hidden), _ptr(d_wqkv), _ptr(positions), _ptr(query_start_loc),
             _ptr(activation_offsets), _ptr(adapter_on), rank, scale, _ptr(Aq), _ptr(Bq), _ptr(Ak), _ptr(Bk),
             _ptr(Av), _ptr(Bv), T, R, _ptr(qkv), _stream(stream))

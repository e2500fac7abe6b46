"""CPU oracle for the aLoRA layer math.  TEST INFRASTRUCTURE ONLY.

Thin numpy/ctypes front end of ``alora_oracle.c`` plus the few compositions (layer, decode step,
decoder stack) that are nothing but calls of those functions in the order the paper lists them
(Prop. 2's proof: new q/k/v rows, cache append, scores over cached-plus-new keys, softmax and
weighted sum).  Only the tests, the smoke check and the benchmark's CPU-baseline leg may import this
package; the CUDA library and its binding never do, and this package imports nothing of theirs.

Arithmetic precision: ``Oracle("f64")`` (default, used for parity) or ``Oracle("f32")`` (the fp32
accumulation the method's tolerance is quoted against).  Weights are float32 arrays, activations
float64 arrays.
"""
from __future__ import annotations

import ctypes as C
import os
import subprocess
from dataclasses import dataclass
from typing import Optional, Sequence

import numpy as np

_HERE = os.path.dirname(os.path.abspath(__file__))
_SRC = os.path.join(_HERE, "alora_oracle.c")
_BUILD = os.path.join(_HERE, "_build")


def build(force: bool = False) -> dict:
    """Compile both precisions of the oracle with gcc; returns {"f64": path, "f32": path}."""
    os.makedirs(_BUILD, exist_ok=True)
    out = {}
    for tag, real in (("f64", "double"), ("f32", "float")):
        so = os.path.join(_BUILD, f"liboracle_{tag}.so")
        if force or not os.path.exists(so) or os.path.getmtime(so) < os.path.getmtime(_SRC):
            tmp = so + f".tmp{os.getpid()}"
            subprocess.check_call(
                ["gcc", "-O2", "-fopenmp", "-shared", "-fPIC", "-Wall", f"-DORACLE_REAL={real}",
                 "-o", tmp, _SRC, "-lm"])
            os.replace(tmp, so)
        out[tag] = so
    return out


@dataclass
class Adapter:
    """One low-rank adapter on q/k/v: Delta_blk = scale * B_blk A_blk (Eq. 4 / Eq. 5)."""
    rank: int
    scale: float
    Aq: np.ndarray  # [r, H]
    Bq: np.ndarray  # [Nq, r]
    Ak: np.ndarray  # [r, H]
    Bk: np.ndarray  # [Nkv, r]
    Av: np.ndarray  # [r, H]
    Bv: np.ndarray  # [Nkv, r]


@dataclass
class MlpAdapter:
    """The same adapter's low-rank pairs on the MLP block's gate, up and down projections (the paper's remark that
    MLP blocks can be adapted in the same manner as q, k and v in Eq. 5)."""
    rank: int
    scale: float
    Ag: np.ndarray  # [r, H]
    Bg: np.ndarray  # [I, r]
    Au: np.ndarray  # [r, H]
    Bu: np.ndarray  # [I, r]
    Ad: np.ndarray  # [r, I]
    Bd: np.ndarray  # [H, r]


def _f32(a):
    return np.ascontiguousarray(a, dtype=np.float32)


def _f64(a):
    return np.ascontiguousarray(a, dtype=np.float64)


def _i32(a):
    return np.ascontiguousarray(a, dtype=np.int32)


def _p(a, ctype):
    return a.ctypes.data_as(C.POINTER(ctype))


class Oracle:
    def __init__(self, precision: str = "f64"):
        self.precision = precision
        self.lib = C.CDLL(build()[precision])
        self.lib.oracle_real_bytes.restype = C.c_int
        assert self.lib.oracle_real_bytes() == (8 if precision == "f64" else 4)

    @property
    def threads(self) -> int:
        return int(self.lib.oracle_num_threads())

    # ---- Eq. 2 -------------------------------------------------------------------------------
    def linear(self, x, W) -> np.ndarray:
        x, W = _f64(x), _f32(W)
        T, K = x.shape
        N = W.shape[0]
        assert W.shape[1] == K
        y = np.empty((T, N), np.float64)
        rc = self.lib.oracle_linear(_p(x, C.c_double), _p(W, C.c_float), T, K, N, _p(y, C.c_double))
        assert rc == 0
        return y

    # ---- Eq. 5 (force_all=False) / Eq. 4 (force_all=True) -----------------------------------------
    def project_qkv(self, x, W, Nq: int, Nkv: int, positions, query_start_loc, activation_offsets,
                    adapter_ids, adapters: Sequence[Adapter], force_all: bool = False):
        """Returns (qkv[T, Nq+2Nkv] float64, gate[T] uint8)."""
        x, W = _f64(x), _f32(W)
        T, H = x.shape
        assert W.shape == (Nq + 2 * Nkv, H)
        positions, qsl = _i32(positions), _i32(query_start_loc)
        R = len(qsl) - 1
        a_req, ids = _i32(activation_offsets), _i32(adapter_ids)
        assert len(positions) == T and len(a_req) == R and len(ids) == R
        n = len(adapters)
        ranks = _i32([a.rank for a in adapters] or [0])
        scales = _f32([a.scale for a in adapters] or [0])
        keep = []

        def ptrs(name, shape_of):
            arr = (C.POINTER(C.c_float) * max(n, 1))()
            for i, a in enumerate(adapters):
                m = _f32(getattr(a, name))
                assert m.shape == shape_of(a), (name, m.shape, shape_of(a))
                keep.append(m)
                arr[i] = _p(m, C.c_float)
            return arr

        Aq = ptrs("Aq", lambda a: (a.rank, H)); Bq = ptrs("Bq", lambda a: (Nq, a.rank))
        Ak = ptrs("Ak", lambda a: (a.rank, H)); Bk = ptrs("Bk", lambda a: (Nkv, a.rank))
        Av = ptrs("Av", lambda a: (a.rank, H)); Bv = ptrs("Bv", lambda a: (Nkv, a.rank))
        qkv = np.empty((T, Nq + 2 * Nkv), np.float64)
        gate = np.zeros(T, np.uint8)
        rc = self.lib.oracle_project_qkv(
            _p(x, C.c_double), _p(W, C.c_float), T, H, Nq, Nkv, _p(positions, C.c_int32),
            _p(qsl, C.c_int32), R, _p(a_req, C.c_int32), _p(ids, C.c_int32), n,
            _p(ranks, C.c_int32), _p(scales, C.c_float), Aq, Bq, Ak, Bk, Av, Bv,
            int(bool(force_all)), _p(qkv, C.c_double), _p(gate, C.c_uint8))
        assert rc == 0, "oracle_project_qkv: bad arguments"
        return qkv, gate

    # ---- Eq. 5's gate applied to one MLP weight matrix -------------- ------------------------------
    def gated_linear(self, x, W, positions, query_start_loc, activation_offsets, adapter_ids, ranks, scales,
                     As, Bs, force_all: bool = False) -> np.ndarray:
        """y_t = W x_t, plus scale * B (A x_t) on the rows of adapter requests at or after the activation offset.
        As[k] is [rank_k, K], Bs[k] is [N, rank_k], indexed by adapter id."""
        x, W = _f64(x), _f32(W)
        T, K = x.shape
        N = W.shape[0]
        assert W.shape[1] == K
        positions, qsl = _i32(positions), _i32(query_start_loc)
        R = len(qsl) - 1
        a_req, ids = _i32(activation_offsets), _i32(adapter_ids)
        n = len(As)
        assert len(Bs) == n and len(ranks) == n and len(scales) == n
        rk, sc = _i32(list(ranks) or [0]), _f32(list(scales) or [0])
        keep_a = [_f32(a) for a in As]
        keep_b = [_f32(b) for b in Bs]
        pa = (C.POINTER(C.c_float) * max(n, 1))()
        pb = (C.POINTER(C.c_float) * max(n, 1))()
        for i in range(n):
            assert keep_a[i].shape == (rk[i], K) and keep_b[i].shape == (N, rk[i])
            pa[i], pb[i] = _p(keep_a[i], C.c_float), _p(keep_b[i], C.c_float)
        y = np.empty((T, N), np.float64)
        rc = self.lib.oracle_gated_linear(_p(x, C.c_double), _p(W, C.c_float), T, K, N, _p(positions, C.c_int32),
                                          _p(qsl, C.c_int32), R, _p(a_req, C.c_int32), _p(ids, C.c_int32), n,
                                          _p(rk, C.c_int32), _p(sc, C.c_float), pa, pb, int(bool(force_all)),
                                          _p(y, C.c_double))
        assert rc == 0, "oracle_gated_linear: bad arguments"
        return y

    # ---- Eq. 1 / Eq. 3 ----------------------------------------------------------------------------
    def attention(self, q, K, V, kv_start_loc, positions, query_start_loc, Hq: int, Hkv: int,
                  hd: int, softmax_scale: Optional[float] = None):
        """q[T, Hq*hd]; K, V[sum len, Hkv*hd] ragged by kv_start_loc.  Returns (out, pairs)."""
        q, K, V = _f64(q), _f64(K), _f64(V)
        T = q.shape[0]
        kvl, positions, qsl = _i32(kv_start_loc), _i32(positions), _i32(query_start_loc)
        R = len(qsl) - 1
        assert q.shape[1] == Hq * hd and K.shape[1] == Hkv * hd and V.shape == K.shape
        assert kvl[-1] == K.shape[0] and len(kvl) == R + 1
        if softmax_scale is None:
            softmax_scale = 1.0 / np.sqrt(hd)
        out = np.empty_like(q)
        pairs = C.c_int64(0)
        rc = self.lib.oracle_attention(
            _p(q, C.c_double), _p(K, C.c_double), _p(V, C.c_double), _p(kvl, C.c_int32),
            _p(positions, C.c_int32), _p(qsl, C.c_int32), T, R, Hq, Hkv, hd,
            C.c_double(float(softmax_scale)), _p(out, C.c_double), C.byref(pairs))
        assert rc == 0, "oracle_attention: bad arguments"
        return out, int(pairs.value)

    # ---- paged cache, integer part ----------------------------------------------------------------
    def slot_mapping(self, positions, query_start_loc, block_tables, page_size: int) -> np.ndarray:
        positions, qsl = _i32(positions), _i32(query_start_loc)
        bt = _i32(block_tables)
        R, max_blocks = bt.shape
        T = len(positions)
        slots = np.empty(T, np.int64)
        rc = self.lib.oracle_slot_mapping(_p(positions, C.c_int32), _p(qsl, C.c_int32),
                                          _p(bt, C.c_int32), max_blocks, page_size, T, R,
                                          _p(slots, C.c_int64))
        assert rc == 0, "oracle_slot_mapping: bad arguments"
        return slots

    def paged_append(self, pool: np.ndarray, k_rows: np.ndarray, v_rows: np.ndarray, slots,
                     Hkv: int, page_size: int, hd: int) -> None:
        """pool [pages, 2, Hkv, page_size, hd] (any dtype), modified in place; rows [T, Hkv*hd]."""
        assert pool.flags.c_contiguous and pool.shape[1:] == (2, Hkv, page_size, hd)
        k_rows = np.ascontiguousarray(k_rows, dtype=pool.dtype)
        v_rows = np.ascontiguousarray(v_rows, dtype=pool.dtype)
        slots = np.ascontiguousarray(slots, dtype=np.int64)
        T = len(slots)
        assert k_rows.shape == (T, Hkv * hd) and v_rows.shape == (T, Hkv * hd)
        rc = self.lib.oracle_paged_append(
            pool.ctypes.data_as(C.POINTER(C.c_uint8)), pool.itemsize,
            k_rows.ctypes.data_as(C.POINTER(C.c_uint8)), v_rows.ctypes.data_as(C.POINTER(C.c_uint8)),
            _p(slots, C.c_int64), T, Hkv, page_size, hd)
        assert rc == 0

    def paged_gather(self, pool: np.ndarray, block_table_row, length: int, Hkv: int, page_size: int,
                     hd: int):
        """Returns contiguous (K, V) [length, Hkv*hd] of one request, dtype of the pool."""
        assert pool.flags.c_contiguous and pool.shape[1:] == (2, Hkv, page_size, hd)
        row = _i32(block_table_row)
        assert len(row) * page_size >= length
        K = np.empty((length, Hkv * hd), pool.dtype)
        V = np.empty((length, Hkv * hd), pool.dtype)
        rc = self.lib.oracle_paged_gather(
            pool.ctypes.data_as(C.POINTER(C.c_uint8)), pool.itemsize, _p(row, C.c_int32), length,
            Hkv, page_size, hd, K.ctypes.data_as(C.POINTER(C.c_uint8)),
            V.ctypes.data_as(C.POINTER(C.c_uint8)))
        assert rc == 0
        return K, V

    # ---- decoder-layer glue -------------------------------------------------------------------
    def rmsnorm(self, x, w, eps: float) -> np.ndarray:
        x, w = _f64(x), _f32(w)
        T, H = x.shape
        y = np.empty_like(x)
        rc = self.lib.oracle_rmsnorm(_p(x, C.c_double), _p(w, C.c_float), T, H, C.c_double(eps),
                                     _p(y, C.c_double))
        assert rc == 0
        return y

    def swiglu(self, gate_up) -> np.ndarray:
        gate_up = _f64(gate_up)
        T, two_i = gate_up.shape
        y = np.empty((T, two_i // 2), np.float64)
        rc = self.lib.oracle_swiglu(_p(gate_up, C.c_double), T, two_i // 2, _p(y, C.c_double))
        assert rc == 0
        return y

    # ---- optional rotary position embedding ------------------------------------------------------
    def rope(self, x, positions, n_heads: int, hd: int, theta: float) -> np.ndarray:
        """Rotate-half rotary embedding of rows [T, n_heads*hd] at the given positions; returns a new array."""
        x = _f64(x).copy()
        positions = _i32(positions)
        T = x.shape[0]
        assert x.shape[1] == n_heads * hd and len(positions) == T
        rc = self.lib.oracle_rope(_p(x, C.c_double), _p(positions, C.c_int32), T, n_heads, hd, C.c_double(float(theta)))
        assert rc == 0, "oracle_rope: bad arguments"
        return x

    # ---- compositions (no arithmetic of their own) ---------------------------------------------
    def attention_block(self, x, W, Nq, Nkv, Hq, Hkv, hd, positions, query_start_loc,
                        activation_offsets, adapter_ids, adapters, prefix_K, prefix_V,
                        force_all=False, softmax_scale=None, rope_theta=0.0):
        """One layer's attention block for new tokens on top of per-request cached K/V.

        prefix_K[r], prefix_V[r]: [P_r, Nkv] arrays (P_r may be 0) holding positions 0..P_r-1 (with
        rope_theta set: keys as cached, i.e. already rotated);
        the new tokens of request r must be positions P_r, P_r+1, ...  Steps, in the order of
        Prop. 2's proof: (1) new q/k/v rows with the gate of Eq. 5, (2) append the new k/v rows
        behind the cached ones, (3) causal softmax attention of the new queries over all rows.
        Returns dict(qkv, gate, K, V (per-request lists incl. new rows), out, pairs).
        """
        qsl = _i32(query_start_loc)
        R = len(qsl) - 1
        positions = _i32(positions)
        qkv, gate = self.project_qkv(x, W, Nq, Nkv, positions, qsl, activation_offsets, adapter_ids,
                                     adapters, force_all)
        if rope_theta:
            # optional: rotate the new query and key rows by their positions before the keys are cached
            # (the cached prefix keys must then be post-rotation too)
            qkv[:, :Nq] = self.rope(qkv[:, :Nq], positions, Hq, hd, rope_theta)
            qkv[:, Nq:Nq + Nkv] = self.rope(qkv[:, Nq:Nq + Nkv], positions, Hkv, hd, rope_theta)
        Ks, Vs, kvl = [], [], [0]
        for r in range(R):
            lo, hi = qsl[r], qsl[r + 1]
            P = 0 if prefix_K is None or prefix_K[r] is None else len(prefix_K[r])
            if hi > lo:
                assert positions[lo] == P and np.all(np.diff(positions[lo:hi]) == 1), \
                    "new tokens must continue the cached prefix"
            k_new, v_new = qkv[lo:hi, Nq:Nq + Nkv], qkv[lo:hi, Nq + Nkv:]
            Ks.append(np.concatenate([_f64(prefix_K[r]), k_new]) if P else k_new.copy())
            Vs.append(np.concatenate([_f64(prefix_V[r]), v_new]) if P else v_new.copy())
            kvl.append(kvl[-1] + len(Ks[-1]))
        Kc = np.concatenate(Ks) if R else np.zeros((0, Nkv))
        Vc = np.concatenate(Vs) if R else np.zeros((0, Nkv))
        out, pairs = self.attention(qkv[:, :Nq], Kc, Vc, kvl, positions, qsl, Hq, Hkv, hd,
                                    softmax_scale)
        return dict(qkv=qkv, gate=gate, K=Ks, V=Vs, out=out, pairs=pairs)

    def decoder_layer(self, h, lw: dict, Nq, Nkv, Hq, Hkv, hd, eps, positions, query_start_loc,
                      activation_offsets, adapter_ids, adapters, prefix_K, prefix_V, force_all=False,
                      rope_theta=0.0, mlp_adapters: Optional[Sequence[MlpAdapter]] = None):
        """Pre-norm residual decoder layer: h + o_proj(attn(norm(h))), then + down(swiglu(gate_up(norm))).
        With `mlp_adapters` (indexed by adapter id like `adapters`) the gate, up and down projections are adapted
        under the same per-token gate as q/k/v."""
        xn = self.rmsnorm(h, lw["norm_attn"], eps)
        blk = self.attention_block(xn, lw["wqkv"], Nq, Nkv, Hq, Hkv, hd, positions, query_start_loc,
                                   activation_offsets, adapter_ids, adapters, prefix_K, prefix_V,
                                   force_all, rope_theta=rope_theta)
        h1 = _f64(h) + self.linear(blk["out"], lw["wo"])
        xm = self.rmsnorm(h1, lw["norm_mlp"], eps)
        if not mlp_adapters:
            h2 = h1 + self.linear(self.swiglu(self.linear(xm, lw["wgate_up"])), lw["wdown"])
            return h2, blk
        inter = lw["wgate_up"].shape[0] // 2
        ranks = [m.rank for m in mlp_adapters]
        scales = [m.scale for m in mlp_adapters]
        gated = lambda x, W, a, b: self.gated_linear(  # noqa: E731
            x, W, positions, query_start_loc, activation_offsets, adapter_ids, ranks, scales,
            [getattr(m, a) for m in mlp_adapters], [getattr(m, b) for m in mlp_adapters], force_all)
        gate = gated(xm, lw["wgate_up"][:inter], "Ag", "Bg")
        up = gated(xm, lw["wgate_up"][inter:], "Au", "Bu")
        act = self.swiglu(np.concatenate([gate, up], axis=1))
        h2 = h1 + gated(act, lw["wdown"], "Ad", "Bd")
        return h2, blk

/*
 * CPU oracle for the Activated-LoRA (aLoRA) layer math.  TEST INFRASTRUCTURE ONLY.
 *
 * This file is the slow, plain statement of what the GPU library must compute.  Only the test
 * suite, the smoke check and the benchmark's CPU-baseline leg may build, load or call it; the
 * product (the CUDA library and its Python binding) never does, and the two share no code.
 *
 * Everything is written the obvious way: one loop nest per formula, no tiling, no online softmax,
 * no blocking, no SIMD intrinsics, no BLAS.  Arithmetic runs in `real`, which is double unless the
 * file is compiled with -DORACLE_REAL=float (the fp32 variant exists because the method's stated
 * comparison precision is fp32 accumulation; parity tests use the double build).  Weights are float
 * arrays, activations and outputs are double arrays (bf16 workloads pass values already rounded to
 * bf16 and widened, which is exact; inside the layer stack activations stay unrounded).
 * OpenMP parallelises the outermost independent loop only (tokens, or token x head).
 *
 * Conventions (0-based): position p of a request is its token index in the whole sequence; the
 * paper's 1-based t_invoke equals a_req + 1, so "rows t_invoke..t are adapted" (Eq. 5) reads
 * "adapted iff p >= a_req".  Weights are stored output-major: y = W x with W[N][H]; the paper's
 * row-vector form X W^Q (Eq. 2) is the same product with W transposed.  The fused output row is
 * [ q heads | k heads | v heads ], N = Nq + 2 Nkv.  Query head h reads KV head h / (Hq / Hkv).
 *
 * Pins (tests/test_oracle_pins.py): Prop. 1 bit-equality of pre-activation rows, the cache-reuse
 * identity, B = 0 => base, a_req = 0 => merged-weight LoRA (Eq. 4) against a library matmul,
 * attention against a library softmax-attention routine and closed forms (single key, uniform
 * scores, two-key logistic weight, constant V), decode == prefill row, page-permutation
 * invariance, brute-force slot indices, the cache layout read back by plain array indexing, and
 * Prop. 2's closed-form pair and row counts; the optional rotary embedding by a complex-multiplication
 * restatement, a hand example, norm preservation and the relative-position property; the gated
 * MLP adaptation by B = 0 => base, a_req = 0 => merged weights against a library matmul, bit-equal
 * pre-activation rows, a library restatement of the adapted layer, and the cache-reuse identity
 * through two adapted layers (which fails when the MLP gate is left open).
 * tests/test_oracle_mutants.py plants one-line
 * mistakes in a copy of this file and checks that the pins notice.
 * No function in this file is "parity unpinned".
 */
#include <math.h>
#include <stdint.h>
#include <stdlib.h>
#include <string.h>
#ifdef _OPENMP
#include <omp.h>
#endif

#ifndef ORACLE_REAL
#define ORACLE_REAL double
#endif
typedef ORACLE_REAL real;

#define ORACLE_OK 0
#define ORACLE_ERR_ARG 1

int oracle_real_bytes(void) { return (int)sizeof(real); }

int oracle_num_threads(void) {
#ifdef _OPENMP
    return omp_get_max_threads();
#else
    return 1;
#endif
}

/* Request that owns flat token index t: the r with query_start_loc[r] <= t < query_start_loc[r+1]. */
static int request_of_token(const int32_t *query_start_loc, int R, int t) {
    for (int r = 0; r < R; ++r)
        if (t >= query_start_loc[r] && t < query_start_loc[r + 1]) return r;
    return -1;
}

/*
 * Plain dense projection y[t][n] = sum_h W[n][h] x[t][h]   (Eq. 2, one weight matrix).
 * Also used for o_proj and the MLP matrices of the decoder-layer stack.
 */
int oracle_linear(const double *x, const float *W, int T, int K, int N, double *y) {
    if (!x || !W || !y || T < 0 || K <= 0 || N <= 0) return ORACLE_ERR_ARG;
#pragma omp parallel for schedule(static)
    for (int t = 0; t < T; ++t) {
        for (int n = 0; n < N; ++n) {
            real acc = 0;
            for (int k = 0; k < K; ++k) acc += (real)W[(size_t)n * K + k] * (real)x[(size_t)t * K + k];
            y[(size_t)t * N + n] = (double)acc;
        }
    }
    return ORACLE_OK;
}

/*
 * Gated q/k/v projection of a ragged batch (Eq. 2 for the base term, Eq. 5 for the gate,
 * Eq. 4 when force_all != 0).
 *
 *   y_t = W x_t                                   if request has no adapter, or p_t < a_req
 *   y_t = W x_t + s * B_blk (A_blk x_t)  per block if adapter k and p_t >= a_req   (blk = q, k, v)
 *
 * x[T][H], W[N][H]; adapters are given as arrays indexed by adapter id: rank, scale and six
 * pointers A_q[r][H], B_q[Nq][r], A_k[r][H], B_k[Nkv][r], A_v[r][H], B_v[Nkv][r].
 * gate_out (optional, [T]) receives 1 where the delta was applied.  A gated-off row executes
 * no adapter arithmetic at all (the paper's "W + 0" is the base product itself).
 */
int oracle_project_qkv(const double *x, const float *W, int T, int H, int Nq, int Nkv,
                       const int32_t *positions, const int32_t *query_start_loc, int R,
                       const int32_t *activation_offsets, const int32_t *adapter_ids,
                       int n_adapters, const int32_t *ranks, const float *scales,
                       const float *const *Aq, const float *const *Bq,
                       const float *const *Ak, const float *const *Bk,
                       const float *const *Av, const float *const *Bv,
                       int force_all, double *qkv, uint8_t *gate_out) {
    if (!x || !W || !qkv || !positions || !query_start_loc || T < 0 || R < 0) return ORACLE_ERR_ARG;
    const int N = Nq + 2 * Nkv;
    int bad = 0;
#pragma omp parallel for schedule(static)
    for (int t = 0; t < T; ++t) {
        const int r = request_of_token(query_start_loc, R, t);
        if (r < 0) { bad = 1; continue; }
        const double *xt = x + (size_t)t * H;
        double *yt = qkv + (size_t)t * N;
        const int k = adapter_ids ? adapter_ids[r] : -1;
        int gate = 0;
        if (k >= 0) {
            if (k >= n_adapters) { bad = 1; continue; }
            gate = force_all ? 1 : (positions[t] >= activation_offsets[r]);
        }
        if (gate_out) gate_out[t] = (uint8_t)gate;
        /* base term, every output column */
        for (int n = 0; n < N; ++n) {
            real acc = 0;
            for (int h = 0; h < H; ++h) acc += (real)W[(size_t)n * H + h] * (real)xt[h];
            yt[n] = (double)acc;
        }
        if (!gate) continue;
        /* low-rank delta, one block at a time: u = A x, d = B u, y_blk += s d */
        const int rk = ranks[k];
        const real s = (real)scales[k];
        const float *As[3] = {Aq[k], Ak[k], Av[k]};
        const float *Bs[3] = {Bq[k], Bk[k], Bv[k]};
        const int width[3] = {Nq, Nkv, Nkv};
        const int first[3] = {0, Nq, Nq + Nkv};
        real *u = (real *)malloc(sizeof(real) * (size_t)(rk > 0 ? rk : 1));
        for (int b = 0; b < 3; ++b) {
            for (int i = 0; i < rk; ++i) {
                real acc = 0;
                for (int h = 0; h < H; ++h) acc += (real)As[b][(size_t)i * H + h] * (real)xt[h];
                u[i] = acc;
            }
            for (int n = 0; n < width[b]; ++n) {
                real d = 0;
                for (int i = 0; i < rk; ++i) d += (real)Bs[b][(size_t)n * rk + i] * u[i];
                yt[first[b] + n] = (double)((real)yt[first[b] + n] + s * d);
            }
        }
        free(u);
    }
    return bad ? ORACLE_ERR_ARG : ORACLE_OK;
}

/*
 * Gated low-rank adaptation of ONE weight matrix of an MLP block (gate, up or down projection).
 * The paper remarks that MLP blocks can be adapted in the same manner as Q, K and V in Eq. 5
 * (Sec. 2, remark on MLP blocks; Sec. 3, the sentence after Eq. 5): a token before the
 * activation offset is multiplied by the base weight alone, a token at or after it by W + s B A.
 *
 *   y_t = W x_t                        if the request has no adapter, or p_t < a_req
 *   y_t = W x_t + s * B (A x_t)        if adapter k and p_t >= a_req
 *
 * x[T][K], W[N][K]; per adapter id: rank, scale, A[r][K], B[N][r].  As in the q/k/v projection a
 * gated-off row executes no adapter arithmetic.  force_all != 0 opens every adapter row's gate (Eq. 4).
 */
int oracle_gated_linear(const double *x, const float *W, int T, int K, int N,
                        const int32_t *positions, const int32_t *query_start_loc, int R,
                        const int32_t *activation_offsets, const int32_t *adapter_ids,
                        int n_adapters, const int32_t *ranks, const float *scales,
                        const float *const *A, const float *const *B, int force_all, double *y) {
    if (!x || !W || !y || !positions || !query_start_loc || T < 0 || R < 0 || K <= 0 || N <= 0) return ORACLE_ERR_ARG;
    int bad = 0;
#pragma omp parallel for schedule(static)
    for (int t = 0; t < T; ++t) {
        const int r = request_of_token(query_start_loc, R, t);
        if (r < 0) { bad = 1; continue; }
        const double *xt = x + (size_t)t * K;
        double *yt = y + (size_t)t * N;
        const int k = adapter_ids ? adapter_ids[r] : -1;
        int gate = 0;
        if (k >= 0) {
            if (k >= n_adapters) { bad = 1; continue; }
            gate = force_all || positions[t] >= activation_offsets[r];   /* the MLP gate */
        }
        for (int n = 0; n < N; ++n) {
            real acc = 0;
            for (int h = 0; h < K; ++h) acc += (real)W[(size_t)n * K + h] * (real)xt[h];
            yt[n] = (double)acc;
        }
        if (!gate) continue;
        const int rk = ranks[k];
        const real s = (real)scales[k];
        real *u = (real *)malloc(sizeof(real) * (size_t)(rk > 0 ? rk : 1));
        for (int i = 0; i < rk; ++i) {
            real acc = 0;
            for (int h = 0; h < K; ++h) acc += (real)A[k][(size_t)i * K + h] * (real)xt[h];
            u[i] = acc;
        }
        for (int n = 0; n < N; ++n) {
            real d = 0;
            for (int i = 0; i < rk; ++i) d += (real)B[k][(size_t)n * rk + i] * u[i];   /* MLP expand */
            yt[n] = (double)((real)yt[n] + s * d);   /* MLP delta add */
        }
        free(u);
    }
    return bad ? ORACLE_ERR_ARG : ORACLE_OK;
}

/*
 * Causal grouped-query softmax attention of new tokens over each request's contiguous K/V
 * (Eq. 1; per-token form Eq. 3: token at position p attends keys 0..p, itself included).
 *
 * q[T][Hq*hd]; K, V hold every request's rows back to back: request r owns rows
 * kv_start_loc[r] .. kv_start_loc[r+1]-1, row j of that range is position j; each row is
 * [Hkv][hd].  out[T][Hq*hd].  softmax_scale multiplies the scores (1/sqrt(hd) per Eq. 1).
 * pair_count (optional) receives the number of (query, key) score pairs evaluated per query
 * head, i.e. sum over new tokens of (p + 1)  (Prop. 2's operation count).
 */
int oracle_attention(const double *q, const double *K, const double *V,
                     const int32_t *kv_start_loc, const int32_t *positions,
                     const int32_t *query_start_loc, int T, int R, int Hq, int Hkv, int hd,
                     double softmax_scale, double *out, int64_t *pair_count) {
    if (!q || !K || !V || !out || Hkv <= 0 || Hq % Hkv != 0) return ORACLE_ERR_ARG;
    const int G = Hq / Hkv;
    const size_t Nq = (size_t)Hq * hd, Nkv = (size_t)Hkv * hd;
    int bad = 0;
    int64_t pairs = 0;
#pragma omp parallel for collapse(2) schedule(dynamic, 4) reduction(+ : pairs)
    for (int t = 0; t < T; ++t) {
        for (int h = 0; h < Hq; ++h) {
            const int r = request_of_token(query_start_loc, R, t);
            if (r < 0) { bad = 1; continue; }
            const int p = positions[t];
            const int len = kv_start_loc[r + 1] - kv_start_loc[r];
            if (p < 0 || p >= len) { bad = 1; continue; }
            const int g = h / G; /* KV head shared by this group of query heads */
            const double *qh = q + (size_t)t * Nq + (size_t)h * hd;
            const int nk = p + 1; /* keys 0..p visible */
            real *w = (real *)malloc(sizeof(real) * (size_t)nk);
            real m = -INFINITY;
            for (int j = 0; j < nk; ++j) {
                const double *kj = K + ((size_t)kv_start_loc[r] + j) * Nkv + (size_t)g * hd;
                real s = 0;
                for (int d = 0; d < hd; ++d) s += (real)qh[d] * (real)kj[d];
                s *= (real)softmax_scale;
                w[j] = s;
                if (s > m) m = s;
            }
            real denom = 0;
            for (int j = 0; j < nk; ++j) {
                w[j] = (real)exp((double)(w[j] - m));
                denom += w[j];
            }
            double *oh = out + (size_t)t * Nq + (size_t)h * hd;
            for (int d = 0; d < hd; ++d) {
                real acc = 0;
                for (int j = 0; j < nk; ++j) {
                    const double *vj = V + ((size_t)kv_start_loc[r] + j) * Nkv + (size_t)g * hd;
                    acc += w[j] * (real)vj[d];
                }
                oh[d] = (double)(acc / denom);
            }
            free(w);
            if (h == 0) pairs += nk;
        }
    }
    if (pair_count) *pair_count = pairs;
    return bad ? ORACLE_ERR_ARG : ORACLE_OK;
}

/*
 * Paged KV cache, integer part.  The pool is [num_pages][2][Hkv][page_size][hd] (K plane then V
 * plane inside a page).  Position p of request r lives in physical page
 * block_tables[r][p / page_size] at row p % page_size; its token slot is page * page_size + row.
 */
int oracle_slot_mapping(const int32_t *positions, const int32_t *query_start_loc,
                        const int32_t *block_tables, int max_blocks, int page_size, int T, int R,
                        int64_t *slots) {
    if (!positions || !query_start_loc || !block_tables || !slots || page_size <= 0) return ORACLE_ERR_ARG;
    for (int t = 0; t < T; ++t) {
        const int r = request_of_token(query_start_loc, R, t);
        if (r < 0) return ORACLE_ERR_ARG;
        const int p = positions[t];
        const int blk = p / page_size;
        if (p < 0 || blk >= max_blocks) return ORACLE_ERR_ARG;
        slots[t] = (int64_t)block_tables[(size_t)r * max_blocks + blk] * page_size + p % page_size;
    }
    return ORACLE_OK;
}

/* Byte offset (in elements) of (slot, plane, kv head) row start inside the pool. */
static size_t pool_row_offset(int64_t slot, int plane, int head, int Hkv, int page_size, int hd) {
    const int64_t page = slot / page_size, row = slot % page_size;
    return ((((size_t)page * 2 + (size_t)plane) * Hkv + (size_t)head) * page_size + (size_t)row) * hd;
}

/*
 * KV append: copy each new token's k and v rows (k_rows/v_rows: [T][Hkv*hd], any element size)
 * to its slot.  Bytes of every other slot are left alone.
 */
int oracle_paged_append(uint8_t *pool, int elem_size, const uint8_t *k_rows, const uint8_t *v_rows,
                        const int64_t *slots, int T, int Hkv, int page_size, int hd) {
    if (!pool || !k_rows || !v_rows || !slots) return ORACLE_ERR_ARG;
    const size_t rowb = (size_t)hd * elem_size;
    for (int t = 0; t < T; ++t)
        for (int g = 0; g < Hkv; ++g) {
            memcpy(pool + pool_row_offset(slots[t], 0, g, Hkv, page_size, hd) * elem_size,
                   k_rows + ((size_t)t * Hkv + g) * rowb, rowb);
            memcpy(pool + pool_row_offset(slots[t], 1, g, Hkv, page_size, hd) * elem_size,
                   v_rows + ((size_t)t * Hkv + g) * rowb, rowb);
        }
    return ORACLE_OK;
}

/*
 * Gather one request's first `len` positions out of the pool into contiguous K[len][Hkv*hd],
 * V[len][Hkv*hd] (same element size as the pool).
 */
int oracle_paged_gather(const uint8_t *pool, int elem_size, const int32_t *block_table_row,
                        int len, int Hkv, int page_size, int hd, uint8_t *K, uint8_t *V) {
    if (!pool || !block_table_row || !K || !V) return ORACLE_ERR_ARG;
    const size_t rowb = (size_t)hd * elem_size;
    for (int p = 0; p < len; ++p) {
        const int64_t slot = (int64_t)block_table_row[p / page_size] * page_size + p % page_size;
        for (int g = 0; g < Hkv; ++g) {
            memcpy(K + ((size_t)p * Hkv + g) * rowb,
                   pool + pool_row_offset(slot, 0, g, Hkv, page_size, hd) * elem_size, rowb);
            memcpy(V + ((size_t)p * Hkv + g) * rowb,
                   pool + pool_row_offset(slot, 1, g, Hkv, page_size, hd) * elem_size, rowb);
        }
    }
    return ORACLE_OK;
}

/*
 * Rotary position embedding, "rotate-half" pairing, applied in place to rows of n_heads heads of hd columns.
 * The paper's equations carry no positional encoding (positions enter only through the gate and the causal
 * mask); the model families it evaluates are rotary models, so the rotation is an OPTION of the layer, off unless
 * a base theta is given.  Reading taken: within a head, column i (0 <= i < hd/2) is paired with column i + hd/2;
 * the pair at position p is turned by the angle p * theta^(-2i/hd):
 *     x'[i]        = x[i] cos(a) - x[i + hd/2] sin(a)
 *     x'[i + hd/2] = x[i + hd/2] cos(a) + x[i] sin(a)
 * It is applied to the query and key rows after the projection (delta included) and before the keys are
 * cached, so cached keys are post-rotation and a query-key score depends on the two positions only through
 * their difference.
 */
int oracle_rope(double *x, const int32_t *positions, int T, int n_heads, int hd, double theta) {
    if (!x || !positions || T < 0 || n_heads <= 0 || hd <= 0 || hd % 2 != 0 || !(theta > 0)) return ORACLE_ERR_ARG;
    const int half = hd / 2;
    for (int t = 0; t < T; ++t)
        for (int h = 0; h < n_heads; ++h) {
            double *v = x + ((size_t)t * n_heads + h) * hd;
            for (int i = 0; i < half; ++i) {
                const double a = (double)positions[t] * pow(theta, -2.0 * (double)i / (double)hd);
                const real c = (real)cos(a), s = (real)sin(a);
                const real lo = (real)v[i], hi = (real)v[i + half];
                v[i] = (double)(lo * c - hi * s);
                v[i + half] = (double)(hi * c + lo * s);
            }
        }
    return ORACLE_OK;
}

/*
 * Decoder-layer glue around the attention block (the paper only says that the MLP acts on each
 * token independently; the concrete form is the benchmark configuration's: RMSNorm, SwiGLU,
 * pre-norm residual).
 *   rmsnorm:  y = x / sqrt(mean(x^2) + eps) * w
 *   swiglu:   y[i] = silu(g[i]) * u[i]  with  gate_up row = [ g (I) | u (I) ],  silu(z) = z / (1 + e^-z)
 */
int oracle_rmsnorm(const double *x, const float *w, int T, int H, double eps, double *y) {
    if (!x || !w || !y) return ORACLE_ERR_ARG;
    for (int t = 0; t < T; ++t) {
        real ss = 0;
        for (int h = 0; h < H; ++h) ss += (real)x[(size_t)t * H + h] * (real)x[(size_t)t * H + h];
        const real inv = (real)1 / (real)sqrt((double)(ss / (real)H + (real)eps));
        for (int h = 0; h < H; ++h)
            y[(size_t)t * H + h] = (double)((real)x[(size_t)t * H + h] * inv * (real)w[h]);
    }
    return ORACLE_OK;
}

int oracle_swiglu(const double *gate_up, int T, int I, double *y) {
    if (!gate_up || !y) return ORACLE_ERR_ARG;
    for (int t = 0; t < T; ++t)
        for (int i = 0; i < I; ++i) {
            const real g = (real)gate_up[(size_t)t * 2 * I + i];
            const real u = (real)gate_up[(size_t)t * 2 * I + I + i];
            y[(size_t)t * I + i] = (double)(g / ((real)1 + (real)exp(-(double)g)) * u);
        }
    return ORACLE_OK;
}

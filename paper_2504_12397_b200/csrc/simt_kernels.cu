// CUDA-core kernels: the fp32 data type's projection and attention (tiny exact-precision
// configurations), and the element-wise / copy steps shared by both data types (adapter repack,
// KV append, RMSNorm, SwiGLU).
#include "alora_internal.h"
#include "tc_common.cuh"

namespace alora {

template <typename T> __device__ __forceinline__ float ldf(const T *p);
template <> __device__ __forceinline__ float ldf<float>(const float *p) { return *p; }
template <> __device__ __forceinline__ float ldf<__nv_bfloat16>(const __nv_bfloat16 *p) { return __bfloat162float(*p); }
template <typename T> __device__ __forceinline__ void stf(T *p, float v);
template <> __device__ __forceinline__ void stf<float>(float *p, float v) { *p = v; }
template <> __device__ __forceinline__ void stf<__nv_bfloat16>(__nv_bfloat16 *p, float v) { *p = __float2bfloat16_rn(v); }

// ---------------------------------------------------------------------------------------------
// Adapter repack: A_dst[3][RP][H] <- (Aq, Ak, Av)[r][H] with zero rows r..RP-1;
// B_dst[N][RP] <- rows of (Bq | Bk | Bv)[.][r] with zero columns r..RP-1.
// ---------------------------------------------------------------------------------------------
template <typename T>
__global__ void repack_adapter_kernel(const T *Aq, const T *Ak, const T *Av, const T *Bq, const T *Bk,
                                      const T *Bv, int rank, int RP, int H, int Nq, int Nkv, T *A_dst,
                                      T *B_dst) {
    const size_t nA = (size_t)3 * RP * H, nB = (size_t)(Nq + 2 * Nkv) * RP;
    for (size_t i = blockIdx.x * (size_t)blockDim.x + threadIdx.x; i < nA + nB;
         i += (size_t)gridDim.x * blockDim.x) {
        if (i < nA) {
            int blk = (int)(i / ((size_t)RP * H));
            int row = (int)((i / H) % RP), h = (int)(i % H);
            const T *src = blk == 0 ? Aq : (blk == 1 ? Ak : Av);
            A_dst[i] = row < rank ? src[(size_t)row * H + h] : T(0.f);
        } else {
            size_t j = i - nA;
            int n = (int)(j / RP), c = (int)(j % RP);
            T v = T(0.f);
            if (c < rank) {
                if (n < Nq) v = Bq[(size_t)n * rank + c];
                else if (n < Nq + Nkv) v = Bk[(size_t)(n - Nq) * rank + c];
                else v = Bv[(size_t)(n - Nq - Nkv) * rank + c];
            }
            B_dst[j] = v;
        }
    }
}

int launch_repack_adapter(alora_ctx *ctx, int rank, const void *Aq, const void *Bq, const void *Ak,
                          const void *Bk, const void *Av, const void *Bv, void *A_dst, void *B_dst,
                          cudaStream_t s) {
    const Dims &d = ctx->d;
    if (ctx->cfg.dtype == ALORA_DTYPE_FP32)
        repack_adapter_kernel<float><<<256, 256, 0, s>>>((const float *)Aq, (const float *)Ak, (const float *)Av,
                                                         (const float *)Bq, (const float *)Bk, (const float *)Bv,
                                                         rank, d.RP, d.H, d.Nq, d.Nkv, (float *)A_dst, (float *)B_dst);
    else
        repack_adapter_kernel<__nv_bfloat16><<<256, 256, 0, s>>>(
            (const __nv_bfloat16 *)Aq, (const __nv_bfloat16 *)Ak, (const __nv_bfloat16 *)Av,
            (const __nv_bfloat16 *)Bq, (const __nv_bfloat16 *)Bk, (const __nv_bfloat16 *)Bv, rank, d.RP, d.H,
            d.Nq, d.Nkv, (__nv_bfloat16 *)A_dst, (__nv_bfloat16 *)B_dst);
    return 1;
}

// ---------------------------------------------------------------------------------------------
// CUDA-core shrink: t[row][blk][i] = scale * sum_h A[blk][i][h] x[row][h] for rows with an applied
// adapter (Eq. 5, inner product of the low-rank delta).  One block per row, one warp per output.
// ---------------------------------------------------------------------------------------------
template <typename T>
__global__ void shrink_simt_kernel(const T *__restrict__ x, const int32_t *__restrict__ row_adapter,
                                  const AdapterDev *__restrict__ adapters, int H, int RP,
                                  float *__restrict__ t) {
    const int row = blockIdx.x;
    const int k = row_adapter[row];
    if (k < 0) return;
    const AdapterDev ad = adapters[k];
    const T *A = (const T *)ad.A;
    const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31, nwarps = blockDim.x >> 5;
    for (int o = warp; o < 3 * RP; o += nwarps) {
        const int i = o % RP;
        float acc = 0.f;
        if (i < ad.rank) {
            const T *a = A + (size_t)o * H;
            for (int h = lane; h < H; h += 32) acc += ldf(a + h) * ldf(x + (size_t)row * H + h);
            for (int off = 16; off; off >>= 1) acc += __shfl_xor_sync(0xffffffffu, acc, off);
        }
        if (lane == 0) t[(size_t)row * 3 * RP + o] = acc * ad.scale;
    }
}

// ---------------------------------------------------------------------------------------------
// Row-wise low-rank delta for batches of few rows per adapter (bf16):
//     delta[row][n] = s * sum_i B[n][i] (A x_row)[blk(n)][i]          (Eq. 5, the term behind the gate)
// for every row with an applied adapter, in fp32.  One block per (row, q/k/v block): the row of x is staged in
// shared memory, each of 32 warps forms one or two of the block's `rank` inner products with A (16-byte loads,
// several in flight per lane), then each thread forms outputs of the block's columns from its B rows.  Adapter storage is the rank-padded tensor-core layout A[3][64][H], B[N][64].  The kernel does
// nothing unless the metadata step chose the row-wise route for this batch (*rowwise_flag).
// ---------------------------------------------------------------------------------------------
constexpr int kDeltaThreads = 1024;  // 32 warps: one or two inner products per warp, many loads in flight per SM

__global__ void __launch_bounds__(kDeltaThreads)
lora_delta_rows_kernel(const __nv_bfloat16 *__restrict__ x, const int32_t *__restrict__ row_adapter,
                       const AdapterDev *__restrict__ adapters, const int32_t *__restrict__ rowwise_flag, int H,
                       int Nq, int Nkv, int N, float *__restrict__ delta) {
    extern __shared__ uint4 x_s4[];  // H bf16
    __shared__ float t_s[kRankPadMax];
    tc::grid_dep_launch();
    tc::grid_dep_wait();   // the flag and the row -> adapter map come from the metadata kernel
    if (*rowwise_flag == 0) return;
    const int row = blockIdx.x, blk = blockIdx.y;
    const int k = row_adapter[row];
    if (k < 0) return;
    const AdapterDev ad = adapters[k];
    const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
    const int hv = H / 8;  // 16-byte vectors per row
    const uint4 *xg = reinterpret_cast<const uint4 *>(x + (size_t)row * H);
    for (int i = threadIdx.x; i < hv; i += blockDim.x) x_s4[i] = xg[i];
    __syncthreads();
    {
        // inner products warp and warp + 32 (rank <= 64)
        const uint4 *A4 = reinterpret_cast<const uint4 *>(ad.A) + (size_t)blk * kRankPadMax * hv;
        const bool on0 = warp < ad.rank, on1 = warp + 32 < ad.rank;
        const uint4 *a0 = A4 + (size_t)warp * hv, *a1 = A4 + (size_t)(warp + 32) * hv;
        float acc0 = 0.f, acc1 = 0.f;
        if (on0) {
#pragma unroll 2
            for (int v = lane; v < hv; v += 32) {
                const uint4 xv = x_s4[v];
                const uint4 av0 = a0[v];
                const uint4 av1 = on1 ? a1[v] : make_uint4(0, 0, 0, 0);
                const __nv_bfloat162 *x2 = reinterpret_cast<const __nv_bfloat162 *>(&xv);
                const __nv_bfloat162 *p0 = reinterpret_cast<const __nv_bfloat162 *>(&av0);
                const __nv_bfloat162 *p1 = reinterpret_cast<const __nv_bfloat162 *>(&av1);
#pragma unroll
                for (int e = 0; e < 4; ++e) {
                    const float2 xf = __bfloat1622float2(x2[e]);
                    const float2 f0 = __bfloat1622float2(p0[e]), f1 = __bfloat1622float2(p1[e]);
                    acc0 = fmaf(f0.x, xf.x, acc0); acc0 = fmaf(f0.y, xf.y, acc0);
                    acc1 = fmaf(f1.x, xf.x, acc1); acc1 = fmaf(f1.y, xf.y, acc1);
                }
            }
        }
        for (int off = 16; off; off >>= 1) {
            acc0 += __shfl_xor_sync(0xffffffffu, acc0, off);
            acc1 += __shfl_xor_sync(0xffffffffu, acc1, off);
        }
        if (lane == 0) {
            t_s[warp] = on0 ? acc0 * ad.scale : 0.f;          // zero beyond the rank
            t_s[warp + 32] = on1 ? acc1 * ad.scale : 0.f;
        }
    }
    __syncthreads();
    const int n_begin = blk == 0 ? 0 : (blk == 1 ? Nq : Nq + Nkv);
    const int n_end = blk == 0 ? Nq : (blk == 1 ? Nq + Nkv : N);
    const uint4 *B4 = reinterpret_cast<const uint4 *>(ad.B);
    const int rv = (ad.rank + 7) / 8;  // 16-byte vectors of a B row that hold non-zero columns (padding is zero)
    for (int n = n_begin + threadIdx.x; n < n_end; n += blockDim.x) {
        const uint4 *brow = B4 + (size_t)n * (kRankPadMax / 8);
        float acc = 0.f;
#pragma unroll
        for (int half = 0; half < 2; ++half) {   // four 16-byte vectors (32 rank columns) at a time, loads first
            if (half * 4 >= rv) break;
            uint4 b[4];
#pragma unroll
            for (int v = 0; v < 4; ++v) b[v] = half * 4 + v < rv ? brow[half * 4 + v] : make_uint4(0, 0, 0, 0);
#pragma unroll
            for (int v = 0; v < 4; ++v) {
                const __nv_bfloat162 *p = reinterpret_cast<const __nv_bfloat162 *>(&b[v]);
#pragma unroll
                for (int e = 0; e < 4; ++e) {
                    const float2 f = __bfloat1622float2(p[e]);
                    acc = fmaf(f.x, t_s[(half * 4 + v) * 8 + 2 * e], acc);
                    acc = fmaf(f.y, t_s[(half * 4 + v) * 8 + 2 * e + 1], acc);
                }
            }
        }
        delta[(size_t)row * N + n] = acc;
    }
}

int launch_lora_delta_rows(alora_ctx *ctx, int layer, const void *hidden, int T, cudaStream_t s) {
    const Dims &d = ctx->d;
    const AdapterDev *ads = ctx->d_adapters + (size_t)layer * ctx->cfg.max_adapters;
    launch_kernel(lora_delta_rows_kernel, dim3(T, 3), dim3(kDeltaThreads), (size_t)d.H * 2, s, true, (const __nv_bfloat16 *)hidden, (const int32_t *)ctx->d_row_adapter, ads,
                                                                   ctx->d_counts + 5, d.H, d.Nq, d.Nkv, d.N,
                                                                   ctx->d_row_delta);
    return 1;
}

// ---------------------------------------------------------------------------------------------
// CUDA-core projection y[row][n] = sum_h W[n][h] x[row][h]  (+ sum_i B[n][i] t[row][blk(n)][i] when the
// row has an applied adapter).  64x64 output tile per block, 16x16 threads, 4x4 outputs each,
// K staged through shared memory 16 columns at a time.  The base sum of a row is formed by the
// same instruction sequence whether or not the delta follows, so gated-off rows equal a base-only
// call bit for bit.  Optional residual: y += residual[row][n] (used by o_proj / down_proj).
// ---------------------------------------------------------------------------------------------
template <typename T>
__global__ void __launch_bounds__(256)
linear_simt_kernel(const T *__restrict__ x, const T *__restrict__ W, int Tn, int K, int N,
                  const int32_t *__restrict__ row_adapter, const AdapterDev *__restrict__ adapters,
                  const float *__restrict__ t, int RP, int Nq, int Nkv, const T *residual /* may alias y */,
                   T *y) {
    __shared__ float xs[16][64 + 1], ws[16][64 + 1];
    const int tx = threadIdx.x & 15, ty = threadIdx.x >> 4;
    const int row0 = blockIdx.y * 64, col0 = blockIdx.x * 64;
    float acc[4][4] = {};
    for (int k0 = 0; k0 < K; k0 += 16) {
        for (int i = threadIdx.x; i < 64 * 16; i += 256) {
            int rr = i >> 4, kk = i & 15;
            int gr = row0 + rr, gc = col0 + rr, gk = k0 + kk;
            xs[kk][rr] = (gr < Tn && gk < K) ? ldf(x + (size_t)gr * K + gk) : 0.f;
            ws[kk][rr] = (gc < N && gk < K) ? ldf(W + (size_t)gc * K + gk) : 0.f;
        }
        __syncthreads();
#pragma unroll
        for (int kk = 0; kk < 16; ++kk) {
            float a[4], b[4];
#pragma unroll
            for (int i = 0; i < 4; ++i) { a[i] = xs[kk][ty * 4 + i]; b[i] = ws[kk][tx * 4 + i]; }
#pragma unroll
            for (int i = 0; i < 4; ++i)
#pragma unroll
                for (int j = 0; j < 4; ++j) acc[i][j] += a[i] * b[j];
        }
        __syncthreads();
    }
#pragma unroll
    for (int i = 0; i < 4; ++i) {
        const int row = row0 + ty * 4 + i;
        if (row >= Tn) continue;
        const int k = row_adapter ? row_adapter[row] : -1;
#pragma unroll
        for (int j = 0; j < 4; ++j) {
            const int n = col0 + tx * 4 + j;
            if (n >= N) continue;
            float v = acc[i][j];
            if (k >= 0) {
                const AdapterDev ad = adapters[k];
                const T *B = (const T *)ad.B + (size_t)n * RP;
                const int blk = n < Nq ? 0 : (n < Nq + Nkv ? 1 : 2);
                const float *tr = t + ((size_t)row * 3 + blk) * RP;
                float dlt = 0.f;
                for (int r = 0; r < ad.rank; ++r) dlt += ldf(B + r) * tr[r];
                v += dlt;
            }
            if (residual) v += ldf(residual + (size_t)row * N + n);
            stf(y + (size_t)row * N + n, v);
        }
    }
}

// ---------------------------------------------------------------------------------------------
// KV append (both data types): one 16-byte vector per thread.  Row t's k part
// qkv[t][Nq .. Nq+Nkv) goes to pool[page][0][head][row][:], its v part to plane 1.  Tokens whose
// slot is -1 (rejected by the metadata step) are skipped.
// ---------------------------------------------------------------------------------------------
__global__ void kv_append_kernel(const uint4 *__restrict__ qkv, const int32_t *__restrict__ slot_map,
                                 int T, int N_vec, int Nq_vec, int Nkv_vec, int hd_vec, int Hkv,
                                 int page_size, int num_pages, uint4 *__restrict__ pool, int32_t *status) {
    const size_t total = (size_t)T * 2 * Nkv_vec;
    for (size_t i = blockIdx.x * (size_t)blockDim.x + threadIdx.x; i < total;
         i += (size_t)gridDim.x * blockDim.x) {
        const int t = (int)(i / (2 * Nkv_vec));
        const int c = (int)(i % (2 * Nkv_vec));   // vector column inside [k | v]
        const int plane = c / Nkv_vec, cc = c % Nkv_vec;
        const int head = cc / hd_vec, dv = cc % hd_vec;
        const int slot = slot_map[t];
        if (slot < 0) continue;
        const int page = slot / page_size, row = slot % page_size;
        if (page >= num_pages) { report(status, ALORA_ERR_PAGE_RANGE); continue; }
        const size_t dst = ((((size_t)page * 2 + plane) * Hkv + head) * page_size + row) * hd_vec + dv;
        pool[dst] = qkv[(size_t)t * N_vec + Nq_vec + c];
    }
}

int launch_kv_append(alora_ctx *ctx, const void *qkv, int T, int num_pages, void *pool, cudaStream_t s) {
    if (T == 0) return 0;
    const Dims &d = ctx->d;
    ProfScope prof(ctx, KK_KV_APPEND, s);
    const int vec = 16 / (int)ctx->esize;  // elements per 16-byte vector
    const size_t total = (size_t)T * 2 * (d.Nkv / vec);
    int blocks = (int)((total + 255) / 256);
    if (blocks > ctx->sm_count * 16) blocks = ctx->sm_count * 16;
    kv_append_kernel<<<blocks, 256, 0, s>>>((const uint4 *)qkv, ctx->d_slot, T, d.N / vec, d.Nq / vec,
                                            d.Nkv / vec, d.hd / vec, d.Hkv, d.page, num_pages, (uint4 *)pool,
                                            ctx->d_status);
    return 1;
}

// ---------------------------------------------------------------------------------------------
// Optional rotary position embedding fused with the KV append (both data types).  The paper's equations carry no
// positional rotation; with a base theta configured, the new query and key rows are rotated by their positions
// ("rotate-half": column i of a head pairs with column i + hd/2, angle p * theta^(-2i/hd)) after the projection and
// before the keys are cached, so the cache holds post-rotation keys.  One thread per (token, head, 16-byte vector
// of pair indices): it rotates the pairs in place in the fused q/k/v row and, for key heads, also writes the rotated
// vectors to the token's cache slot; a second index range copies the value rows to the cache.  The angle is formed
// and reduced to [-pi, pi] in double precision (positions reach tens of thousands of radians), the sine and
// cosine of the remainder in single.  Without a pool only the in-place rotation happens.
// ---------------------------------------------------------------------------------------------
template <typename T> struct Vec16;
template <> struct Vec16<float> { static constexpr int kElems = 4; };
template <> struct Vec16<__nv_bfloat16> { static constexpr int kElems = 8; };

__device__ __forceinline__ void unpack16(const uint4 &u, float (&f)[4]) {
    f[0] = __uint_as_float(u.x); f[1] = __uint_as_float(u.y); f[2] = __uint_as_float(u.z); f[3] = __uint_as_float(u.w);
}
__device__ __forceinline__ void unpack16(const uint4 &u, float (&f)[8]) {
    const uint32_t w[4] = {u.x, u.y, u.z, u.w};
#pragma unroll
    for (int e = 0; e < 4; ++e) {
        const __nv_bfloat162 b2 = *reinterpret_cast<const __nv_bfloat162 *>(&w[e]);
        f[2 * e] = __low2float(b2); f[2 * e + 1] = __high2float(b2);
    }
}
__device__ __forceinline__ uint4 pack16(const float (&f)[4]) {
    return make_uint4(__float_as_uint(f[0]), __float_as_uint(f[1]), __float_as_uint(f[2]), __float_as_uint(f[3]));
}
__device__ __forceinline__ uint4 pack16(const float (&f)[8]) {
    uint4 u;
    __nv_bfloat162 v;
    v = __floats2bfloat162_rn(f[0], f[1]); u.x = *reinterpret_cast<uint32_t *>(&v);
    v = __floats2bfloat162_rn(f[2], f[3]); u.y = *reinterpret_cast<uint32_t *>(&v);
    v = __floats2bfloat162_rn(f[4], f[5]); u.z = *reinterpret_cast<uint32_t *>(&v);
    v = __floats2bfloat162_rn(f[6], f[7]); u.w = *reinterpret_cast<uint32_t *>(&v);
    return u;
}

template <typename T>
__global__ void rope_append_kernel(uint4 *__restrict__ qkv, const int32_t *__restrict__ positions,
                                   const int32_t *__restrict__ slot_map, const double *__restrict__ inv_freq, int Tn,
                                   int N_vec, int n_rot_heads, int n_q_heads, int hd_vec, int Hkv, int page_size,
                                   int num_pages, uint4 *__restrict__ pool, int32_t *status) {
    constexpr int kE = Vec16<T>::kElems;
    const int half_vec = hd_vec / 2;                       // vectors per half head
    const int rot_units = n_rot_heads * half_vec;          // per token: (head, vector of pair indices)
    const int copy_units = pool != nullptr ? Hkv * hd_vec : 0;   // per token: vectors of the value row
    const int per_tok = rot_units + copy_units;
    const size_t total = (size_t)Tn * per_tok;
    for (size_t idx = blockIdx.x * (size_t)blockDim.x + threadIdx.x; idx < total; idx += (size_t)gridDim.x * blockDim.x) {
        const int t = (int)(idx / per_tok), u = (int)(idx % per_tok);
        int page = -1, prow = 0;
        if (pool != nullptr) {
            const int slot = slot_map[t];
            if (slot >= 0) {
                page = slot / page_size; prow = slot % page_size;
                if (page >= num_pages) { report(status, ALORA_ERR_PAGE_RANGE); page = -1; }
            }
        }
        uint4 *row = qkv + (size_t)t * N_vec;
        if (u < rot_units) {
            const int h = u / half_vec, iv = u % half_vec;   // heads 0 .. n_q_heads-1 are queries, the rest keys
            uint4 *lo_p = row + (size_t)h * hd_vec + iv, *hi_p = lo_p + half_vec;
            float lo[kE], hi[kE];
            unpack16(*lo_p, lo); unpack16(*hi_p, hi);
            const double p = (double)positions[t];
#pragma unroll
            for (int e = 0; e < kE; ++e) {
                const double a = p * inv_freq[iv * kE + e];
                const float r = (float)(a - 6.283185307179586476925 * rint(a * 0.15915494309189533577));
                float sn, cs;
                sincosf(r, &sn, &cs);
                const float x0 = lo[e], x1 = hi[e];
                lo[e] = x0 * cs - x1 * sn;
                hi[e] = x1 * cs + x0 * sn;
            }
            const uint4 lo_u = pack16(lo), hi_u = pack16(hi);
            *lo_p = lo_u; *hi_p = hi_u;
            if (h >= n_q_heads && page >= 0) {   // a key head: the rotated vectors also go to the cache slot
                const int kh = h - n_q_heads;
                uint4 *dst = pool + ((((size_t)page * 2 + 0) * Hkv + kh) * page_size + prow) * hd_vec + iv;
                dst[0] = lo_u; dst[half_vec] = hi_u;
            }
        } else if (page >= 0) {
            const int c = u - rot_units, kh = c / hd_vec, dv = c % hd_vec;
            pool[((((size_t)page * 2 + 1) * Hkv + kh) * page_size + prow) * hd_vec + dv] =
                row[(size_t)(n_rot_heads + kh) * hd_vec + dv];
        }
    }
}

// ---------------------------------------------------------------------------------------------
// Copy-on-write of a shared partial tail page.  Requests that reuse one base-model cache point at the same physical
// pages; when the reused length is not a multiple of the page size, the page that holds the last cached positions
// would also receive the request's first new rows.  Before the layer call, every such request gets a page of its
// own: rows 0 .. (first new position % page_size) - 1 of the shared page are copied to the fresh page (both planes,
// all KV heads) and the request's block-table entry is redirected.  One block per request.
// ---------------------------------------------------------------------------------------------
__global__ void cow_tail_pages_kernel(const int32_t *__restrict__ qsl, const int32_t *__restrict__ seq_lens,
                                      int32_t *__restrict__ block_tables, int max_blocks, int num_pages, int page_size,
                                      int Hkv, int hd_vec, const int32_t *__restrict__ fresh_pages,
                                      uint4 *__restrict__ pool, int32_t *status) {
    const int r = blockIdx.x;
    const int fresh = fresh_pages[r];
    if (fresh < 0) return;
    const int n_new = qsl[r + 1] - qsl[r];
    const int p_first = seq_lens[r] - n_new;
    const int blk = p_first / page_size, rows = p_first % page_size;
    if (n_new <= 0 || p_first < 0 || blk >= max_blocks) { if (threadIdx.x == 0) report(status, ALORA_ERR_BAD_BATCH); return; }
    const int old = block_tables[(size_t)r * max_blocks + blk];
    if (fresh >= num_pages || old < 0 || old >= num_pages) { if (threadIdx.x == 0) report(status, ALORA_ERR_PAGE_RANGE); return; }
    const int per_head = rows * hd_vec, total = 2 * Hkv * per_head;
    for (int i = threadIdx.x; i < total; i += blockDim.x) {
        const int ph = i / per_head, v = i % per_head;    // (plane, head), vector inside the head's first `rows` rows
        const size_t off = (size_t)ph * page_size * hd_vec + v;
        pool[(size_t)fresh * 2 * Hkv * page_size * hd_vec + off] = pool[(size_t)old * 2 * Hkv * page_size * hd_vec + off];
    }
    __syncthreads();
    if (threadIdx.x == 0) block_tables[(size_t)r * max_blocks + blk] = fresh;
}

int launch_cow_tail_pages(alora_ctx *ctx, const int32_t *qsl, const int32_t *seq_lens, int32_t *block_tables, int max_blocks,
                          int num_pages, int R, const int32_t *fresh_pages, void *pool, cudaStream_t s) {
    if (R == 0) return 0;
    const Dims &d = ctx->d;
    const int vec = 16 / (int)ctx->esize;
    cow_tail_pages_kernel<<<R, 256, 0, s>>>(qsl, seq_lens, block_tables, max_blocks, num_pages, d.page, d.Hkv, d.hd / vec,
                                            fresh_pages, (uint4 *)pool, ctx->d_status);
    return 1;
}

// Rotates the query and key parts of qkv[T][N] in place; with a pool also appends the (rotated) keys and the values.
int launch_rope(alora_ctx *ctx, void *qkv, const int32_t *positions, int T, void *pool, int num_pages, cudaStream_t s) {
    if (T == 0) return 0;
    const Dims &d = ctx->d;
    if (ctx->d_rope_inv_freq == nullptr) return -1;
    const int vec = 16 / (int)ctx->esize;
    if (d.hd % (2 * vec) != 0) return -1;
    ProfScope prof(ctx, KK_KV_APPEND, s);
    const int hd_vec = d.hd / vec;
    const size_t per_tok = (size_t)(d.Hq + d.Hkv) * (hd_vec / 2) + (pool ? (size_t)d.Hkv * hd_vec : 0);
    const size_t total = (size_t)T * per_tok;
    int blocks = (int)std::min<size_t>((total + 255) / 256, (size_t)ctx->sm_count * 16);
    if (ctx->cfg.dtype == ALORA_DTYPE_FP32)
        rope_append_kernel<float><<<blocks, 256, 0, s>>>((uint4 *)qkv, positions, ctx->d_slot, ctx->d_rope_inv_freq, T,
                                                         d.N / vec, d.Hq + d.Hkv, d.Hq, hd_vec, d.Hkv, d.page, num_pages,
                                                         (uint4 *)pool, ctx->d_status);
    else
        rope_append_kernel<__nv_bfloat16><<<blocks, 256, 0, s>>>((uint4 *)qkv, positions, ctx->d_slot,
                                                                 ctx->d_rope_inv_freq, T, d.N / vec, d.Hq + d.Hkv, d.Hq,
                                                                 hd_vec, d.Hkv, d.page, num_pages, (uint4 *)pool,
                                                                 ctx->d_status);
    return 1;
}

// ---------------------------------------------------------------------------------------------
// CUDA-core attention (Eq. 1 / Eq. 3): one warp per (token, query head); the block holds the G query
// heads that share a KV head.  Keys are taken 32 at a time: lane j scores key j0 + j against the
// query kept in shared memory, the warp combines the 32 scores with shuffles (running maximum and
// sum: online softmax), then every lane accumulates its slice of the head dimension over the 32
// value rows.
// ---------------------------------------------------------------------------------------------
template <typename T, int HD>
__global__ void attn_simt_kernel(const T *__restrict__ qkv, const int32_t *__restrict__ positions,
                                const int32_t *__restrict__ token_req, const int32_t *__restrict__ slot_map,
                                const int32_t *__restrict__ block_tables, int max_blocks, int num_pages, int page_size, int N, int Nq, int Hkv, int G,
                                float scale, const T *__restrict__ pool, T *__restrict__ out,
                                 int32_t *status) {
    extern __shared__ float q_s[];  // [G][HD]
    constexpr int DPL = HD / 32;    // head-dim elements per lane
    const int t = blockIdx.x, kvh = blockIdx.y;
    const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
    const int h = kvh * G + warp;
    const int r = token_req[t];
    const int p = positions[t];
    if (slot_map[t] < 0) {  // token rejected by the metadata step: defined output, no cache access
        for (int d = lane; d < HD; d += 32) stf(out + (size_t)t * Nq + (size_t)h * HD + d, 0.f);
        return;
    }
    float *qs = q_s + warp * HD;
    for (int d = lane; d < HD; d += 32) qs[d] = ldf(qkv + (size_t)t * N + (size_t)h * HD + d) * scale;
    __syncwarp();
    float m = -INFINITY, l = 0.f, acc[DPL];
#pragma unroll
    for (int i = 0; i < DPL; ++i) acc[i] = 0.f;
    const size_t plane_stride = (size_t)Hkv * page_size * HD;
    for (int j0 = 0; j0 <= p; j0 += 32) {
        const int j = j0 + lane;
        float s = -INFINITY;
        const T *krow = nullptr;
        if (j <= p) {
            const int page = block_tables[(size_t)r * max_blocks + j / page_size];
            if (page >= 0 && page < num_pages) {
                krow = pool + ((size_t)page * 2 * Hkv + kvh) * page_size * HD + (size_t)(j % page_size) * HD;
                float dot = 0.f;
#pragma unroll 8
                for (int d = 0; d < HD; ++d) dot += qs[d] * ldf(krow + d);
                s = dot;
            } else {
                report(status, ALORA_ERR_PAGE_RANGE);
            }
        }
        float mx = s;
        for (int off = 16; off; off >>= 1) mx = fmaxf(mx, __shfl_xor_sync(0xffffffffu, mx, off));
        const float m_new = fmaxf(m, mx);
        if (m_new == -INFINITY) continue;  // nothing visible in this group (only on bad pages)
        const float w = (s == -INFINITY) ? 0.f : __expf(s - m_new);
        float wsum = w;
        for (int off = 16; off; off >>= 1) wsum += __shfl_xor_sync(0xffffffffu, wsum, off);
        const float corr = (m == -INFINITY) ? 0.f : __expf(m - m_new);
        l = l * corr + wsum;
#pragma unroll
        for (int i = 0; i < DPL; ++i) acc[i] *= corr;
        const int nvis = min(32, p - j0 + 1);
        for (int jj = 0; jj < nvis; ++jj) {
            const float wj = __shfl_sync(0xffffffffu, w, jj);
            const unsigned long long kp = __shfl_sync(0xffffffffu, (unsigned long long)krow, jj);
            if (kp == 0ull) continue;
            const T *vrow = (const T *)kp + plane_stride;
#pragma unroll
            for (int i = 0; i < DPL; ++i) acc[i] += wj * ldf(vrow + lane + 32 * i);
        }
        m = m_new;
    }
    const float inv = l > 0.f ? 1.f / l : 0.f;
#pragma unroll
    for (int i = 0; i < DPL; ++i) stf(out + (size_t)t * Nq + (size_t)h * HD + lane + 32 * i, acc[i] * inv);
}

// ---------------------------------------------------------------------------------------------
// RMSNorm and SwiGLU (decoder-stack glue; both data types, fp32 arithmetic).
// ---------------------------------------------------------------------------------------------
template <typename T>
__global__ void rmsnorm_kernel(const T *__restrict__ x, const T *__restrict__ w, int H, float eps,
                               T *__restrict__ y) {
    const size_t row = blockIdx.x;
    __shared__ float red[32];
    float ss = 0.f;
    for (int h = threadIdx.x; h < H; h += blockDim.x) { float v = ldf(x + row * H + h); ss += v * v; }
    for (int off = 16; off; off >>= 1) ss += __shfl_xor_sync(0xffffffffu, ss, off);
    if ((threadIdx.x & 31) == 0) red[threadIdx.x >> 5] = ss;
    __syncthreads();
    if (threadIdx.x < 32) {
        float v = threadIdx.x < (blockDim.x >> 5) ? red[threadIdx.x] : 0.f;
        for (int off = 16; off; off >>= 1) v += __shfl_xor_sync(0xffffffffu, v, off);
        if (threadIdx.x == 0) red[0] = rsqrtf(v / (float)H + eps);
    }
    __syncthreads();
    const float inv = red[0];
    for (int h = threadIdx.x; h < H; h += blockDim.x)
        stf(y + row * H + h, ldf(x + row * H + h) * inv * ldf(w + h));
}

template <typename T>
__global__ void swiglu_kernel(const T *__restrict__ gate_up, int I, size_t total, T *__restrict__ y) {
    for (size_t i = blockIdx.x * (size_t)blockDim.x + threadIdx.x; i < total;
         i += (size_t)gridDim.x * blockDim.x) {
        const size_t row = i / I, c = i % I;
        const float g = ldf(gate_up + row * 2 * I + c), u = ldf(gate_up + row * 2 * I + I + c);
        stf(y + i, g / (1.f + __expf(-g)) * u);
    }
}

// bf16 rows of up to 8192 elements (H a multiple of 8): the row is read once, 16 bytes per load and all of a thread's
// loads in flight together, kept in registers across the reduction, and written with 16-byte stores.  (The generic
// kernel above reads the row twice with one dependent 2-byte load per loop trip: 17 us for 8 rows of 4096, most of it
// memory latency.)  Launched as a programmatic dependent: the next kernel's prologue may start under this one.
constexpr int kNormVecs = 4;
__global__ void __launch_bounds__(256) rmsnorm_bf16_kernel(const __nv_bfloat16 *__restrict__ x,
                                                           const __nv_bfloat16 *__restrict__ w, int H, float eps,
                                                           __nv_bfloat16 *__restrict__ y) {
    tc::grid_dep_launch();
    tc::grid_dep_wait();
    const size_t row = blockIdx.x;
    const int nvec = H >> 3;
    __shared__ float red[32];
    uint4 v[kNormVecs];
    float ss = 0.f;
#pragma unroll
    for (int i = 0; i < kNormVecs; ++i) {
        const int idx = (int)threadIdx.x + i * 256;
        v[i] = idx < nvec ? *reinterpret_cast<const uint4 *>(x + row * H + (size_t)idx * 8) : make_uint4(0u, 0u, 0u, 0u);
    }
#pragma unroll
    for (int i = 0; i < kNormVecs; ++i) {
        const __nv_bfloat162 *p = reinterpret_cast<const __nv_bfloat162 *>(&v[i]);
#pragma unroll
        for (int e = 0; e < 4; ++e) { const float2 f = __bfloat1622float2(p[e]); ss = fmaf(f.x, f.x, fmaf(f.y, f.y, ss)); }
    }
    for (int off = 16; off; off >>= 1) ss += __shfl_xor_sync(0xffffffffu, ss, off);
    if ((threadIdx.x & 31) == 0) red[threadIdx.x >> 5] = ss;
    __syncthreads();
    if (threadIdx.x < 32) {
        float t = threadIdx.x < 8 ? red[threadIdx.x] : 0.f;
        for (int off = 4; off; off >>= 1) t += __shfl_xor_sync(0xffffffffu, t, off);
        if (threadIdx.x == 0) red[0] = rsqrtf(t / (float)H + eps);
    }
    __syncthreads();
    const float inv = red[0];
#pragma unroll
    for (int i = 0; i < kNormVecs; ++i) {
        const int idx = (int)threadIdx.x + i * 256;
        if (idx >= nvec) continue;
        const uint4 wv = *reinterpret_cast<const uint4 *>(w + (size_t)idx * 8);
        const __nv_bfloat162 *px = reinterpret_cast<const __nv_bfloat162 *>(&v[i]);
        const __nv_bfloat162 *pw = reinterpret_cast<const __nv_bfloat162 *>(&wv);
        uint4 o;
        __nv_bfloat162 *po = reinterpret_cast<__nv_bfloat162 *>(&o);
#pragma unroll
        for (int e = 0; e < 4; ++e) {
            const float2 a = __bfloat1622float2(px[e]), g = __bfloat1622float2(pw[e]);
            po[e] = __floats2bfloat162_rn(a.x * inv * g.x, a.y * inv * g.y);
        }
        *reinterpret_cast<uint4 *>(y + row * H + (size_t)idx * 8) = o;
    }
}

// SwiGLU on bf16 rows, eight columns per thread (I a multiple of 8): 16-byte loads of gate and up, 16-byte store.
__global__ void __launch_bounds__(256) swiglu_bf16_kernel(const __nv_bfloat16 *__restrict__ gate_up, int I, size_t total_vecs,
                                                          __nv_bfloat16 *__restrict__ y) {
    tc::grid_dep_launch();
    tc::grid_dep_wait();
    const int vecs_per_row = I >> 3;
    for (size_t i = blockIdx.x * (size_t)blockDim.x + threadIdx.x; i < total_vecs; i += (size_t)gridDim.x * blockDim.x) {
        const size_t row = i / vecs_per_row, c = (i - row * vecs_per_row) * 8;
        const uint4 gv = *reinterpret_cast<const uint4 *>(gate_up + row * 2 * I + c);
        const uint4 uv = *reinterpret_cast<const uint4 *>(gate_up + row * 2 * I + I + c);
        const __nv_bfloat162 *pg = reinterpret_cast<const __nv_bfloat162 *>(&gv);
        const __nv_bfloat162 *pu = reinterpret_cast<const __nv_bfloat162 *>(&uv);
        uint4 o;
        __nv_bfloat162 *po = reinterpret_cast<__nv_bfloat162 *>(&o);
#pragma unroll
        for (int e = 0; e < 4; ++e) {
            const float2 g = __bfloat1622float2(pg[e]), u = __bfloat1622float2(pu[e]);
            po[e] = __floats2bfloat162_rn(g.x / (1.f + __expf(-g.x)) * u.x, g.y / (1.f + __expf(-g.y)) * u.y);
        }
        *reinterpret_cast<uint4 *>(y + row * I + c) = o;
    }
}

int launch_rmsnorm(alora_ctx *ctx, const void *x, const void *w, int T, void *y, cudaStream_t s) {
    if (T == 0) return 0;
    ProfScope prof(ctx, KK_GLUE, s);
    const int H = ctx->d.H;
    const bool al16 = (((uintptr_t)x | (uintptr_t)w | (uintptr_t)y) & 15) == 0;
    if (ctx->cfg.dtype == ALORA_DTYPE_BF16 && H % 8 == 0 && H <= 8 * 256 * kNormVecs && al16)
        return launch_kernel(rmsnorm_bf16_kernel, dim3(T), dim3(256), 0, s, true, (const __nv_bfloat16 *)x,
                             (const __nv_bfloat16 *)w, H, ctx->cfg.rms_eps, (__nv_bfloat16 *)y) == cudaSuccess ? 1 : -1;
    if (ctx->cfg.dtype == ALORA_DTYPE_FP32)
        rmsnorm_kernel<float><<<T, 256, 0, s>>>((const float *)x, (const float *)w, ctx->d.H, ctx->cfg.rms_eps, (float *)y);
    else
        rmsnorm_kernel<__nv_bfloat16><<<T, 256, 0, s>>>((const __nv_bfloat16 *)x, (const __nv_bfloat16 *)w, ctx->d.H,
                                                        ctx->cfg.rms_eps, (__nv_bfloat16 *)y);
    return 1;
}

int launch_swiglu(alora_ctx *ctx, const void *gate_up, int T, void *y, cudaStream_t s) {
    if (T == 0) return 0;
    ProfScope prof(ctx, KK_GLUE, s);
    const size_t total = (size_t)T * ctx->d.I;
    int blocks = (int)((total + 255) / 256);
    if (blocks > ctx->sm_count * 16) blocks = ctx->sm_count * 16;
    if (ctx->cfg.dtype == ALORA_DTYPE_BF16 && ctx->d.I % 8 == 0 && (((uintptr_t)gate_up | (uintptr_t)y) & 15) == 0) {
        const size_t vecs = total / 8;
        const int vblocks = (int)std::min<size_t>((vecs + 255) / 256, (size_t)ctx->sm_count * 16);
        return launch_kernel(swiglu_bf16_kernel, dim3(vblocks), dim3(256), 0, s, true, (const __nv_bfloat16 *)gate_up,
                             ctx->d.I, vecs, (__nv_bfloat16 *)y) == cudaSuccess ? 1 : -1;
    }
    if (ctx->cfg.dtype == ALORA_DTYPE_FP32)
        swiglu_kernel<float><<<blocks, 256, 0, s>>>((const float *)gate_up, ctx->d.I, total, (float *)y);
    else
        swiglu_kernel<__nv_bfloat16><<<blocks, 256, 0, s>>>((const __nv_bfloat16 *)gate_up, ctx->d.I, total,
                                                           (__nv_bfloat16 *)y);
    return 1;
}

// ---- launchers of the CUDA-core projection / attention, by data type -------------------------------
template <typename T>
static int project_simt(alora_ctx *ctx, int layer, const void *hidden, int Tn, void *qkv, cudaStream_t s) {
    const Dims &d = ctx->d;
    const AdapterDev *ads = ctx->d_adapters + (size_t)layer * ctx->cfg.max_adapters;
    {
        ProfScope prof(ctx, KK_SHRINK, s);
        shrink_simt_kernel<T><<<Tn, 256, 0, s>>>((const T *)hidden, ctx->d_row_adapter, ads, d.H, d.RP, (float *)ctx->d_t);
    }
    ProfScope prof(ctx, KK_PROJECT, s);
    dim3 grid((d.N + 63) / 64, (Tn + 63) / 64);
    linear_simt_kernel<T><<<grid, 256, 0, s>>>((const T *)hidden, (const T *)ctx->layers[layer].wqkv, Tn, d.H, d.N,
                                               ctx->d_row_adapter, ads, (const float *)ctx->d_t, d.RP, d.Nq, d.Nkv,
                                               nullptr, (T *)qkv);
    return 2;
}

int launch_project_simt(alora_ctx *ctx, int layer, const void *hidden, int T, void *qkv, cudaStream_t s) {
    if (T == 0) return 0;
    return ctx->cfg.dtype == ALORA_DTYPE_FP32 ? project_simt<float>(ctx, layer, hidden, T, qkv, s)
                                              : project_simt<__nv_bfloat16>(ctx, layer, hidden, T, qkv, s);
}

int launch_linear_simt(alora_ctx *ctx, const void *x, const void *W, int T, int K, int N, void *y,
                       const void *residual, cudaStream_t s) {
    if (T == 0) return 0;
    ProfScope prof(ctx, KK_LINEAR, s);
    dim3 grid((N + 63) / 64, (T + 63) / 64);
    if (ctx->cfg.dtype == ALORA_DTYPE_FP32)
        linear_simt_kernel<float><<<grid, 256, 0, s>>>((const float *)x, (const float *)W, T, K, N, nullptr, nullptr,
                                                       nullptr, 0, 0, 0, (const float *)residual, (float *)y);
    else
        linear_simt_kernel<__nv_bfloat16><<<grid, 256, 0, s>>>((const __nv_bfloat16 *)x, (const __nv_bfloat16 *)W, T, K,
                                                               N, nullptr, nullptr, nullptr, 0, 0, 0,
                                                               (const __nv_bfloat16 *)residual, (__nv_bfloat16 *)y);
    return 1;
}

template <typename T>
static int attend_simt(alora_ctx *ctx, const void *qkv, const BatchArgs &b, const void *pool, void *out,
                       cudaStream_t s) {
    const Dims &d = ctx->d;
    ProfScope prof(ctx, KK_ATTENTION, s);
    dim3 grid(b.T, d.Hkv);
    const int threads = 32 * d.G;
    const size_t smem = (size_t)d.G * d.hd * sizeof(float);
#define ALORA_ATTN_SIMT(HD)                                                                              \
    attn_simt_kernel<T, HD><<<grid, threads, smem, s>>>((const T *)qkv, b.positions, ctx->d_token_req,   \
                                                        ctx->d_slot, b.block_tables, b.max_blocks, b.num_pages, d.page, \
                                                        d.N, d.Nq, d.Hkv, d.G, d.softmax_scale,           \
                                                        (const T *)pool, (T *)out, ctx->d_status)
    if (d.hd == 32) ALORA_ATTN_SIMT(32);
    else if (d.hd == 64) ALORA_ATTN_SIMT(64);
    else if (d.hd == 128) ALORA_ATTN_SIMT(128);
    else return -1;
#undef ALORA_ATTN_SIMT
    return 1;
}

int launch_attend_simt(alora_ctx *ctx, const void *qkv, const BatchArgs &b, const void *pool, void *out,
                       cudaStream_t s) {
    if (b.T == 0) return 0;
    return ctx->cfg.dtype == ALORA_DTYPE_FP32 ? attend_simt<float>(ctx, qkv, b, pool, out, s)
                                              : attend_simt<__nv_bfloat16>(ctx, qkv, b, pool, out, s);
}

}  // namespace alora

// alora_project_qkv_static: the gated q/k/v projection for callers that must not allocate.
//
// Who needs this: code that runs after a serving engine has handed the whole device to its own memory
// pool (a cudaMalloc there fails or fragments the pool), code on a latency-critical path where the
// implicit device synchronisation of cudaMalloc / cudaFree is not acceptable, and plug-ins that are
// simply forbidden to call the allocator.  Such a caller cannot use alora_create (it allocates the
// context's workspaces), so this entry point takes every input and output as an argument and keeps
// its scratch (the per-row gate and the rank-r intermediate t = s * A x) in a fixed array that is
// part of the loaded library image.  It calls no cudaMalloc / cudaFree and no allocating library
// routine.
//
// The array below occupies kScratchBytes of device memory on EVERY GPU that loads this library, from
// load until the process exits.  All calls on one device share it and it keeps the previous call's
// contents: a call rewrites every scratch element it later reads (the gate of all T rows, t of every
// gated row), so nothing has to be cleared, but two calls that overlap on the same GPU (different
// streams, or different host threads) race on it and must be serialised by the caller.
#include <cuda_bf16.h>
#include <cuda_runtime.h>
#include <stdint.h>

#include "alora.h"

namespace {

constexpr int kMaxTokens = ALORA_STATIC_MAX_TOKENS;
constexpr int kMaxRank = ALORA_STATIC_MAX_RANK;
constexpr size_t kGateBytes = (size_t)kMaxTokens * sizeof(int32_t);
constexpr size_t kTBytes = (size_t)kMaxTokens * 3 * kMaxRank * sizeof(float);
constexpr size_t kScratchBytes = kGateBytes + kTBytes;  // 16 KiB + 3 MiB

// In host code this name is only a handle for cudaGetSymbolAddress; it is not a device address.
static __device__ __align__(256) unsigned char g_static_scratch[kScratchBytes];

constexpr int kMaxDevices = 64;
void *g_scratch_addr[kMaxDevices] = {};  // device address of g_static_scratch, per device ordinal

template <typename T> __device__ __forceinline__ float ldf(const T *p);
template <> __device__ __forceinline__ float ldf<float>(const float *p) { return *p; }
template <> __device__ __forceinline__ float ldf<__nv_bfloat16>(const __nv_bfloat16 *p) { return __bfloat162float(*p); }
template <typename T> __device__ __forceinline__ void stf(T *p, float v);
template <> __device__ __forceinline__ void stf<float>(float *p, float v) { *p = v; }
template <> __device__ __forceinline__ void stf<__nv_bfloat16>(__nv_bfloat16 *p, float v) { *p = __float2bfloat16_rn(v); }

// gate[t] = 1 iff the row's request uses the adapter and position >= activation offset (Eq. 5).
__global__ void static_gate_kernel(const int32_t *__restrict__ positions, const int32_t *__restrict__ qsl,
                                   const int32_t *__restrict__ a_req, const int32_t *__restrict__ adapter_on,
                                   int T, int R, int32_t *__restrict__ gate) {
    const int t = blockIdx.x * blockDim.x + threadIdx.x;
    if (t >= T) return;
    int lo = 0, hi = R;
    while (hi - lo > 1) {
        const int mid = (lo + hi) >> 1;
        if (qsl[mid] <= t) lo = mid; else hi = mid;
    }
    const bool on = adapter_on == nullptr || adapter_on[lo] != 0;
    gate[t] = (on && positions[t] >= a_req[lo]) ? 1 : 0;
}

// t[row][blk][i] = scale * sum_h A_blk[i][h] x[row][h] for gated rows; one block per row.
template <typename T>
__global__ void static_shrink_kernel(const T *__restrict__ x, const int32_t *__restrict__ gate, const T *Aq,
                                     const T *Ak, const T *Av, int rank, float scale, int H,
                                     float *__restrict__ t) {
    const int row = blockIdx.x;
    if (!gate[row]) return;
    const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31, nwarps = blockDim.x >> 5;
    for (int o = warp; o < 3 * rank; o += nwarps) {
        const int blk = o / rank, i = o % rank;
        const T *a = (blk == 0 ? Aq : (blk == 1 ? Ak : Av)) + (size_t)i * H;
        float acc = 0.f;
        for (int h = lane; h < H; h += 32) acc += ldf(a + h) * ldf(x + (size_t)row * H + h);
        for (int off = 16; off; off >>= 1) acc += __shfl_xor_sync(0xffffffffu, acc, off);
        if (lane == 0) t[((size_t)row * 3 + blk) * rank + i] = acc * scale;
    }
}

// y[row][n] = sum_h W[n][h] x[row][h] (+ sum_i B_blk[n'][i] t[row][blk][i] on gated rows).
// 64x64 tile per block, 4x4 outputs per thread, K staged through shared memory.
template <typename T>
__global__ void __launch_bounds__(256)
static_project_kernel(const T *__restrict__ x, const T *__restrict__ W, int Tn, int H, int Nq, int Nkv,
                      const int32_t *__restrict__ gate, const float *__restrict__ t, const T *Bq, const T *Bk,
                      const T *Bv, int rank, T *__restrict__ y) {
    __shared__ float xs[16][64 + 1], ws[16][64 + 1];
    const int N = Nq + 2 * Nkv;
    const int tx = threadIdx.x & 15, ty = threadIdx.x >> 4;
    const int row0 = blockIdx.y * 64, col0 = blockIdx.x * 64;
    float acc[4][4] = {};
    for (int k0 = 0; k0 < H; k0 += 16) {
        for (int i = threadIdx.x; i < 64 * 16; i += 256) {
            const int rr = i >> 4, kk = i & 15;
            const int gr = row0 + rr, gc = col0 + rr, gk = k0 + kk;
            xs[kk][rr] = (gr < Tn && gk < H) ? ldf(x + (size_t)gr * H + gk) : 0.f;
            ws[kk][rr] = (gc < N && gk < H) ? ldf(W + (size_t)gc * H + gk) : 0.f;
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
        const bool on = gate[row] != 0;
#pragma unroll
        for (int j = 0; j < 4; ++j) {
            const int n = col0 + tx * 4 + j;
            if (n >= N) continue;
            float v = acc[i][j];
            if (on) {
                const int blk = n < Nq ? 0 : (n < Nq + Nkv ? 1 : 2);
                const T *B = blk == 0 ? Bq + (size_t)n * rank
                                      : (blk == 1 ? Bk + (size_t)(n - Nq) * rank : Bv + (size_t)(n - Nq - Nkv) * rank);
                const float *tr = t + ((size_t)row * 3 + blk) * rank;
                float d = 0.f;
                for (int r = 0; r < rank; ++r) d += ldf(B + r) * tr[r];
                v += d;
            }
            stf(y + (size_t)row * N + n, v);
        }
    }
}

template <typename T>
void launch_all(const void *x, const void *W, const int32_t *pos, const int32_t *qsl, const int32_t *a_req,
                const int32_t *on, int rank, float scale, const void *Aq, const void *Bq, const void *Ak,
                const void *Bk, const void *Av, const void *Bv, int Tn, int R, int H, int Nq, int Nkv, void *y,
                void *scratch, cudaStream_t s) {
    int32_t *gate = (int32_t *)scratch;
    float *t = (float *)((unsigned char *)scratch + kGateBytes);
    static_gate_kernel<<<(Tn + 255) / 256, 256, 0, s>>>(pos, qsl, a_req, on, Tn, R, gate);
    static_shrink_kernel<T><<<Tn, 256, 0, s>>>((const T *)x, gate, (const T *)Aq, (const T *)Ak, (const T *)Av, rank,
                                               scale, H, t);
    dim3 grid((Nq + 2 * Nkv + 63) / 64, (Tn + 63) / 64);
    static_project_kernel<T><<<grid, 256, 0, s>>>((const T *)x, (const T *)W, Tn, H, Nq, Nkv, gate, t, (const T *)Bq,
                                                  (const T *)Bk, (const T *)Bv, rank, (T *)y);
}

}  // namespace

extern "C" alora_status alora_project_qkv_static(int dtype, int hidden, int n_q, int n_kv, const void *d_hidden,
                                                 const void *d_wqkv, const int32_t *d_positions,
                                                 const int32_t *d_query_start_loc,
                                                 const int32_t *d_activation_offsets,
                                                 const int32_t *d_adapter_on, int rank, float scale,
                                                 const void *d_Aq, const void *d_Bq, const void *d_Ak,
                                                 const void *d_Bk, const void *d_Av, const void *d_Bv, int T, int R,
                                                 void *d_qkv, void *stream) {
    if (!d_hidden || !d_wqkv || !d_positions || !d_query_start_loc || !d_activation_offsets || !d_qkv || !d_Aq ||
        !d_Bq || !d_Ak || !d_Bk || !d_Av || !d_Bv)
        return ALORA_ERR_INVALID_ARG;
    if (hidden <= 0 || n_q <= 0 || n_kv <= 0 || T < 0 || R < 0) return ALORA_ERR_INVALID_ARG;
    if (dtype != ALORA_DTYPE_BF16 && dtype != ALORA_DTYPE_FP32) return ALORA_ERR_UNSUPPORTED;
    if (T > kMaxTokens || rank < 1 || rank > kMaxRank) return ALORA_ERR_CAPACITY;  // beyond the static scratch
    if (T == 0) return ALORA_OK;
    if (R == 0) return ALORA_ERR_INVALID_ARG;
    int dev = -1;
    if (cudaGetDevice(&dev) != cudaSuccess || dev < 0 || dev >= kMaxDevices) return ALORA_ERR_NO_DEVICE;
    if (!g_scratch_addr[dev]) {
        // first call on this device: resolve the array's device address with this device current
        void *p = nullptr;
        if (cudaGetSymbolAddress(&p, g_static_scratch) != cudaSuccess || !p) {
            cudaGetLastError();
            return ALORA_ERR_CUDA;
        }
        g_scratch_addr[dev] = p;
    }
    cudaStream_t s = (cudaStream_t)stream;
    if (dtype == ALORA_DTYPE_FP32)
        launch_all<float>(d_hidden, d_wqkv, d_positions, d_query_start_loc, d_activation_offsets, d_adapter_on, rank,
                          scale, d_Aq, d_Bq, d_Ak, d_Bk, d_Av, d_Bv, T, R, hidden, n_q, n_kv, d_qkv,
                          g_scratch_addr[dev], s);
    else
        launch_all<__nv_bfloat16>(d_hidden, d_wqkv, d_positions, d_query_start_loc, d_activation_offsets,
                                  d_adapter_on, rank, scale, d_Aq, d_Bq, d_Ak, d_Bk, d_Av, d_Bv, T, R, hidden, n_q,
                                  n_kv, d_qkv, g_scratch_addr[dev], s);
    return cudaGetLastError() == cudaSuccess ? ALORA_OK : ALORA_ERR_CUDA;
}

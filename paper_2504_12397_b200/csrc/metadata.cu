// Batch metadata: per-token request / applied-adapter / KV-slot arrays and the projection's
// row-tile list.  Integer work only; every output is compared exactly against the CPU oracle.
#include <algorithm>
#include <climits>
#include "alora_internal.h"
#include "tc_common.cuh"

namespace alora {

constexpr int kProjTileRows = 128;
constexpr int kMetaSmemInts = 7168;   // 28 KB of builder scratch: batches of up to 511 requests
constexpr int kMetaStageR = 1024;     // per-request inputs of up to this many requests are staged in shared memory

// Request owning flat token t: largest r with query_start_loc[r] <= t (binary search; empty
// requests are skipped because their start equals their successor's).
__device__ __forceinline__ int find_request(const int32_t *qsl, int R, int t) {
    int lo = 0, hi = R;  // invariant: qsl[lo] <= t < qsl[hi]
    while (hi - lo > 1) {
        int mid = (lo + hi) >> 1;
        if (qsl[mid] <= t) lo = mid; else hi = mid;
    }
    return lo;
}

// Per token: request index, adapter applied to the row (the gate of Eq. 5: position >= activation
// offset; always open in full-LoRA mode, always closed in base mode), and the token slot
// page * page_size + position % page_size.  Findings (inconsistent positions, page id out of
// range, adapter id out of range, an open gate on an adapter that was never registered on the layer) go
// to the status word; the row then gets adapter -1 / slot -1 so that later kernels skip it.
__device__ __forceinline__ void metadata_tokens(const int32_t *__restrict__ positions,
                                      const int32_t *__restrict__ a_req,
                                      const int32_t *__restrict__ adapter_ids,
                                      const int32_t *__restrict__ qsl, const int32_t *__restrict__ seq_lens,
                                      const int32_t *__restrict__ block_tables, int max_blocks,
                                      int num_pages, int page_size, int max_adapters, int T, int R, int mode,
                                      int32_t *__restrict__ token_req, int32_t *__restrict__ row_adapter,
                                      int32_t *__restrict__ slot_map, const AdapterDev *__restrict__ adapters,
                                      int32_t *status) {
    int t = blockIdx.x * blockDim.x + threadIdx.x;
    if (t >= T) return;
    int r = find_request(qsl, R, t);
    int p = positions[t];
    // positions of a request are consecutive and end at seq_len - 1
    int expect = seq_lens[r] - (qsl[r + 1] - t);
    bool ok = (p == expect) && p >= 0;
    if (!ok) report(status, ALORA_ERR_BAD_BATCH);
    int k = -1;
    if (mode != ALORA_MODE_BASE && adapter_ids != nullptr) {
        k = adapter_ids[r];
        if (k >= max_adapters || k < -1) { report(status, ALORA_ERR_BAD_BATCH); k = -1; }
        if (k >= 0 && mode == ALORA_MODE_ALORA && p < a_req[r]) k = -1;
        // a row whose gate is open needs its adapter's weights on this layer
        if (k >= 0 && adapters != nullptr && adapters[k].rank == 0) { report(status, ALORA_ERR_NO_WEIGHTS); k = -1; }
    }
    if (token_req) token_req[t] = r;
    if (row_adapter) row_adapter[t] = ok ? k : -1;
    if (slot_map) {
        int slot = -1;
        if (ok && block_tables != nullptr) {
            int blk = p / page_size;
            if (blk < max_blocks) {
                int page = block_tables[(size_t)r * max_blocks + blk];
                if (page >= 0 && page < num_pages) slot = page * page_size + p % page_size;
                else report(status, ALORA_ERR_PAGE_RANGE);
            } else {
                report(status, ALORA_ERR_BAD_BATCH);
            }
        }
        slot_map[t] = slot;
    }
}

// Row tiles of the projection.  Each request contributes up to two runs of rows: its gated-off
// rows (applied adapter -1) and its gated-on rows; neighbouring runs with the same applied adapter
// are merged across requests, and every merged run is cut into tiles of at most kProjTileRows rows.
// One block; R is small (a scheduler batch).
__device__ __forceinline__ void metadata_tiles(const int32_t *__restrict__ a_req, const int32_t *__restrict__ adapter_ids,
                                      const int32_t *__restrict__ qsl, const int32_t *__restrict__ seq_lens,
                                      int R, int mode, int max_adapters, int max_tiles,
                                      ProjTile *__restrict__ tiles, int32_t *__restrict__ counts,
                                      int32_t *seg_scratch /* [14R + 5] */, int T, int rowwise_cap, int32_t *__restrict__ shrink_tiles,
                                      int32_t *__restrict__ t_ready, int32_t *status) {
    int32_t *seg_start = seg_scratch, *seg_len = seg_scratch + (2 * R + 1);
    int32_t *seg_adapter = seg_scratch + 2 * (2 * R + 1), *seg_tile0 = seg_scratch + 3 * (2 * R + 1);
    int32_t *seg_shrink0 = seg_scratch + 4 * (2 * R + 1);  // adapter tiles before the segment
    int32_t *rq_start = seg_scratch + 5 * (2 * R + 1), *rq_new = rq_start + R, *rq_off = rq_new + R, *rq_k = rq_off + R;
    __shared__ int n_seg, n_tiles;
    // per request, in parallel: first row, new rows, gated-off rows, adapter
    for (int r = threadIdx.x; r < R; r += blockDim.x) {
        const int n_new = qsl[r + 1] - qsl[r];
        int k = (mode == ALORA_MODE_BASE || adapter_ids == nullptr) ? -1 : adapter_ids[r];
        if (k >= max_adapters || k < -1) k = -1;
        int n_off = 0;
        if (k < 0) n_off = max(n_new, 0);
        else if (mode == ALORA_MODE_ALORA) {
            const int p_first = seq_lens[r] - n_new;
            const long long d = (long long)a_req[r] - p_first;
            n_off = d <= 0 ? 0 : (d >= n_new ? n_new : (int)d);
        }
        rq_start[r] = qsl[r]; rq_new[r] = n_new; rq_off[r] = n_off; rq_k[r] = k;
    }
    __syncthreads();
    if (threadIdx.x == 0) {
        int ns = 0, nt = 0;
        int cur_start = 0, cur_len = 0, cur_ad = -1;   // the run being grown, kept in registers
        bool have = false;
#pragma unroll 4
        for (int r = 0; r < R; ++r) {
            const int n_new = rq_new[r];
            if (n_new <= 0) continue;
            const int n_off = rq_off[r];
            const int start[2] = {rq_start[r], rq_start[r] + n_off};
            const int len[2] = {n_off, n_new - n_off};
            const int ad[2] = {-1, rq_k[r]};
#pragma unroll
            for (int i = 0; i < 2; ++i) {
                if (len[i] <= 0) continue;
                if (have && cur_ad == ad[i] && cur_start + cur_len == start[i]) {
                    cur_len += len[i];
                } else {
                    if (have) { seg_start[ns] = cur_start; seg_len[ns] = cur_len; seg_adapter[ns] = cur_ad; ++ns; }
                    cur_start = start[i]; cur_len = len[i]; cur_ad = ad[i];
                    have = true;
                }
            }
        }
        if (have) { seg_start[ns] = cur_start; seg_len[ns] = cur_len; seg_adapter[ns] = cur_ad; ++ns; }
        int n_ad = 0;
        for (int s = 0; s < ns; ++s) {
            seg_tile0[s] = nt;
            seg_shrink0[s] = n_ad;
            const int n = (seg_len[s] + kProjTileRows - 1) / kProjTileRows;
            nt += n;
            if (seg_adapter[s] >= 0) n_ad += n;
        }
        seg_tile0[ns] = nt;
        if (nt > max_tiles) { report(status, ALORA_ERR_CAPACITY); nt = 0; ns = 0; n_ad = 0; }
        n_seg = ns; n_tiles = nt;
        counts[0] = nt;
        counts[2] = n_ad;
        // Row tiles that hold only a few rows each (decode steps, short suffixes of many requests with different
        // adapters) waste the tensor cores: when the tiles cover more than twice the batch's rows, and always when
        // the batch has at most kRowwiseAlwaysRows rows, the projection takes the row-wise route (dense row tiles + a
        // per-row delta) instead.  (The per-row delta costs about 0.4 us per row, the tensor-core shrink of a few
        // tiles about 8 us whatever their rows.)
        const bool wasteful = (long long)nt * kProjTileRows > 2ll * T + 2 * kProjTileRows;
        counts[5] = (n_ad > 0 && T <= rowwise_cap && (T <= kRowwiseAlwaysRows || wasteful)) ? 1 : 0;
    }
    __syncthreads();
    for (int i = threadIdx.x; i < n_tiles; i += blockDim.x) {
        int lo = 0, hi = n_seg;  // seg_tile0[lo] <= i < seg_tile0[hi]
        while (hi - lo > 1) {
            int mid = (lo + hi) >> 1;
            if (seg_tile0[mid] <= i) lo = mid; else hi = mid;
        }
        int off = (i - seg_tile0[lo]) * kProjTileRows;
        ProjTile pt;
        pt.row_start = seg_start[lo] + off;
        pt.row_count = min(kProjTileRows, seg_len[lo] - off);
        pt.adapter = seg_adapter[lo];
        pt.pad_ = 0;
        tiles[i] = pt;
        // list of the tiles that need t = s A x, and their "t is ready" counters, cleared for this batch
        if (pt.adapter >= 0) shrink_tiles[seg_shrink0[lo] + (i - seg_tile0[lo])] = i;
        t_ready[i] = 0;
    }
}

// Which requests the few-row kernel takes (1 .. returned limit new tokens; the others go to the tensor-core
// kernel).  Normally the limit is small_max.  When the requests with 2 .. small_max new tokens alone make at least
// two KV streams per SM, they fill the tensor-core kernel's blocks, which then reads the cache faster than the
// few-row kernel (64 requests x 4 tokens on 4096 cached ones: 0.82 against 0.67 of the HBM bandwidth), and the limit
// is 1.  Called by all threads of a block; both list builders take the same decision.
__device__ __forceinline__ int few_row_limit(const int32_t *__restrict__ qsl, int R, int Hkv, int n_sm, int small_max) {
    __shared__ int n_multi;
    if (threadIdx.x == 0) n_multi = 0;
    __syncthreads();
    int mine = 0;
    for (int r = threadIdx.x; r < R; r += blockDim.x) {
        const int n_new = qsl[r + 1] - qsl[r];
        mine += n_new >= 2 && n_new <= small_max;
    }
    if (mine) atomicAdd(&n_multi, mine);
    __syncthreads();
    const int n = n_multi;
    __syncthreads();   // (the counter may be reused by a second call in this block)
    return (long long)n * Hkv >= 2ll * n_sm ? min(1, small_max) : small_max;
}

// Attention work items of a prefill batch: each request's new tokens are cut into blocks of
// `q_block` tokens; one item per (request, KV head, block), blocks of the same KV stream adjacent so
// that blocks running at the same time share their K/V pages in L2.  Keys 0 .. position of the
// block's last token are visible to the block (causal limit); per-row limits are applied in the kernel.
__device__ __forceinline__ void metadata_attn_items(const int32_t *__restrict__ qsl, const int32_t *__restrict__ seq_lens,
                                           int R, int Hkv, int q_block, int small_max, int max_items,
                                           AttnWork *__restrict__ items, int32_t *__restrict__ counts,
                                           int32_t *blk_off /* [R+1] */, int n_blocks, int32_t *__restrict__ cta_start,
                                           int32_t *status) {
    __shared__ int total;
    small_max = few_row_limit(qsl, R, Hkv, n_blocks, small_max);
    for (int r = threadIdx.x; r < R; r += blockDim.x) {
        const int n_new = qsl[r + 1] - qsl[r];
        blk_off[r] = n_new > small_max ? (n_new + q_block - 1) / q_block : 0;  // short requests: few-row list
    }
    __syncthreads();
    if (threadIdx.x == 0) {
        int acc = 0;
        for (int r = 0; r < R; ++r) {
            const int n = blk_off[r];
            blk_off[r] = acc;
            acc += n;
        }
        blk_off[R] = acc;
        int n = acc * Hkv;
        if (n > max_items) { report(status, ALORA_ERR_CAPACITY); n = 0; }
        total = n;
        counts[1] = n;
    }
    __syncthreads();
    int sum = 0, tmin = INT_MAX, tmax = 0;   // key tiles of this thread's items
    for (int i = threadIdx.x; i < total; i += blockDim.x) {
        int lo = 0, hi = R;      // blk_off[lo] * Hkv <= i < blk_off[hi] * Hkv
        while (hi - lo > 1) {
            const int mid = (lo + hi) >> 1;
            if (blk_off[mid] * Hkv <= i) lo = mid; else hi = mid;
        }
        const int r = lo;
        const int nblk = blk_off[r + 1] - blk_off[r];
        const int rem = i - blk_off[r] * Hkv;
        const int kvh = rem / nblk, blk = rem % nblk;
        const int n_new = qsl[r + 1] - qsl[r];
        AttnWork w;
        w.req = r;
        w.q_start = qsl[r] + blk * q_block;
        w.q_count = min(q_block, n_new - blk * q_block);
        w.kv_head = kvh;
        w.kv_start = 0;
        w.kv_end = seq_lens[r] - n_new + blk * q_block + w.q_count;  // last token's position + 1
        w.split = 0;
        w.n_splits = 1;
        items[i] = w;
        const int n = (w.kv_end + kAttnKeysPerTile - 1) / kAttnKeysPerTile;
        sum += n; tmin = min(tmin, n); tmax = max(tmax, n);
    }
    // Work split of the attention kernel over its n_blocks blocks (the launch uses that many whenever a cut is
    // possible).  Normally every item is taken whole, round-robin.
    // Long batches (at least kAttnCutMinTiles key tiles per block) of items of nearly equal length that make at
    // least kAttnCutMinWaves full rounds: the first n_whole = n_blocks * floor(items / n_blocks) items are taken
    // whole, round-robin; the key tiles of the remaining items are concatenated and cut into runs of equal length,
    // one per block, so an item can be cut into parts that different blocks work on (a merge kernel adds the
    // parts up).
    //   items[i].split = tiles before item i;  counts[6] = tiles in the concatenation, counts[7] = run length,
    //   counts[8] = n_whole, counts[9] = tiles before item n_whole;
    //   cta_start[c] = the item that holds the first tile of block c's run.
    __shared__ int warp_sum[32], warp_min[32], warp_max[32];
    __shared__ int run_len, run_off, run_first;
    const int lane = threadIdx.x & 31, wid = threadIdx.x >> 5;
    for (int o = 1; o < 32; o <<= 1) {
        sum += __shfl_xor_sync(0xffffffffu, sum, o);
        tmin = min(tmin, __shfl_xor_sync(0xffffffffu, tmin, o));
        tmax = max(tmax, __shfl_xor_sync(0xffffffffu, tmax, o));
    }
    if (lane == 0) { warp_sum[wid] = sum; warp_min[wid] = tmin; warp_max[wid] = tmax; }
    __syncthreads();   // (also: this block's writes to items[] are visible to all of its threads)
    if (threadIdx.x == 0) {
        int acc = 0, mn = INT_MAX, mx = 0;
        for (int w = 0; w < (int)(blockDim.x + 31) / 32; ++w) {
            acc += warp_sum[w];
            mn = min(mn, warp_min[w]); mx = max(mx, warp_max[w]);
        }
        // cutting pays when most of the work is still done on whole items (whose sibling query blocks share their
        // K/V tiles in L2): items of nearly equal length, at least kAttnCutMinWaves full rounds of whole items
        const bool uniform = mx - mn <= max(1, mx / 16);
        const bool long_batch = acc >= kAttnCutMinTiles * n_blocks && uniform && total >= kAttnCutMinWaves * n_blocks &&
                                total % n_blocks != 0;
        // ... and a batch with fewer items than blocks (a few requests with long contexts) is spread over all blocks
        // when that still leaves every block a run of at least kAttnMinRunTiles key tiles and shortens the longest
        // block's work by more than the merge costs (about the time of kAttnSpreadMinGain key tiles, measured)
        const bool few_items = total > 0 && total < n_blocks && acc >= kAttnMinRunTiles * n_blocks &&
                               mx >= acc / n_blocks + kAttnSpreadMinGain;
        const bool cut = long_batch || few_items;
        run_first = !cut ? -1 : n_blocks * (total / n_blocks);
        run_len = acc;   // all tiles, for now
        if (!cut) { counts[6] = 0; counts[7] = kAttnMinRunTiles; counts[8] = total; counts[9] = acc; }
    }
    __syncthreads();
    if (run_first < 0) return;   // short batch: every item whole, nothing more to prepare
    // tiles before each item: contiguous chunks of items per thread, scanned over the block
    const int chunk = (total + (int)blockDim.x - 1) / (int)blockDim.x;
    const int lo = min(total, (int)threadIdx.x * chunk), hi = min(total, lo + chunk);
    sum = 0;
    for (int i = lo; i < hi; ++i) sum += (items[i].kv_end + kAttnKeysPerTile - 1) / kAttnKeysPerTile;
    int incl = sum;
    for (int o = 1; o < 32; o <<= 1) {
        const int v = __shfl_up_sync(0xffffffffu, incl, o);
        if (lane >= o) incl += v;
    }
    __syncthreads();   // warp_sum is reused
    if (lane == 31) warp_sum[wid] = incl;
    __syncthreads();
    int acc = incl - sum;
    for (int w = 0; w < wid; ++w) acc += warp_sum[w];
    for (int i = lo; i < hi; ++i) {
        items[i].split = acc;
        acc += (items[i].kv_end + kAttnKeysPerTile - 1) / kAttnKeysPerTile;
    }
    __syncthreads();
    if (threadIdx.x == 0) {
        const int all = run_len, first = run_first;
        const int off = first < total ? items[first].split : all;
        const int len = max((all - off + n_blocks - 1) / n_blocks, kAttnMinRunTiles);
        counts[6] = all - off;
        counts[7] = len;
        counts[8] = first;
        counts[9] = off;
        run_len = len;
        run_off = off;
    }
    __syncthreads();
    const int len = run_len, off = run_off;
    for (int i = max(lo, run_first); i < hi; ++i) {
        const int rel = items[i].split - off;
        const int n = (items[i].kv_end + kAttnKeysPerTile - 1) / kAttnKeysPerTile;
        for (int c = (rel + len - 1) / len; c * len < rel + n && c < n_blocks; ++c) cta_start[c] = i;
    }
}

// Work list of the few-row attention kernel: requests with 1 .. small_max new tokens.  Their score rows
// (token, query head of the group) are cut into blocks of 16 * mt rows (mt = 1, 2 or 4 tiles, the
// smallest that holds all rows, else 4), and the keys 0 .. causal limit of each block into ranges of
// at most `chunk` 64-key units (see the choice of `chunk` below; at most kSplitItemsPerSm ranges per SM).
// The ranges of one (block, KV head) are consecutive items.
__device__ __forceinline__ void small_block_shape(int n_new, int G, int &mt, int &tok_per_blk, int &nblk) {
    const int rows = n_new * G;
    mt = rows <= 16 ? 1 : (rows <= 32 ? 2 : 4);
    tok_per_blk = 16 * mt / G;
    nblk = (n_new + tok_per_blk - 1) / tok_per_blk;
}

// Requests that read one shared prefix cache (several adapters invoked on the same conversation: their block tables
// start with the same physical pages).  Neighbouring requests of the few-row route are put into one PREFIX GROUP when
// they have leading pages in common, so that the attention reads those pages once for all of them:
//   common(r)  = the number of leading block-table entries that requests r-1 and r have in common, counted only over
//                pages that lie wholly before both requests' first new position;
//   a group starts at an eligible request f (1 .. small_max new tokens) and is extended by f+1, f+2, ... while the
//   next request is eligible, common(next) * page_size >= kMinSharedKeys, and the stacked score rows (new tokens of
//   all members x G) still fit into 64;  a group needs at least two members;
//   its shared length is the smallest common() of its pairs, in keys, rounded down to a multiple of 64.
// Output per request: grp_first (index of the group's first request; r itself when ungrouped) and grp_shared (the
// shared keys, 0 when ungrouped).  Called by all threads of a block.
constexpr int kMinSharedKeys = 256;
__device__ __forceinline__ void metadata_prefix_groups(const int32_t *__restrict__ qsl, const int32_t *__restrict__ seq_lens,
                                                       const int32_t *__restrict__ block_tables, int max_blocks, int R,
                                                       int page_size, int G, int small_max,
                                                       int32_t *__restrict__ grp_first, int32_t *__restrict__ grp_shared) {
    // common(r) for all pairs.  First the pairs that can share at all (both on this route, same first page): most
    // pairs of unrelated requests end here.  Then, pair after pair, all threads compare the table entries below the
    // pair's limit at once and keep the smallest mismatching index; no thread waits for another pair's loads.
    for (int r = threadIdx.x; r < R; r += blockDim.x) {
        int lim = 0;
        if (r > 0) {
            const int na = qsl[r] - qsl[r - 1], nb = qsl[r + 1] - qsl[r];
            if (na > 0 && nb > 0 && na <= small_max && nb <= small_max) {
                lim = min(min((seq_lens[r - 1] - na) / page_size, (seq_lens[r] - nb) / page_size), max_blocks);
                if (lim > 0 && block_tables[(size_t)(r - 1) * max_blocks] != block_tables[(size_t)r * max_blocks]) lim = 0;
            }
        }
        grp_first[r] = max(lim, 0);    // for now: the pair's limit (0: nothing in common)
        grp_shared[r] = max(lim, 0);   // for now: the first mismatching entry found so far (none yet)
    }
    __syncthreads();
    for (int r = 1; r < R; ++r) {
        const int lim = grp_first[r];
        if (lim <= 1) continue;
        const int32_t *ta = block_tables + (size_t)(r - 1) * max_blocks, *tb = block_tables + (size_t)r * max_blocks;
        for (int b = 1 + (int)threadIdx.x; b < lim; b += blockDim.x)
            if (ta[b] != tb[b]) atomicMin(&grp_shared[r], b);
    }
    __syncthreads();
    // keys in common with the left neighbour; most batches have no pair that shares enough: then nobody is grouped and
    // the serial pass below (one thread walking the requests) is not needed
    bool any = false;
    for (int r = threadIdx.x; r < R; r += blockDim.x) {
        const int keys = grp_shared[r] * page_size;
        grp_shared[r] = keys;
        any |= keys >= kMinSharedKeys;
    }
    if (!__syncthreads_or(any)) {
        for (int r = threadIdx.x; r < R; r += blockDim.x) { grp_first[r] = r; grp_shared[r] = 0; }
        __syncthreads();
        return;
    }
    if (threadIdx.x == 0) {
        int f = 0;
        while (f < R) {
            const int nf = qsl[f + 1] - qsl[f];
            int e = f + 1;
            int shared = 0;
            if (nf > 0 && nf <= small_max) {
                int rows = nf * G, mn = 0x7fffffff;
                while (e < R) {
                    const int ne = qsl[e + 1] - qsl[e];
                    const int c = grp_shared[e];
                    if (!(ne > 0 && ne <= small_max) || c < kMinSharedKeys || rows + ne * G > 64) break;
                    rows += ne * G;
                    mn = min(mn, c);
                    ++e;
                }
                if (e - f >= 2) shared = mn & ~63;
            }
            if (shared <= 0) { e = f + 1; shared = 0; }
            for (int m = f; m < e; ++m) { grp_first[m] = f; }
            // grp_shared[f + 1 .. e) still hold the pair values that the loop above read; overwrite after use
            for (int m = f; m < e; ++m) grp_shared[m] = shared;
            f = e;
        }
    }
    __syncthreads();
}

// Work list of the few-row attention kernel.  A STREAM is one block of score rows with the keys it reads: for an
// ungrouped request its blocks of up to 16 * mt rows over keys 0 .. causal limit; for a prefix group the stacked rows
// of all members, over the shared prefix (read once, nothing masked) followed by every member's own keys beyond it
// (masked so that only that member's rows see them).  A stream's keys are cut into ranges of at most `chunk` 64-key
// units; the ranges of one (stream, KV head) are consecutive items and are merged by whichever block finishes last.
// A group is owned by its first request: that request accounts for all of the group's items.
struct GroupShape {
    int n_members, n_tok, shared, mt;
};
__device__ __forceinline__ GroupShape group_shape(const int32_t *qsl, const int32_t *grp_first, const int32_t *grp_shared,
                                                  int R, int f, int G) {
    GroupShape g;
    g.shared = grp_shared[f];
    int e = f + 1;
    while (e < R && grp_first[e] == f) ++e;
    g.n_members = e - f;
    g.n_tok = qsl[e] - qsl[f];
    const int rows = g.n_tok * G;
    g.mt = rows <= 16 ? 1 : (rows <= 32 ? 2 : 4);
    return g;
}
// ranges of request r's share of the list for a given range length; also the 64-key units (weighted by row tiles)
__device__ __forceinline__ void request_ranges(const int32_t *qsl, const int32_t *seq_lens, const int32_t *grp_first,
                                               const int32_t *grp_shared, int R, int r, int G, int small_max, int chunk,
                                               int &n_ranges, int &weighted_units, int &mt_out) {
    n_ranges = 0; weighted_units = 0; mt_out = 1;
    const int n_new = qsl[r + 1] - qsl[r];
    if (n_new <= 0 || n_new > small_max) return;
    if (grp_first[r] != r) return;                       // a member of a group: accounted for by the group's owner
    if (grp_shared[r] > 0) {
        const GroupShape g = group_shape(qsl, grp_first, grp_shared, R, r, G);
        const int pu = g.shared / 64;
        int tu = 0;   // the members' own keys beyond the shared ones, member after member, in 64-key stages
        for (int m = r; m < r + g.n_members; ++m) tu += (seq_lens[m] - g.shared + 63) / 64;
        n_ranges = (pu + chunk - 1) / chunk + (tu + chunk - 1) / chunk;
        weighted_units = (pu + tu) * g.mt;
        mt_out = g.mt;
        return;
    }
    int mt, tpb, nblk;
    small_block_shape(n_new, G, mt, tpb, nblk);
    for (int blk = 0; blk < nblk; ++blk) {
        const int kv_end = seq_lens[r] - n_new + min(n_new, (blk + 1) * tpb);
        const int u = (kv_end + 63) / 64;
        weighted_units += u * mt;
        n_ranges += (u + chunk - 1) / chunk;
    }
    mt_out = mt;
}

__device__ __forceinline__ void metadata_split_items(const int32_t *__restrict__ qsl, const int32_t *__restrict__ seq_lens,
                                                     const int32_t *__restrict__ block_tables, int max_blocks, int page_size,
                                                     int R, int Hkv, int G, int n_sm, int small_max, int max_items, int max_rows,
                                                     AttnSplitWork *__restrict__ items, int32_t *__restrict__ counts,
                                                     int32_t *req_scratch /* [5][R] */,
                                                     int32_t *__restrict__ group_done, int32_t *__restrict__ groups_out,
                                                     int part, int n_parts, int32_t *status) {
    // (several blocks may build the list together: each repeats the cheap per-request passes and fills the items
    // part, part + n_parts, ..; block `part` 0 alone writes the counts and reports findings)
    __shared__ unsigned long long tot_units;
    __shared__ int chunk_units, total_items, few_ranges;
    small_max = few_row_limit(qsl, R, Hkv, n_sm, small_max);
    int32_t *req_cnt = req_scratch, *req_off = req_scratch + R, *req_row = req_scratch + 2 * R;
    int32_t *grp_first = req_scratch + 3 * R, *grp_shared = req_scratch + 4 * R;
    metadata_prefix_groups(qsl, seq_lens, block_tables, max_blocks, R, page_size, G, small_max, grp_first, grp_shared);
    if (groups_out != nullptr && part == 0)
        for (int r = threadIdx.x; r < R; r += blockDim.x) { groups_out[r] = grp_first[r]; groups_out[R + r] = grp_shared[r]; }
    // 64-key units of all streams, weighted by their row tiles (an item of mt tiles needs mt * 16 partial rows):
    // per request in parallel, summed by one thread (a shared 64-bit atomic under contention is far slower)
    for (int r = threadIdx.x; r < R; r += blockDim.x) {
        int n, wu, mt;
        request_ranges(qsl, seq_lens, grp_first, grp_shared, R, r, G, small_max, 1 << 20, n, wu, mt);
        req_cnt[r] = wu * Hkv;
    }
    __syncthreads();
    if (threadIdx.x == 0) {
        unsigned long long sum = 0ull;
        for (int r = 0; r < R; ++r) sum += (unsigned long long)req_cnt[r];
        tot_units = sum;
    }
    __syncthreads();
    if (threadIdx.x == 0) {
        // Range length: a range costs a fixed time beyond its streaming time (item claim, first table window and
        // first copies, query fetch, combining the warps, publishing the partial result, a share of the merge), and
        // the last ranges of a launch leave SMs idle for up to one range.  With t = streaming time of all units on
        // one SM (0.74 us per 64-key unit at an SM's share of the HBM bandwidth) the sum of both losses is smallest
        // near sqrt(t / c) ranges per SM, capped by the capacity of the work list; c = 12 us is what batches of 2
        // to 64 requests with 4096 to 32768 cached tokens run fastest with (3 us: 5 .. 16 % slower on the small ones).
        const float t_us = (float)tot_units * 0.74f / (float)max(n_sm, 1);
        const float per_sm = fminf(fmaxf(sqrtf(t_us / 12.f), 1.f), (float)kSplitItemsPerSm);
        const unsigned long long target = (unsigned long long)ceilf(per_sm * (float)max(n_sm, 1));
        chunk_units = (int)max(4ull, (tot_units + target - 1) / target);
        few_ranges = (tot_units > 0 && per_sm < 2.5f) ? 1 : 0;
    }
    __syncthreads();
    // With only one or two ranges per SM the rule above ignores how the ranges fall into rounds over the SMs: 192
    // equal ranges on 148 SMs take as long as 296.  Such batches (a few requests) instead take the shortest range
    // length whose ranges fit into exactly one round, or into two, whichever the same cost model says is faster:
    // rounds x (12 us + range length x 0.74 us).  The range count for a given length is a sum over the requests.
    if (few_ranges) {
        // every thread tries one candidate length (a grid over 4 .. the longest stream) and counts the ranges of the
        // whole batch for it; the shortest candidates that fit one round and two rounds are kept
        __shared__ int max_units, best1, best2;
        if (threadIdx.x == 0) { max_units = 4; best1 = 0x7fffffff; best2 = 0x7fffffff; }
        __syncthreads();
        int mu = 0;
        for (int r = threadIdx.x; r < R; r += blockDim.x) mu = max(mu, (seq_lens[r] + 63) / 64);
        if (mu > 4) atomicMax(&max_units, mu);
        __syncthreads();
        const int step = (max_units - 4 + (int)blockDim.x - 1) / (int)blockDim.x + 0, cand = 4 + (int)threadIdx.x * max(step, 1);
        if (cand <= max_units + max(step, 1)) {
            int cnt = 0;
            for (int r = 0; r < R; ++r) {
                int n, wu, mt;
                request_ranges(qsl, seq_lens, grp_first, grp_shared, R, r, G, small_max, cand, n, wu, mt);
                cnt += n * Hkv;
            }
            if (cnt <= n_sm) atomicMin(&best1, cand);
            if (cnt <= 2 * n_sm) atomicMin(&best2, cand);
        }
        __syncthreads();
        if (threadIdx.x == 0) {
            const float c1 = 12.f + 0.74f * (float)best1, c2 = 2.f * (12.f + 0.74f * (float)best2);
            if (best1 != 0x7fffffff && c1 <= c2) chunk_units = best1;
            else if (best2 != 0x7fffffff) chunk_units = best2;
        }
        __syncthreads();
    }
    const int chunk = chunk_units;
    for (int r = threadIdx.x; r < R; r += blockDim.x) {
        int n, wu, mt;
        request_ranges(qsl, seq_lens, grp_first, grp_shared, R, r, G, small_max, chunk, n, wu, mt);
        req_cnt[r] = n * Hkv;
        req_row[r] = n * Hkv * 16 * mt;
    }
    __syncthreads();
    if (threadIdx.x == 0) {
        int acc = 0, rows = 0;
        for (int r = 0; r < R; ++r) {
            const int c = req_cnt[r], n = req_row[r];
            req_off[r] = acc; req_row[r] = rows;
            acc += c; rows += n;
        }
        if (acc > max_items || rows > max_rows) {
            if (part == 0) report(status, ALORA_ERR_CAPACITY);
            acc = 0;
        }
        total_items = acc;
        if (part == 0) {
            counts[3] = acc;
            counts[4] = 0;   // work counter of the few-row kernel
        }
    }
    __syncthreads();
    if (total_items == 0) return;
    // one item per thread and step: owner request by binary search over the item offsets, then stream / KV head / range
    for (int i = part * (int)blockDim.x + (int)threadIdx.x; i < total_items; i += n_parts * (int)blockDim.x) {
        int lo = 0, hi = R;   // largest r with req_off[r] <= i among requests that own items
        while (hi - lo > 1) {
            const int mid = (lo + hi) >> 1;
            if (req_off[mid] <= i) lo = mid; else hi = mid;
        }
        const int r = lo;
        int local = i - req_off[r], row0 = req_row[r];
        AttnSplitWork w;
        if (grp_shared[r] > 0) {
            // ---- a prefix group: per KV head [ranges of the shared prefix | ranges of the members' own keys]; the own
            // keys of all members form one sequence of 64-key stages (member after member) that is cut like any other
            const GroupShape g = group_shape(qsl, grp_first, grp_shared, R, r, G);
            const int pu = g.shared / 64, np = (pu + chunk - 1) / chunk;
            int tu = 0;
            for (int m = r; m < r + g.n_members; ++m) tu += (seq_lens[m] - g.shared + 63) / 64;
            const int nt = (tu + chunk - 1) / chunk;
            const int n_splits = np + nt;
            const int kvh = local / n_splits, sp = local % n_splits;
            w.q_start = qsl[r]; w.q_count = g.n_tok; w.kv_head = kvh; w.mt = g.mt; w.split = sp; w.n_splits = n_splits;
            w.part_row0 = row0 + local * 16 * g.mt;
            if (sp < np) {
                const int per = (pu + np - 1) / np;
                w.req = r; w.kv_start = sp * per * 64; w.kv_end = min(g.shared, (sp + 1) * per * 64);
                w.pos0 = g.shared;    // every row sees every key of the shared prefix
                w.pad_ = 0;
            } else {
                // stages [kv_start / 64, kv_end / 64) of the members' own keys (not key positions: the kernel walks the
                // members to find each stage's request, key positions and rows)
                const int sp2 = sp - np, per = (tu + nt - 1) / nt;
                w.req = r; w.kv_start = sp2 * per * 64; w.kv_end = min(tu, (sp2 + 1) * per) * 64;
                w.pos0 = g.shared;
                w.pad_ = kSplitOwnKeys | g.n_members;
            }
            group_done[i] = 0;
            items[i] = w;
            continue;
        }
        const int n_new = qsl[r + 1] - qsl[r];
        int mt, tpb, nblk;
        small_block_shape(n_new, G, mt, tpb, nblk);
        for (int blk = 0; blk < nblk; ++blk) {
            const int q_count = min(tpb, n_new - blk * tpb);
            const int pos0 = seq_lens[r] - n_new + blk * tpb;
            const int kv_end = pos0 + q_count;   // last token's position + 1
            const int units = (kv_end + 63) / 64;
            const int n_splits = (units + chunk - 1) / chunk;
            if (local >= n_splits * Hkv && blk + 1 < nblk) {
                local -= n_splits * Hkv;
                row0 += n_splits * Hkv * 16 * mt;
                continue;
            }
            const int per = (units + n_splits - 1) / n_splits;   // equal ranges rather than full ones and a stub
            const int kvh = local / n_splits, sp = local % n_splits;
            w.req = r; w.q_start = qsl[r] + blk * tpb; w.q_count = q_count; w.kv_head = kvh;
            w.kv_start = sp * per * 64; w.kv_end = min(kv_end, (sp + 1) * per * 64);
            w.pos0 = pos0; w.mt = mt; w.split = sp; w.n_splits = n_splits; w.part_row0 = row0 + local * 16 * mt; w.pad_ = 0;
            group_done[i] = 0;
            items[i] = w;
            break;
        }
    }
}

// FewRowMeta of a batch of at most kFewRowMax rows (all of them in block 0): the adapters that occur in
// row_adapter[0 .. T), ascending, each one's padded rank and scale, and every row's slot.  Called by all
// threads of block 0 after they have written row_adapter.
__device__ __forceinline__ void metadata_few_row(const int32_t *row_adapter, const AdapterDev *__restrict__ adapters,
                                                 int T, int max_adapters, FewRowMeta *__restrict__ meta) {
    __shared__ uint32_t bits[32];
    __shared__ int16_t ids[kFewRowMax];
    __shared__ int n_present;
    if (threadIdx.x < 32) bits[threadIdx.x] = 0u;
    __syncthreads();   // (also orders this block's row_adapter writes before the reads below)
    int k_mine = -1;
    if ((int)threadIdx.x < T && (int)threadIdx.x < kFewRowMax) {
        k_mine = row_adapter[threadIdx.x];
        if (k_mine >= 0 && k_mine < max_adapters && k_mine < 1024) atomicOr(&bits[k_mine >> 5], 1u << (k_mine & 31));
        else k_mine = -1;
    }
    __syncthreads();
    if (threadIdx.x == 0) {
        int n = 0;
        for (int w = 0; w < 32; ++w) {
            uint32_t b = bits[w];
            while (b && n < kFewRowMax) {
                const int i = __ffs(b) - 1;
                b &= b - 1;
                ids[n++] = (int16_t)(w * 32 + i);
            }
        }
        n_present = n;
        meta->n_present = n;
    }
    __syncthreads();
    const int n = n_present;
    if ((int)threadIdx.x < n) {
        const AdapterDev ad = adapters[ids[threadIdx.x]];
        meta->id[threadIdx.x] = ids[threadIdx.x]; meta->rpad[threadIdx.x] = ad.rpad; meta->scale[threadIdx.x] = ad.scale;
    }
    if ((int)threadIdx.x < kFewRowMax) {
        int slot = -1;
        if (k_mine >= 0)
            for (int p = 0; p < n; ++p) if (ids[p] == k_mine) slot = p;
        meta->slot_of_row[threadIdx.x] = slot;
    }
}

// The metadata step.  Phase bit 0: every block handles 256 tokens (request, applied adapter, slot); block 0 then
// builds the projection's row-tile list, or the few-row route's adapter facts.  Phase bit 1: the two attention
// work lists, one block each (their serial parts are O(R)).  Both phases in one launch: blocks 0, 1, 2 take one
// builder each.  The attention phase alone is launched as a programmatic dependent of the projection kernel, beside
// which it runs (it reads nothing that kernel writes); its blocks wait for that kernel before they exit, so that
// whatever follows in the stream still sees the projection complete.
__global__ void __launch_bounds__(256)
metadata_kernel(const int32_t *__restrict__ positions, const int32_t *a_req, const int32_t *adapter_ids,
                const int32_t *qsl, const int32_t *seq_lens, const int32_t *__restrict__ block_tables, int max_blocks,
                int num_pages, int page_size, int max_adapters, int T, int R, int mode,
                int32_t *__restrict__ token_req, int32_t *__restrict__ row_adapter, int32_t *__restrict__ slot_map,
                int max_tiles, ProjTile *__restrict__ tiles, int32_t *__restrict__ counts, int32_t *seg_scratch,
                int32_t *__restrict__ shrink_tiles, int32_t *__restrict__ t_ready,
                int Hkv, int q_block, int max_items, AttnWork *__restrict__ items, int32_t *blk_off,
                int G, int n_sm, int small_max, int max_split_items, int max_split_rows,
                AttnSplitWork *__restrict__ split_items,
                int32_t *req_scratch, int32_t *__restrict__ group_done, int rowwise_cap,
                int32_t *__restrict__ attn_cta_start, const AdapterDev *__restrict__ adapters, int phases,
                FewRowMeta *__restrict__ few_row_meta, int32_t *__restrict__ prefix_groups, int32_t *status) {
    // The per-request inputs are read many times (binary searches, list builders): one parallel pass stages them
    // in shared memory, so that the later steps do not each pay a round trip to global memory.
    __shared__ int32_t s_req[4 * kMetaStageR + 1];
    tc::grid_dep_launch();   // the next kernel's blocks may start their set-up; they wait for this kernel's results
    if (R <= kMetaStageR) {
        int32_t *s_qsl = s_req, *s_len = s_req + R + 1, *s_ids = s_len + R, *s_areq = s_ids + R;
        for (int i = threadIdx.x; i <= R; i += blockDim.x) s_qsl[i] = qsl[i];
        for (int i = threadIdx.x; i < R; i += blockDim.x) {
            s_len[i] = seq_lens[i];
            if (adapter_ids) s_ids[i] = adapter_ids[i];
            if (a_req) s_areq[i] = a_req[i];
        }
        __syncthreads();
        qsl = s_qsl; seq_lens = s_len;
        if (adapter_ids) adapter_ids = s_ids;
        if (a_req) a_req = s_areq;
    }
    if (phases & kMetaProjection)
        metadata_tokens(positions, a_req, adapter_ids, qsl, seq_lens, block_tables, max_blocks, num_pages, page_size,
                        max_adapters, T, R, mode, token_req, row_adapter, slot_map, adapters, status);
    // The three list builders are independent of one another: blocks 0, 1 and 2 take one each (a launch of both
    // phases has at least three blocks, one of the attention phase alone two).
    const int nb = (int)gridDim.x;
    const bool proj = (phases & kMetaProjection) != 0, attn = (phases & kMetaAttention) != 0;
    const int b_tiles = proj ? 0 : -1;
    const int b_attn = !attn ? -1 : (proj ? (nb > 1 ? 1 : 0) : 0);
    const int b_split = !attn ? -1 : (proj ? (nb > 2 ? 2 : 0) : (nb > 1 ? 1 : 0));
    // the attention phase alone: block 0 builds the tensor-core kernel's list, all the others share the few-row list
    const int split_parts = (!proj && attn && nb > 1) ? nb - 1 : 1;
    const bool split_helper = !proj && attn && (int)blockIdx.x > b_split;
    if ((int)blockIdx.x != b_tiles && (int)blockIdx.x != b_attn && (int)blockIdx.x != b_split && !split_helper) {
        if (!proj) tc::grid_dep_wait();
        return;
    }
    // the per-request scratch of the list builders (their serial parts walk it) lives in shared memory when the
    // batch is small enough, else in the context's global scratch (one buffer per builder)
    __shared__ int32_t smem_scratch[kMetaSmemInts];
    if (14 * R + 5 <= kMetaSmemInts) seg_scratch = blk_off = req_scratch = smem_scratch;
    __syncthreads();
    if ((int)blockIdx.x == b_tiles) {
        if (few_row_meta != nullptr && adapters != nullptr && row_adapter != nullptr)
            metadata_few_row(row_adapter, adapters, T, max_adapters, few_row_meta);   // the few-row route has no row tiles
        else
            metadata_tiles(a_req, adapter_ids, qsl, seq_lens, R, mode, max_adapters, max_tiles, tiles, counts, seg_scratch,
                           T, rowwise_cap, shrink_tiles, t_ready, status);
        __syncthreads();  // a builder that follows in this block reuses the scratch
    }
    if ((int)blockIdx.x == b_attn && items != nullptr && block_tables != nullptr) {
        metadata_attn_items(qsl, seq_lens, R, Hkv, q_block, small_max, max_items, items, counts, blk_off,
                            n_sm, attn_cta_start, status);
        __syncthreads();
    }
    if (((int)blockIdx.x == b_split || split_helper) && split_items != nullptr && block_tables != nullptr)
        metadata_split_items(qsl, seq_lens, block_tables, max_blocks, page_size, R, Hkv, G, n_sm, small_max, max_split_items,
                             max_split_rows, split_items, counts, req_scratch, group_done, prefix_groups,
                             split_helper ? (int)blockIdx.x - b_split : 0, split_parts, status);
    if (!proj) tc::grid_dep_wait();
}

// The projection phase for a batch on the few-row route (at most kFewRowMax tokens, one block): per-token arrays
// and the adapter facts, nothing else.  A kernel of its own because every step of a decode loop waits for it: it
// runs once per call on one SM, so what it costs is mostly the fetch of its instructions, and this one is short.
__global__ void __launch_bounds__(kFewRowMax)
metadata_few_row_kernel(const int32_t *__restrict__ positions, const int32_t *a_req, const int32_t *adapter_ids,
                        const int32_t *qsl, const int32_t *seq_lens, const int32_t *__restrict__ block_tables,
                        int max_blocks, int num_pages, int page_size, int max_adapters, int T, int R, int mode,
                        int32_t *__restrict__ token_req, int32_t *__restrict__ row_adapter,
                        int32_t *__restrict__ slot_map, const AdapterDev *__restrict__ adapters,
                        FewRowMeta *__restrict__ few_row_meta, int32_t *status) {
    __shared__ int32_t s_req[4 * kFewRowMax + 1];
    tc::grid_dep_launch();
    if (R <= kFewRowMax) {   // the per-request inputs are read several times (binary search): stage them
        int32_t *s_qsl = s_req, *s_len = s_req + R + 1, *s_ids = s_len + R, *s_areq = s_ids + R;
        for (int i = threadIdx.x; i <= R; i += blockDim.x) s_qsl[i] = qsl[i];
        for (int i = threadIdx.x; i < R; i += blockDim.x) {
            s_len[i] = seq_lens[i];
            if (adapter_ids) s_ids[i] = adapter_ids[i];
            if (a_req) s_areq[i] = a_req[i];
        }
        __syncthreads();
        qsl = s_qsl; seq_lens = s_len;
        if (adapter_ids) adapter_ids = s_ids;
        if (a_req) a_req = s_areq;
    }
    metadata_tokens(positions, a_req, adapter_ids, qsl, seq_lens, block_tables, max_blocks, num_pages, page_size,
                    max_adapters, T, R, mode, token_req, row_adapter, slot_map, adapters, status);
    if (few_row_meta != nullptr) metadata_few_row(row_adapter, adapters, T, max_adapters, few_row_meta);
}

int launch_metadata(alora_ctx *ctx, const BatchArgs &b, cudaStream_t s, int phases, bool timed) {
    if (b.T == 0) {
        if (phases & kMetaProjection) cudaMemsetAsync(ctx->d_counts, 0, 6 * sizeof(int32_t), s);
        return 0;
    }
    const bool saved = ctx->profiling;
    if (!timed) ctx->profiling = false;
    ProfScope prof(ctx, KK_METADATA, s);
    ctx->profiling = saved;
    const int threads = 256;
    const bool attn_only = phases == kMetaAttention;
    // (attention phase alone: one block for the tensor-core list, kSplitBuilders for the few-row list; they need the
    // shared-memory scratch, i.e. batches of at most 511 requests, else one block builds it in the global scratch)
    constexpr int kSplitBuilders = 8;
    const int grid = attn_only ? (14 * b.R + 5 <= kMetaSmemInts ? 1 + kSplitBuilders : 2) : std::max((phases & kMetaAttention) ? 3 : 1, (b.T + threads - 1) / threads);
    const AdapterDev *ads = b.layer >= 0 ? ctx->d_adapters + (size_t)b.layer * ctx->cfg.max_adapters : nullptr;
    FewRowMeta *few = (b.few_row && ads != nullptr) ? (FewRowMeta *)ctx->d_skinny_meta : nullptr;
    if (phases == kMetaProjection && b.few_row && b.T <= kFewRowMax) {
        metadata_few_row_kernel<<<1, kFewRowMax, 0, s>>>(
            b.positions, b.activation_offsets, b.adapter_ids, b.query_start_loc, b.seq_lens, b.block_tables, b.max_blocks,
            b.num_pages, ctx->d.page, ctx->cfg.max_adapters, b.T, b.R, b.mode, ctx->d_token_req, ctx->d_row_adapter,
            ctx->d_slot, ads, few, ctx->d_status);
        return 1;
    }
    const cudaError_t e = launch_kernel(metadata_kernel, dim3(grid), dim3(threads), 0, s, attn_only,
        b.positions, b.activation_offsets, b.adapter_ids, b.query_start_loc, b.seq_lens, b.block_tables,
        b.max_blocks, b.num_pages, ctx->d.page, ctx->cfg.max_adapters, b.T, b.R, b.mode, ctx->d_token_req,
        ctx->d_row_adapter, ctx->d_slot, ctx->max_tiles, ctx->d_tiles, ctx->d_counts, ctx->d_seg_scratch,
        ctx->d_shrink_tiles, ctx->d_t_ready,
        ctx->d.Hkv, ctx->attn_q_block, ctx->max_attn_items, ctx->d_attn_items, ctx->d_attn_off, ctx->d.G,
        ctx->sm_count, ctx->small_max_tokens, ctx->max_split_items, ctx->max_split_rows, ctx->d_split_items,
        ctx->d_req_scratch, ctx->d_group_done, ctx->d_row_delta ? kRowwiseMaxTokens : 0,
        ctx->d_attn_cta_start, ads, phases, few, ctx->d_prefix_groups, ctx->d_status);
    return e == cudaSuccess ? 1 : -1;
}

}  // namespace alora

// Self-test of the bounded wait that every tensor-core kernel of the library relies on: one block waits on an
// mbarrier that nobody arrives at, with a caller-given cycle limit.  The wait must give up, the block records
// ALORA_ERR_TIMEOUT in the context's status word and returns through its normal exit; nothing is left waiting.
#include "alora_internal.h"
#include "tc_common.cuh"
#include "claim_order.h"
#include <vector>

namespace alora {

__global__ void __launch_bounds__(32) wait_timeout_selftest_kernel(long long limit_cycles, int32_t *status) {
    __shared__ uint64_t bar;
    __shared__ int abort_flag;
    if (threadIdx.x == 0) {
        abort_flag = 0;
        tc::mbar_init(tc::smem_u32(&bar), 1);
        tc::fence_barrier_init();
    }
    __syncthreads();
    // phase 0 of a barrier with one expected arrival and no arriver never completes
    const bool done = tc::mbar_wait(tc::smem_u32(&bar), 0, &abort_flag, limit_cycles);
    __syncthreads();
    if (threadIdx.x == 0 && (!done || abort_flag)) report(status, ALORA_ERR_TIMEOUT);
}

}  // namespace alora

extern "C" alora_status alora_selftest_wait_timeout(alora_ctx *ctx, int64_t limit_cycles, void *stream) {
    if (!ctx) return ALORA_ERR_INVALID_ARG;
    // at most about a tenth of a second at 2 GHz: this is a check of the give-up path, not a way to stall a GPU
    if (limit_cycles < 1 || limit_cycles > 200000000LL) return ALORA_ERR_INVALID_ARG;
    ALORA_CUDA(ctx, cudaSetDevice(ctx->cfg.device));
    alora::wait_timeout_selftest_kernel<<<1, 32, 0, (cudaStream_t)stream>>>((long long)limit_cycles, ctx->d_status);
    ALORA_CUDA(ctx, cudaGetLastError());
    ctx->launches += 1;
    return ALORA_OK;
}

// Host-side model of a projection launch's item order (claim_order.h) on a GPU that keeps only `resident_slots`
// blocks running at a time.  Shrink item m serves row tile m (m < n_shrink); projection item
// n_shrink + m * n_col_tiles + n waits for shrink item m when m < n_shrink.  An item with no unmet dependency
// completes as soon as a running block holds it.  Blocks enter free slots highest index first or lowest first; a
// block leaves its slot when its list is exhausted.  `static_order` != 0 models the order that deals EVERY item by
// block index (shrink items included), which lets running blocks wait for blocks that never get a slot.
extern "C" alora_status alora_selftest_claim_order(int grid, int n_shrink, int n_row_tiles, int n_col_tiles,
                                                   int resident_slots, int high_blocks_first, int static_order,
                                                   int *completed) {
    if (!completed || grid < 1 || n_shrink < 0 || n_row_tiles < n_shrink || n_col_tiles < 1 || resident_slots < 1 ||
        grid > 65536 || (long long)n_row_tiles * n_col_tiles > (1 << 24))
        return ALORA_ERR_INVALID_ARG;
    using alora::claims_at_once;
    using alora::next_dealt_item;
    const int total = n_shrink + n_row_tiles * n_col_tiles;
    struct Block {
        int stat; bool started, finished, shrink_phase, looking_on; int pending;   // pending: an item held but blocked
    };
    std::vector<Block> blocks((size_t)grid);
    for (int b = 0; b < grid; ++b) blocks[b] = Block{b, false, false, false, false, -1};
    std::vector<char> shrink_done((size_t)std::max(n_shrink, 1), 0);
    int counter = 0, done_items = 0, running = 0, next_to_start = 0;
    auto dep_met = [&](int item) {
        if (item < n_shrink) return true;
        const int m = (item - n_shrink) / n_col_tiles;
        return m >= n_shrink || shrink_done[m] != 0;
    };
    auto complete = [&](int item) { if (item < n_shrink) shrink_done[item] = 1; ++done_items; };
    for (;;) {
        while (running < resident_slots && next_to_start < grid) {   // free slots take the next blocks
            Block &k = blocks[high_blocks_first ? grid - 1 - next_to_start : next_to_start];
            const int idx = high_blocks_first ? grid - 1 - next_to_start : next_to_start;
            k.started = true;
            k.shrink_phase = !static_order && n_shrink > 0;
            k.looking_on = k.shrink_phase && !claims_at_once(idx, n_shrink);
            ++next_to_start; ++running;
        }
        bool progress = false;
        for (int b = 0; b < grid; ++b) {
            Block &k = blocks[b];
            if (!k.started || k.finished) continue;
            for (;;) {
                if (k.pending >= 0) {                       // an item this block already holds
                    if (!dep_met(k.pending)) break;
                    complete(k.pending); k.pending = -1; progress = true;
                    continue;
                }
                int item = -1;
                if (static_order) {
                    if (k.stat < total) { item = k.stat; k.stat += grid; }
                } else {
                    if (k.looking_on) {
                        if (counter < n_shrink) break;       // still looking on (expires below when nothing else moves)
                        k.looking_on = false; k.shrink_phase = false;
                    }
                    if (k.shrink_phase) {
                        item = counter++;
                        if (item >= n_shrink) { k.shrink_phase = false; item = -1; }
                    }
                    if (!k.shrink_phase && item < 0) item = next_dealt_item(k.stat, n_shrink, total, grid);
                }
                if (item < 0) { k.finished = true; --running; progress = true; break; }
                k.pending = item;
            }
        }
        if (done_items == total) { *completed = 1; return ALORA_OK; }
        if (progress) continue;
        // nothing moved: the look-on period of the waiting blocks runs out and they join the claiming
        bool joined = false;
        for (int b = 0; b < grid; ++b)
            if (blocks[b].started && !blocks[b].finished && blocks[b].looking_on) { blocks[b].looking_on = false; joined = true; }
        if (joined) continue;
        *completed = 0;                                     // running blocks wait for items nobody running holds
        return ALORA_OK;
    }
}

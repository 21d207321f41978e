// Refinement of the maps against the real response lengths (paper Sec. 4.3.1, the paragraph
// after the map update): a request that ends before its predicted length has the rest of its
// ramp taken out of its instance's map; a request still running at its predicted end is
// extended by a fifth of its length (rounded up) and the extension added.
//
// One pass over the table, HBM-bound: 20 bytes per table row (five int32 columns) plus a
// read-modify-write of the touched map cells.  Few rows change per tick (those whose real end
// is now), so the map updates are done by whole warps: a warp takes 32 consecutive rows, votes
// which of them changed, and applies each changed row's ramp with consecutive lanes on
// consecutive map cells (64-bit integer reductions, order-independent, hence deterministic).
#include "pre_common.cuh"

namespace {

constexpr int REFINE_THREADS = 256;
constexpr int REFINE_WARPS = REFINE_THREADS / 32;
constexpr int32_t REFINE_MAX_D = 1 << 30;   // D + ceil(D/5) stays an int32

__global__ void __launch_bounds__(REFINE_THREADS)
pre_refine_requests(const int32_t* __restrict__ prompt, const int32_t* __restrict__ generated,
                    int32_t* __restrict__ predicted, const int32_t* __restrict__ instance,
                    const int32_t* __restrict__ actual, const int64_t* __restrict__ n_requests, int I, int H,
                    const int64_t* __restrict__ head_p, int64_t* __restrict__ curves, int64_t* __restrict__ current_d,
                    unsigned long long* __restrict__ counts, int* __restrict__ status) {
    __shared__ unsigned int sh_tally[3];
    if (threadIdx.x < 3) sh_tally[threadIdx.x] = 0;
    __syncthreads();
    const int64_t n = *n_requests;
    // dense maps: step j of a row is cell j; maps kept as a ring: cell (head + j) mod H
    const unsigned int head = head_p ? (unsigned int)(*head_p % H) : 0u;
    const int lane = threadIdx.x & 31, warp = threadIdx.x >> 5;
    const int64_t stride = (int64_t)gridDim.x * REFINE_WARPS * 32;
    unsigned int n_early = 0, n_ext = 0, n_bad = 0;
    for (int64_t base = ((int64_t)blockIdx.x * REFINE_WARPS + warp) * 32; base < n; base += stride) {
        const int64_t r = base + lane;
        int kind = 0;            // 1: finished early, 2: extended
        int32_t inst = 0, new_d = 0;
        long long first = 0;     // tokens held at window step 0 by the part of the ramp that changes
        int32_t steps = 0;       // length of that part
        if (r < n) {
            const int32_t P = prompt[r], g = generated[r], D = predicted[r], act = actual[r];
            inst = instance[r];
            if (!pre_request_ok(P, g, D, inst, I) || act < 1 || D > REFINE_MAX_D) {
                ++n_bad;
            } else if (g < D && act <= g) {
                kind = 1; steps = D - g; new_d = g;
            } else if (g == D && act > g) {
                kind = 2; steps = (int32_t)(((int64_t)D + 4) / 5); new_d = D + steps;
            }
            first = (long long)P + g;
        }
        unsigned int todo = __ballot_sync(0xffffffffu, kind != 0);
        while (todo) {
            const int src = __ffs(todo) - 1;
            todo &= todo - 1;
            const int row = __shfl_sync(0xffffffffu, inst, src);
            const long long f = __shfl_sync(0xffffffffu, first, src);
            const int len0 = __shfl_sync(0xffffffffu, steps, src);
            const bool take_out = __shfl_sync(0xffffffffu, kind, src) == 1;
            const int len = len0 < H ? len0 : H;
            unsigned long long* c = reinterpret_cast<unsigned long long*>(curves + (size_t)row * H);
            for (int j = lane; j < len; j += 32) {
                const long long v = f + j;
                unsigned int at = head + (unsigned int)j;
                if (at >= (unsigned int)H) at -= (unsigned int)H;
                atomicAdd(c + at, (unsigned long long)(take_out ? -v : v));
            }
        }
        if (kind != 0) {
            predicted[r] = new_d;
            const long long delta = kind == 1 ? -(long long)steps : (long long)steps;
            atomicAdd(reinterpret_cast<unsigned long long*>(current_d + inst), (unsigned long long)delta);
            if (kind == 1) ++n_early; else ++n_ext;
        }
    }
    n_early = __reduce_add_sync(0xffffffffu, n_early);
    n_ext = __reduce_add_sync(0xffffffffu, n_ext);
    n_bad = __reduce_add_sync(0xffffffffu, n_bad);
    if (lane == 0) {
        if (n_early) atomicAdd(&sh_tally[0], n_early);
        if (n_ext) atomicAdd(&sh_tally[1], n_ext);
        if (n_bad) atomicAdd(&sh_tally[2], n_bad);
    }
    __syncthreads();
    if (threadIdx.x < 3 && sh_tally[threadIdx.x]) {
        if (counts) atomicAdd(&counts[threadIdx.x], (unsigned long long)sh_tally[threadIdx.x]);
        if (threadIdx.x == 2) atomicOr(status, PRE_ST_BADREQ);
    }
}

}  // namespace

// `width` and `head`: the maps are rows of `width` cells; with `head` (a device word) they are
// rings and step j lies at cell (head + j) mod width, without it step j is cell j.
cudaError_t pre_launch_refine(pre_ctx* ctx, const int32_t* prompt, const int32_t* generated, int32_t* predicted,
                              const int32_t* instance, const int32_t* actual, const int64_t* n_requests,
                              int64_t* curves, int width, const int64_t* head, int64_t* current_d, int64_t* counts,
                              cudaStream_t s) {
    if (counts) {
        cudaError_t e = cudaMemsetAsync(counts, 0, 3 * sizeof(int64_t), s);
        if (e != cudaSuccess) return e;
    }
    // The row count lives on the device: size the grid for the table's capacity, a warp per 32 rows,
    // at most eight blocks per SM (grid-stride beyond that).
    int64_t blocks = (ctx->cfg.max_requests + REFINE_THREADS - 1) / REFINE_THREADS;
    const int64_t cap = 8 * (int64_t)ctx->n_sm;
    if (blocks > cap) blocks = cap;
    if (blocks < 1) blocks = 1;
    pre_refine_requests<<<(int)blocks, REFINE_THREADS, 0, s>>>(
        prompt, generated, predicted, instance, actual, n_requests, ctx->cfg.n_instances, width, head, curves,
        current_d, reinterpret_cast<unsigned long long*>(counts), ctx->d_status);
    return cudaGetLastError();
}

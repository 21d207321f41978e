// Refinement of the maps against the real response lengths (paper Sec. 4.3.1, the paragraph
// after the map update): a request that ends before its predicted length has the rest of its
// ramp taken out of its instance's map; a request still running at its predicted end is
// extended by a fifth of its length (rounded up) and the extension added.
//
// One pass over the table, HBM-bound: 20 bytes per table row (five int32 columns) plus a
// read-modify-write of the touched map cells.  Few rows change per tick (those whose real end
// is now), so the map updates are done by whole warps: a warp takes 128 consecutive rows (four
// per lane, one 16-byte load per column), votes which of them changed, and applies each changed
// row's ramp with consecutive lanes on consecutive map cells (64-bit integer reductions, order-independent, hence deterministic).
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
    const int64_t stride = (int64_t)gridDim.x * REFINE_WARPS * 128;
    unsigned int n_early = 0, n_ext = 0, n_bad = 0;
    // A warp takes 128 consecutive rows, four per lane (16-byte loads when the columns allow it).
    const bool vec = ((reinterpret_cast<uintptr_t>(prompt) | reinterpret_cast<uintptr_t>(generated) |
                       reinterpret_cast<uintptr_t>(predicted) | reinterpret_cast<uintptr_t>(instance) |
                       reinterpret_cast<uintptr_t>(actual)) & 15) == 0;
    for (int64_t base = ((int64_t)blockIdx.x * REFINE_WARPS + warp) * 128; base < n; base += stride) {
        const int64_t r0 = base + lane * 4;
        int32_t P[4], g[4], D[4], act[4], inst[4];
        if (vec && r0 + 4 <= n) {
            const int4 p4 = __ldg(reinterpret_cast<const int4*>(prompt + r0));
            const int4 g4 = __ldg(reinterpret_cast<const int4*>(generated + r0));
            const int4 d4 = *reinterpret_cast<const int4*>(predicted + r0);
            const int4 i4 = __ldg(reinterpret_cast<const int4*>(instance + r0));
            const int4 a4 = __ldg(reinterpret_cast<const int4*>(actual + r0));
            P[0] = p4.x; P[1] = p4.y; P[2] = p4.z; P[3] = p4.w;
            g[0] = g4.x; g[1] = g4.y; g[2] = g4.z; g[3] = g4.w;
            D[0] = d4.x; D[1] = d4.y; D[2] = d4.z; D[3] = d4.w;
            inst[0] = i4.x; inst[1] = i4.y; inst[2] = i4.z; inst[3] = i4.w;
            act[0] = a4.x; act[1] = a4.y; act[2] = a4.z; act[3] = a4.w;
        } else {
            #pragma unroll
            for (int e = 0; e < 4; ++e) {
                const bool in = r0 + e < n;
                P[e] = in ? prompt[r0 + e] : 0; g[e] = in ? generated[r0 + e] : 0;
                D[e] = in ? predicted[r0 + e] : 1; inst[e] = in ? instance[r0 + e] : 0;
                act[e] = in ? actual[r0 + e] : 2;     // a row beyond the table: well formed, nothing to do
            }
        }
        #pragma unroll
        for (int e = 0; e < 4; ++e) {
            int kind = 0;            // 1: finished early, 2: extended
            int32_t new_d = 0, steps = 0;   // steps: length of the part of the ramp that changes
            if (r0 + e < n) {
                if (!pre_request_ok(P[e], g[e], D[e], inst[e], I) || act[e] < 1 || D[e] > REFINE_MAX_D) {
                    ++n_bad;
                } else if (g[e] < D[e] && act[e] <= g[e]) {
                    kind = 1; steps = D[e] - g[e]; new_d = g[e];
                } else if (g[e] == D[e] && act[e] > g[e]) {
                    kind = 2; steps = (int32_t)(((int64_t)D[e] + 4) / 5); new_d = D[e] + steps;
                }
            }
            const long long first = (long long)P[e] + g[e];   // tokens held at window step 0 by that part
            unsigned int todo = __ballot_sync(0xffffffffu, kind != 0);
            while (todo) {
                const int src = __ffs(todo) - 1;
                todo &= todo - 1;
                const int row = __shfl_sync(0xffffffffu, inst[e], src);
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
                predicted[r0 + e] = new_d;
                const long long delta = kind == 1 ? -(long long)steps : (long long)steps;
                atomicAdd(reinterpret_cast<unsigned long long*>(current_d + inst[e]), (unsigned long long)delta);
                if (kind == 1) ++n_early; else ++n_ext;
            }
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
    // (A last-block reduction of the counts instead of this clear was measured 12 us slower: its
    // fence waits for the block's map reductions in flight.)
    if (counts) {
        cudaError_t e = cudaMemsetAsync(counts, 0, 3 * sizeof(int64_t), s);
        if (e != cudaSuccess) return e;
    }
    // The row count lives on the device: size the grid for the table's capacity, a warp per 128 rows,
    // at most eight blocks per SM (grid-stride beyond that).
    int64_t blocks = (ctx->cfg.max_requests + 4 * REFINE_THREADS - 1) / (4 * REFINE_THREADS);
    const int64_t cap = 8 * (int64_t)ctx->n_sm;
    if (blocks > cap) blocks = cap;
    if (blocks < 1) blocks = 1;
    pre_refine_requests<<<(int)blocks, REFINE_THREADS, 0, s>>>(
        prompt, generated, predicted, instance, actual, n_requests, ctx->cfg.n_instances, width, head, curves,
        current_d, reinterpret_cast<unsigned long long*>(counts), ctx->d_status);
    return cudaGetLastError();
}

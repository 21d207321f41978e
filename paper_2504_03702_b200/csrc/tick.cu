// One scheduler tick in two passes: the decode iteration (iteration-level batching, paper Sec. 2),
// the refinement of the maps against real response lengths (Sec. 4.3.1) and the scaler's signals
// (Sec. 4.3.2), which pre_step, pre_refine and pre_scaler_signals compute in four passes.
//
//   pre_tick_requests  one pass over the request table (five columns): g += 1 for live requests,
//                      live counts and what enters the window, and, on the advanced row, the
//                      refinement: the changed part of the ramp is taken out of (or added to) the
//                      map as it will be AFTER the shift, i.e. step j of the new map is cell j+1 of
//                      the map as it still stands, and step H-1 is the entering column;
//   pre_tick_shift     one pass over the maps: shift every row left by one cell, write the entering
//                      column, update current_d and queued_p, and take the row's maximum and its
//                      number of cells above the overload level from the values being written.
// All map updates are integer additions, so doing the refinement's before the shift gives the
// same cells as doing them after it.
#include <cmath>

#include "pre_common.cuh"

namespace {

constexpr int TICK_THREADS = 512;
constexpr int TICK_WARPS = TICK_THREADS / 32;
constexpr int SHIFT_THREADS = 256;
constexpr int SHIFT_WARPS = SHIFT_THREADS / 32;
constexpr int32_t REFINE_MAX_D = 1 << 30;   // D + ceil(D/5) stays an int32
constexpr long long I64_MIN = (-9223372036854775807LL - 1);

__device__ __forceinline__ long long warp_max64(long long v) {
    const unsigned int hi = (unsigned int)((unsigned long long)v >> 32) ^ 0x80000000u;  // order preserving
    const unsigned int lo = (unsigned int)v;
    const unsigned int mh = __reduce_max_sync(0xffffffffu, hi);
    const unsigned int ml = __reduce_max_sync(0xffffffffu, hi == mh ? lo : 0u);
    return (long long)(((unsigned long long)(mh ^ 0x80000000u) << 32) | ml);
}

__global__ void __launch_bounds__(TICK_THREADS)
pre_tick_requests(const int32_t* __restrict__ prompt, int32_t* __restrict__ generated, int32_t* __restrict__ predicted,
                  const int32_t* __restrict__ instance, const int32_t* __restrict__ actual,
                  const int64_t* __restrict__ n_requests, long long max_requests, int I, int H,
                  int64_t* __restrict__ curves, int64_t* __restrict__ current_d, unsigned int* __restrict__ active,
                  unsigned long long* __restrict__ enter, unsigned long long* __restrict__ counts,
                  long long* __restrict__ summary, int* __restrict__ status) {
    extern __shared__ unsigned int sh_active[];
    __shared__ unsigned int sh_tally[3];
    const bool use_sh = I <= PRE_SMEM_BINS;
    long long n = *n_requests;
    if (n > max_requests) n = max_requests;
    if (use_sh)
        for (int i = threadIdx.x; i < I; i += blockDim.x) sh_active[i] = 0;
    if (threadIdx.x < 3) sh_tally[threadIdx.x] = 0;
    if (summary && blockIdx.x == 0 && threadIdx.x < 3) summary[threadIdx.x] = 0;   // the map pass adds its block totals
    __syncthreads();
    const int lane = threadIdx.x & 31, warp = threadIdx.x >> 5;
    const bool vec = ((reinterpret_cast<uintptr_t>(prompt) | reinterpret_cast<uintptr_t>(generated) |
                       reinterpret_cast<uintptr_t>(predicted) | reinterpret_cast<uintptr_t>(instance) |
                       reinterpret_cast<uintptr_t>(actual)) & 15) == 0;
    bool any_bad = false;
    unsigned int n_early = 0, n_ext = 0, n_bad = 0;
    // A warp takes 128 consecutive rows, four per lane (16-byte loads when the columns allow it).
    const long long stride = (long long)gridDim.x * TICK_WARPS * 128;
    for (long long base = ((long long)blockIdx.x * TICK_WARPS + warp) * 128; base < n; base += stride) {
        const long long r0 = base + lane * 4;
        int32_t P[4], g[4], D[4], inst[4], act[4];
        if (vec && r0 + 4 <= n) {
            const int4 p4 = __ldg(reinterpret_cast<const int4*>(prompt + r0));
            const int4 g4 = *reinterpret_cast<const int4*>(generated + r0);
            const int4 d4 = *reinterpret_cast<const int4*>(predicted + r0);
            const int4 i4 = __ldg(reinterpret_cast<const int4*>(instance + r0));
            P[0] = p4.x; P[1] = p4.y; P[2] = p4.z; P[3] = p4.w;
            g[0] = g4.x; g[1] = g4.y; g[2] = g4.z; g[3] = g4.w;
            D[0] = d4.x; D[1] = d4.y; D[2] = d4.z; D[3] = d4.w;
            inst[0] = i4.x; inst[1] = i4.y; inst[2] = i4.z; inst[3] = i4.w;
            if (actual) {
                const int4 a4 = __ldg(reinterpret_cast<const int4*>(actual + r0));
                act[0] = a4.x; act[1] = a4.y; act[2] = a4.z; act[3] = a4.w;
            }
        } else {
            #pragma unroll
            for (int e = 0; e < 4; ++e) {
                const bool in = r0 + e < n;
                P[e] = in ? prompt[r0 + e] : 0; g[e] = in ? generated[r0 + e] : 1;
                D[e] = in ? predicted[r0 + e] : 1; inst[e] = in ? instance[r0 + e] : 0;   // beyond the table: a tombstone
                if (actual) act[e] = in ? actual[r0 + e] : 1;
            }
        }
        int32_t g1[4];
        bool moved = false;
        #pragma unroll
        for (int e = 0; e < 4; ++e) {
            g1[e] = g[e];
            const bool in = r0 + e < n;
            const bool ok = in && pre_request_ok(P[e], g[e], D[e], inst[e], I);
            any_bad |= in && !ok;
            // ---- the decode iteration
            if (ok && g[e] < D[e]) {
                g1[e] = g[e] + 1;
                moved = true;
                if (use_sh) atomicAdd(&sh_active[inst[e]], 1u); else atomicAdd(&active[inst[e]], 1u);
                if ((long long)D[e] - g1[e] >= (long long)H)   // still running when step H-1 enters the window
                    atomicAdd(&enter[inst[e]], (unsigned long long)((long long)P[e] + g1[e] + (H - 1)));
            }
            // ---- the refinement, on the advanced row
            int kind = 0;            // 1: finished early, 2: extended
            int32_t new_d = 0, steps = 0;
            if (actual && in) {
                if (!ok || act[e] < 1 || D[e] > REFINE_MAX_D) {
                    ++n_bad;
                } else if (g1[e] < D[e] && act[e] <= g1[e]) {
                    kind = 1; steps = D[e] - g1[e]; new_d = g1[e];
                } else if (g1[e] == D[e] && act[e] > g1[e]) {
                    kind = 2; steps = (int32_t)(((int64_t)D[e] + 4) / 5); new_d = D[e] + steps;
                }
            }
            const long long first = (long long)P[e] + g1[e];   // tokens held at step 0 of the new map by the changed part
            unsigned int todo = actual ? __ballot_sync(0xffffffffu, kind != 0) : 0u;
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
                    const long long v = take_out ? -(f + j) : f + j;
                    // step j of the map after the shift: cell j+1 as the map stands, the entering column for the last one
                    if (j + 1 < H) atomicAdd(c + j + 1, (unsigned long long)v);
                    else atomicAdd(&enter[row], (unsigned long long)v);
                }
            }
            if (kind != 0) {
                D[e] = new_d;
                moved = true;
                const long long delta = kind == 1 ? -(long long)steps : (long long)steps;
                atomicAdd(reinterpret_cast<unsigned long long*>(current_d + inst[e]), (unsigned long long)delta);
                if (kind == 1) ++n_early; else ++n_ext;
            }
        }
        if (moved) {
            if (vec && r0 + 4 <= n) {
                *reinterpret_cast<int4*>(generated + r0) = make_int4(g1[0], g1[1], g1[2], g1[3]);
                if (actual) *reinterpret_cast<int4*>(predicted + r0) = make_int4(D[0], D[1], D[2], D[3]);
            } else {
                #pragma unroll
                for (int e = 0; e < 4; ++e) {
                    if (r0 + e < n) {
                        generated[r0 + e] = g1[e];
                        if (actual) predicted[r0 + e] = D[e];
                    }
                }
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
    if (use_sh) {
        for (int i = threadIdx.x; i < I; i += blockDim.x) {
            const unsigned int c = sh_active[i];
            if (c) atomicAdd(&active[i], c);
        }
    }
    if (threadIdx.x < 3 && sh_tally[threadIdx.x]) {
        if (counts) atomicAdd(&counts[threadIdx.x], (unsigned long long)sh_tally[threadIdx.x]);
        if (threadIdx.x == 2) atomicOr(status, PRE_ST_BADREQ);
    }
    if (any_bad) atomicOr(status, PRE_ST_BADREQ);
}

// One block per row and trip.  The row is moved in passes of four cells per thread; a pass reads all
// its cells before it writes any, and pass p reads cell (p+1)*1024 before pass p+1 writes it.
__global__ void __launch_bounds__(SHIFT_THREADS)
pre_tick_shift(int64_t* __restrict__ curves, int64_t* __restrict__ queued_p, int64_t* __restrict__ current_d,
               unsigned int* __restrict__ active, unsigned long long* __restrict__ enter, int I, int H,
               long long hot, double many, double idle, int32_t* __restrict__ over_count,
               int64_t* __restrict__ row_max, long long* __restrict__ summary) {
    __shared__ int sh_cnt[2][SHIFT_WARPS];          // per-warp partials of a row, by parity of the block's row count:
    __shared__ long long sh_max[2][SHIFT_WARPS];    // thread 0 adds them up one row later, after the barrier that ends the row
    const int lane = threadIdx.x & 31, warp = threadIdx.x >> 5;
    const bool signals = summary != nullptr;
    long long n_over = 0, n_busy = 0, sum = 0;     // thread 0 only
    auto close_row = [&](int row, int par) {       // thread 0: the signals of a row whose partials are complete
        int c = 0;
        long long m = I64_MIN;
        for (int w = 0; w < SHIFT_WARPS; ++w) { c += sh_cnt[par][w]; m = sh_max[par][w] > m ? sh_max[par][w] : m; }
        over_count[row] = c;
        row_max[row] = m;
        n_over += (double)c > many;
        n_busy += !((double)m < idle);
        sum += m;
    };
    int it = 0;
    for (int row = blockIdx.x; row < I; row += gridDim.x, ++it) {
        int64_t* rp = curves + (size_t)row * H;
        const long long last = (long long)enter[row];
        int cnt = 0;
        long long mx = I64_MIN;
        for (int base = 0; base < H; base += SHIFT_THREADS * 4) {
            long long v[4];
            #pragma unroll
            for (int u = 0; u < 4; ++u) {
                const int j = base + u * SHIFT_THREADS + threadIdx.x;
                v[u] = (j + 1 < H) ? rp[j + 1] : last;
            }
            __syncthreads();
            #pragma unroll
            for (int u = 0; u < 4; ++u) {
                const int j = base + u * SHIFT_THREADS + threadIdx.x;
                if (j < H) {
                    rp[j] = v[u];
                    cnt += v[u] > hot;
                    mx = v[u] > mx ? v[u] : mx;
                }
            }
            __syncthreads();
        }
        if (signals) {
            cnt = __reduce_add_sync(0xffffffffu, cnt);
            mx = warp_max64(mx);
            if (lane == 0) { sh_cnt[it & 1][warp] = cnt; sh_max[it & 1][warp] = mx; }
        }
        if (threadIdx.x == 0) {
            current_d[row] -= (long long)active[row];
            queued_p[row] = 0;
            active[row] = 0;
            enter[row] = 0;
            if (signals && it > 0) close_row(row - (int)gridDim.x, (it - 1) & 1);
        }
        __syncthreads();
    }
    if (signals && threadIdx.x == 0) {
        if (it > 0) close_row(blockIdx.x + (it - 1) * (int)gridDim.x, (it - 1) & 1);
        // integer sums into words that the table pass cleared: no fence, no waiting for the block's stores
        if (n_over) atomicAdd(reinterpret_cast<unsigned long long*>(summary), (unsigned long long)n_over);
        if (n_busy) atomicAdd(reinterpret_cast<unsigned long long*>(summary) + 1, (unsigned long long)n_busy);
        if (sum) atomicAdd(reinterpret_cast<unsigned long long*>(summary) + 2, (unsigned long long)sum);
    }
}

}  // namespace

cudaError_t pre_launch_tick(pre_ctx* ctx, int32_t* prompt, int32_t* generated, int32_t* predicted, int32_t* instance,
                            const int32_t* actual, const int64_t* n_requests, int64_t* curves, int64_t* queued_p,
                            int64_t* current_d, double overload_level, double overload_share, double idle_level,
                            int32_t* over_count, int64_t* row_max, int64_t* summary, int64_t* counts, cudaStream_t s) {
    const int I = ctx->cfg.n_instances, H = ctx->cfg.horizon;
    if (counts) {
        cudaError_t e = cudaMemsetAsync(counts, 0, 3 * sizeof(int64_t), s);
        if (e != cudaSuccess) return e;
    }
    const size_t smem = I <= PRE_SMEM_BINS ? (size_t)I * sizeof(unsigned int) : 0;
    long long want = (ctx->cfg.max_requests + TICK_THREADS * 4 - 1) / (TICK_THREADS * 4);
    // two blocks per SM: every block flushes its live counts with one global atomic per instance
    int grid = (int)(want < 2LL * ctx->n_sm ? want : 2LL * ctx->n_sm);
    if (grid < 1) grid = 1;
    pre_tick_requests<<<grid, TICK_THREADS, smem, s>>>(prompt, generated, predicted, instance, actual, n_requests,
                                                      ctx->cfg.max_requests, I, H, curves, current_d, ctx->d_active,
                                                      ctx->d_enter, reinterpret_cast<unsigned long long*>(counts),
                                                      reinterpret_cast<long long*>(summary), ctx->d_status);
    // For a whole number c, c > x holds exactly when c > floor(x): the per-cell test is done on integers.
    double hot_d = floor(overload_level * (double)ctx->cfg.capacity_tokens);
    if (hot_d > 9.2e18) hot_d = 9.2e18;
    if (hot_d < -9.2e18) hot_d = -9.2e18;
    const double many = overload_share * (double)H;
    const double idle = idle_level * (double)ctx->cfg.capacity_tokens;
    int sgrid = I < 16 * ctx->n_sm ? I : 16 * ctx->n_sm;
    pre_tick_shift<<<sgrid, SHIFT_THREADS, 0, s>>>(curves, queued_p, current_d, ctx->d_active, ctx->d_enter, I, H,
                                                  (long long)hot_d, many, idle, over_count, row_max,
                                                  reinterpret_cast<long long*>(summary));
    return cudaGetLastError();
}

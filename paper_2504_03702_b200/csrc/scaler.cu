// Signals for the proactive instance scaler (paper Sec. 4.3.2), one pass over the maps:
// per instance the number of steps above the overload level and the row maximum; for the
// whole service the number of potentially overloaded instances, the number of instances that
// do not stay below the idle level, and the sum of the row maxima.
//
// HBM-bound by definition (8*I*H bytes read once).  One warp per row and trip, 16-byte
// loads, eight in flight per lane.  Block totals go to a scratch array; the block that finishes
// last adds them up and writes the summary (no memset, no atomics on the result, same sum order
// every time).
#include <cmath>

#include "pre_common.cuh"

namespace {

constexpr int SCALER_THREADS = 256;
constexpr int SCALER_WARPS = SCALER_THREADS / 32;
constexpr int SCALER_BATCH = 8;            // 16-byte loads a lane has in flight
constexpr int SCALER_BLOCKS_PER_SM = 8;
constexpr long long I64_MIN = (-9223372036854775807LL - 1);

__device__ __forceinline__ long long warp_max64(long long v) {
    const unsigned int hi = (unsigned int)((unsigned long long)v >> 32) ^ 0x80000000u;  // order preserving
    const unsigned int lo = (unsigned int)v;
    const unsigned int mh = __reduce_max_sync(0xffffffffu, hi);
    const unsigned int ml = __reduce_max_sync(0xffffffffu, hi == mh ? lo : 0u);
    return (long long)(((unsigned long long)(mh ^ 0x80000000u) << 32) | ml);
}

__global__ void __launch_bounds__(SCALER_THREADS)
pre_scaler_rows(const int64_t* __restrict__ curves, int I, int H, long long hot, double many, double idle,
                int32_t* __restrict__ over_count, int64_t* __restrict__ row_max, long long* __restrict__ summary,
                long long* __restrict__ partial, unsigned int* __restrict__ done) {
    __shared__ int sh_over[SCALER_WARPS], sh_busy[SCALER_WARPS];
    __shared__ long long sh_sum[SCALER_WARPS];
    const int lane = threadIdx.x & 31, warp = threadIdx.x >> 5;
    const bool vec = (H & 1) == 0;
    int n_over = 0, n_busy = 0;
    long long sum = 0;
    for (int row = blockIdx.x * SCALER_WARPS + warp; row < I; row += gridDim.x * SCALER_WARPS) {
        const int64_t* rp = curves + (size_t)row * H;
        int cnt = 0;
        long long mx = I64_MIN;
        if (vec) {
            int j = lane * 2;
            for (; j + (SCALER_BATCH - 1) * 64 < H; j += SCALER_BATCH * 64) {
                longlong2 v[SCALER_BATCH];
                #pragma unroll
                for (int u = 0; u < SCALER_BATCH; ++u) v[u] = __ldcs(reinterpret_cast<const longlong2*>(rp + j + u * 64));
                #pragma unroll
                for (int u = 0; u < SCALER_BATCH; ++u) {
                    cnt += (v[u].x > hot) + (v[u].y > hot);
                    mx = v[u].x > mx ? v[u].x : mx;
                    mx = v[u].y > mx ? v[u].y : mx;
                }
            }
            for (; j < H; j += 64) {
                const longlong2 v = __ldcs(reinterpret_cast<const longlong2*>(rp + j));
                cnt += (v.x > hot) + (v.y > hot);
                mx = v.x > mx ? v.x : mx;
                mx = v.y > mx ? v.y : mx;
            }
        } else {
            for (int j = lane; j < H; j += 32) {
                const long long v = __ldcs(rp + j);
                cnt += v > hot;
                mx = v > mx ? v : mx;
            }
        }
        cnt = __reduce_add_sync(0xffffffffu, cnt);
        mx = warp_max64(mx);
        if (lane == 0) {
            over_count[row] = cnt;
            row_max[row] = mx;
            n_over += (double)cnt > many;
            n_busy += !((double)mx < idle);
            sum += mx;
        }
    }
    if (lane == 0) { sh_over[warp] = n_over; sh_busy[warp] = n_busy; sh_sum[warp] = sum; }
    __syncthreads();
    __shared__ bool sh_last;
    if (threadIdx.x == 0) {
        long long o = 0, b = 0, s = 0;
        for (int w = 0; w < SCALER_WARPS; ++w) { o += sh_over[w]; b += sh_busy[w]; s += sh_sum[w]; }
        partial[blockIdx.x * 3 + 0] = o;
        partial[blockIdx.x * 3 + 1] = b;
        partial[blockIdx.x * 3 + 2] = s;
        __threadfence();
        sh_last = atomicAdd(done, 1u) == gridDim.x - 1;
    }
    __syncthreads();
    if (sh_last && threadIdx.x < 32) {   // every other block's totals are visible (fence before its count)
        __threadfence();
        long long o = 0, b = 0, s = 0;
        for (int g = lane; g < (int)gridDim.x; g += 32) {
            o += __ldcg(&partial[g * 3 + 0]); b += __ldcg(&partial[g * 3 + 1]); s += __ldcg(&partial[g * 3 + 2]);
        }
        #pragma unroll
        for (int off = 16; off > 0; off >>= 1) {
            o += __shfl_xor_sync(0xffffffffu, o, off);
            b += __shfl_xor_sync(0xffffffffu, b, off);
            s += __shfl_xor_sync(0xffffffffu, s, off);
        }
        if (lane == 0) { summary[0] = o; summary[1] = b; summary[2] = s; *done = 0; }   // ready for the next call
    }
}

}  // namespace

cudaError_t pre_launch_scaler(pre_ctx* ctx, const int64_t* curves, double overload_level, double overload_share,
                              double idle_level, int32_t* over_count, int64_t* row_max, int64_t* summary,
                              cudaStream_t s) {
    const int I = ctx->cfg.n_instances, H = ctx->cfg.horizon;
    // For a whole number c, c > x holds exactly when c > floor(x): the per-cell test is done on integers.
    double hot_d = floor(overload_level * (double)ctx->cfg.capacity_tokens);
    if (hot_d > 9.2e18) hot_d = 9.2e18;
    if (hot_d < -9.2e18) hot_d = -9.2e18;
    const long long hot = (long long)hot_d;
    const double many = overload_share * (double)H;
    const double idle = idle_level * (double)ctx->cfg.capacity_tokens;
    int grid = (I + SCALER_WARPS - 1) / SCALER_WARPS;
    const int cap = SCALER_BLOCKS_PER_SM * ctx->n_sm;
    if (grid > cap) grid = cap;
    pre_scaler_rows<<<grid, SCALER_THREADS, 0, s>>>(curves, I, H, hot, many, idle, over_count, row_max,
                                                    reinterpret_cast<long long*>(summary), ctx->d_scaler_partial,
                                                    ctx->d_scaler_done);
    return cudaGetLastError();
}

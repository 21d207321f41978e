// One decode iteration: every live request generates a token, finished requests retire,
// every load-look-ahead map moves one iteration closer (iteration-level batching, paper
// Sec. 2; "the next iterations" of the map, Sec. 4.3.1).
//
//   pre_step_requests  one pass over the request table: g += 1 for live requests, count
//                      them per instance, and collect what enters the window at step H-1;
//   pre_step_shift     one pass over the maps: shift every row left by one cell, write the
//                      entering column, update current_d and queued_p, clear the scratch.
#include "pre_common.cuh"

namespace {

constexpr int STEP_THREADS = 512;
constexpr int SHIFT_THREADS = 256;

__global__ void __launch_bounds__(STEP_THREADS)
pre_step_requests(const int32_t* __restrict__ prompt, int32_t* __restrict__ generated,
                  const int32_t* __restrict__ predicted, const int32_t* __restrict__ instance,
                  const int64_t* __restrict__ n_requests, long long max_requests, int I, int H,
                  unsigned int* __restrict__ active, unsigned long long* __restrict__ enter,
                  int* __restrict__ status) {
    extern __shared__ unsigned int sh_active[];
    const bool use_sh = I <= PRE_SMEM_BINS;
    long long n = *n_requests;
    if (n > max_requests) n = max_requests;
    if (use_sh) {
        for (int i = threadIdx.x; i < I; i += blockDim.x) sh_active[i] = 0;
        __syncthreads();
    }
    bool any_bad = false;
    // one request: returns the new g (the old one when nothing changes)
    auto tick = [&](int32_t P, int32_t g, int32_t D, int32_t inst) -> int32_t {
        if (P < 0 || g < 0 || D < 1 || (uint32_t)inst >= (uint32_t)I) { any_bad = true; return g; }
        if (g >= D) return g;  // tombstone
        const int32_t g1 = g + 1;
        if (use_sh) atomicAdd(&sh_active[inst], 1u); else atomicAdd(&active[inst], 1u);
        if ((long long)D - g1 >= (long long)H)   // still running when step H-1 enters the window
            atomicAdd(&enter[inst], (unsigned long long)((long long)P + g1 + (H - 1)));
        return g1;
    };
    const long long stride = (long long)gridDim.x * blockDim.x;
    const long long gtid = (long long)blockIdx.x * blockDim.x + threadIdx.x;
    const bool vec = ((reinterpret_cast<uintptr_t>(prompt) | reinterpret_cast<uintptr_t>(generated) |
                       reinterpret_cast<uintptr_t>(predicted) | reinterpret_cast<uintptr_t>(instance)) & 15) == 0;
    if (vec) {
        const long long n4 = n >> 2;
        for (long long q = gtid; q < n4; q += stride) {
            const int4 p = __ldg(reinterpret_cast<const int4*>(prompt) + q);
            int4 g = *(reinterpret_cast<const int4*>(generated) + q);
            const int4 d = __ldg(reinterpret_cast<const int4*>(predicted) + q);
            const int4 i = __ldg(reinterpret_cast<const int4*>(instance) + q);
            const int4 o = g;
            g.x = tick(p.x, g.x, d.x, i.x); g.y = tick(p.y, g.y, d.y, i.y);
            g.z = tick(p.z, g.z, d.z, i.z); g.w = tick(p.w, g.w, d.w, i.w);
            if (g.x != o.x || g.y != o.y || g.z != o.z || g.w != o.w) *(reinterpret_cast<int4*>(generated) + q) = g;
        }
        for (long long r = (n4 << 2) + gtid; r < n; r += stride) {
            const int32_t g = generated[r];
            const int32_t g1 = tick(prompt[r], g, predicted[r], instance[r]);
            if (g1 != g) generated[r] = g1;
        }
    } else {
        for (long long r = gtid; r < n; r += stride) {
            const int32_t g = generated[r];
            const int32_t g1 = tick(prompt[r], g, predicted[r], instance[r]);
            if (g1 != g) generated[r] = g1;
        }
    }
    if (use_sh) {
        __syncthreads();
        for (int i = threadIdx.x; i < I; i += blockDim.x) {
            const unsigned int c = sh_active[i];
            if (c) atomicAdd(&active[i], c);
        }
    }
    if (any_bad) atomicOr(status, PRE_ST_BADREQ);
}

// One block per row.  The row is moved in passes of blockDim cells; a pass reads all its
// cells before it writes any, and pass p reads cell (p+1)*blockDim before pass p+1 writes it.
__global__ void __launch_bounds__(SHIFT_THREADS)
pre_step_shift(int64_t* __restrict__ curves, int64_t* __restrict__ queued_p, int64_t* __restrict__ current_d,
               unsigned int* __restrict__ active, unsigned long long* __restrict__ enter, int I, int H) {
    for (int row = blockIdx.x; row < I; row += gridDim.x) {
        int64_t* rp = curves + (size_t)row * H;
        const long long last = (long long)enter[row];
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
                if (j < H) rp[j] = v[u];
            }
            __syncthreads();
        }
        if (threadIdx.x == 0) {
            current_d[row] -= (long long)active[row];
            queued_p[row] = 0;
            active[row] = 0;
            enter[row] = 0;
        }
        __syncthreads();
    }
}

}  // namespace

// The pass over the request table alone, for a map of `width` steps (the shift of a dense map,
// or the advance of a ring, follows).
cudaError_t pre_launch_step_requests(pre_ctx* ctx, int32_t* prompt, int32_t* generated, int32_t* predicted,
                                     int32_t* instance, const int64_t* n_requests, int width, cudaStream_t s) {
    const int I = ctx->cfg.n_instances;
    const size_t smem = I <= PRE_SMEM_BINS ? (size_t)I * sizeof(unsigned int) : 0;
    long long want = (ctx->cfg.max_requests + STEP_THREADS * 4 - 1) / (STEP_THREADS * 4);
    int grid = (int)(want < 2LL * ctx->n_sm ? want : 2LL * ctx->n_sm);   // fewer blocks, fewer per-block flushes of the live counts
    if (grid < 1) grid = 1;
    pre_step_requests<<<grid, STEP_THREADS, smem, s>>>(prompt, generated, predicted, instance, n_requests,
                                                     ctx->cfg.max_requests, I, width, ctx->d_active, ctx->d_enter,
                                                     ctx->d_status);
    return cudaGetLastError();
}

cudaError_t pre_launch_step(pre_ctx* ctx, int32_t* prompt, int32_t* generated, int32_t* predicted,
                            int32_t* instance, const int64_t* n_requests, int64_t* curves,
                            int64_t* queued_p, int64_t* current_d, cudaStream_t s) {
    const int I = ctx->cfg.n_instances, H = ctx->cfg.horizon;
    cudaError_t e = pre_launch_step_requests(ctx, prompt, generated, predicted, instance, n_requests, H, s);
    if (e != cudaSuccess) return e;
    int sgrid = I < 16 * ctx->n_sm ? I : 16 * ctx->n_sm;
    pre_step_shift<<<sgrid, SHIFT_THREADS, 0, s>>>(curves, queued_p, current_d, ctx->d_active, ctx->d_enter, I, H);
    return cudaGetLastError();
}

// Full-width load-look-ahead maps kept as a ring over absolute iterations.
//
// Paper Sec. 4.3.1: the map of an instance covers the next L iterations, L being the largest
// response the model can produce (e.g. 4,096), while the load is projected "over the next l
// iterations" (e.g. l = 100) for the router and the scaler.  Here a row of the map is a ring
//     ring[i*L + (head + j) mod L] = tokens of instance i at j iterations from now, 0 <= j < L,
// so that a decode iteration moves no map data: the head advances and the slot that fell out of
// the past becomes step L-1.  The router works on the window, the first l steps, copied into a
// dense array (pre_ring_window); its real updates beyond the window are applied to the ring
// afterwards, all arrivals of the batch in parallel (pre_ring_fold): integer additions commute,
// and no score of the batch depends on a step beyond the window.
//
//   pre_ring_window_copy   window[i][j] = ring[i][(head + j) mod L], j < l
//   pre_ring_fold_ramps    a warp per routed arrival: ring[choice][(head + j) mod L] += P + j, j < min(D, L)
//   pre_ring_advance       after the pass over the request table of pre_step: the freed slot of
//                          every row receives what enters at step L-1, backlog and queue words
//                          are updated, the block that finishes last advances the head
#include "pre_common.cuh"

namespace {

constexpr int RING_THREADS = 256;

__global__ void __launch_bounds__(RING_THREADS)
pre_ring_window_copy(const int64_t* __restrict__ ring, int I, int L, int l, const int64_t* __restrict__ head_p,
                     int64_t* __restrict__ window) {
    const unsigned int head = (unsigned int)(*head_p % L);
    const long long total = (long long)I * l;
    const long long stride = (long long)gridDim.x * blockDim.x;
    for (long long idx = (long long)blockIdx.x * blockDim.x + threadIdx.x; idx < total; idx += stride) {
        const unsigned int i = (unsigned int)(idx / l), j = (unsigned int)(idx - (long long)i * l);
        unsigned int at = head + j;
        if (at >= (unsigned int)L) at -= (unsigned int)L;
        window[idx] = ring[(size_t)i * L + at];
    }
}

__global__ void __launch_bounds__(RING_THREADS)
pre_ring_fold_ramps(const int32_t* __restrict__ arr_prompt, const int32_t* __restrict__ arr_predicted,
                    const int32_t* __restrict__ choice, long long n_arrivals, int I, int L,
                    const int64_t* __restrict__ head_p, int64_t* __restrict__ ring) {
    const unsigned int head = (unsigned int)(*head_p % L);
    const int lane = threadIdx.x & 31;
    const long long warps = (long long)gridDim.x * (RING_THREADS / 32);
    for (long long k = (long long)blockIdx.x * (RING_THREADS / 32) + (threadIdx.x >> 5); k < n_arrivals; k += warps) {
        const int32_t c = choice[k];
        if (c < 0 || c >= I) continue;                      // not routed (malformed, table full, waiting)
        const long long P = arr_prompt[k];
        const int32_t D = arr_predicted[k];
        const int len = D < L ? D : L;
        unsigned long long* row = reinterpret_cast<unsigned long long*>(ring) + (size_t)c * L;
        for (int j = lane; j < len; j += 32) {
            unsigned int at = head + (unsigned int)j;
            if (at >= (unsigned int)L) at -= (unsigned int)L;
            atomicAdd(row + at, (unsigned long long)(P + j));
        }
    }
}

__global__ void __launch_bounds__(RING_THREADS)
pre_ring_advance(int64_t* __restrict__ ring, int I, int L, int64_t* __restrict__ head_p,
                 int64_t* __restrict__ queued_p, int64_t* __restrict__ current_d, unsigned int* __restrict__ active,
                 unsigned long long* __restrict__ enter, unsigned int* __restrict__ done) {
    const unsigned int head = (unsigned int)(*head_p % L);
    for (int row = blockIdx.x * blockDim.x + threadIdx.x; row < I; row += gridDim.x * blockDim.x) {
        ring[(size_t)row * L + head] = (int64_t)enter[row];     // step 0 of the old map is step L-1 of the new one
        current_d[row] -= (long long)active[row];
        queued_p[row] = 0;
        active[row] = 0;
        enter[row] = 0;
    }
    // every block has read the head before the last one to finish moves it
    __syncthreads();
    if (threadIdx.x == 0) {
        __threadfence();
        if (atomicAdd(done, 1u) == gridDim.x - 1) {
            *head_p = (int64_t)((head + 1u) % (unsigned int)L);
            *done = 0;
        }
    }
}

}  // namespace

cudaError_t pre_launch_ring_window(pre_ctx* ctx, const int64_t* ring, int width, const int64_t* head,
                                   int64_t* window, cudaStream_t s) {
    const int I = ctx->cfg.n_instances, l = ctx->cfg.horizon;
    long long blocks = ((long long)I * l + RING_THREADS - 1) / RING_THREADS;
    if (blocks > 16LL * ctx->n_sm) blocks = 16LL * ctx->n_sm;
    pre_ring_window_copy<<<(int)blocks, RING_THREADS, 0, s>>>(ring, I, width, l, head, window);
    return cudaGetLastError();
}

cudaError_t pre_launch_ring_fold(pre_ctx* ctx, const int32_t* arr_prompt, const int32_t* arr_predicted,
                                 const int32_t* choice, int64_t n_arrivals, int64_t* ring, int width,
                                 const int64_t* head, cudaStream_t s) {
    if (n_arrivals == 0) return cudaSuccess;
    long long blocks = (n_arrivals + RING_THREADS / 32 - 1) / (RING_THREADS / 32);
    if (blocks > 16LL * ctx->n_sm) blocks = 16LL * ctx->n_sm;
    pre_ring_fold_ramps<<<(int)blocks, RING_THREADS, 0, s>>>(arr_prompt, arr_predicted, choice, n_arrivals,
                                                           ctx->cfg.n_instances, width, head, ring);
    return cudaGetLastError();
}

cudaError_t pre_launch_ring_step(pre_ctx* ctx, int32_t* prompt, int32_t* generated, int32_t* predicted,
                                 int32_t* instance, const int64_t* n_requests, int64_t* ring, int width,
                                 int64_t* head, int64_t* queued_p, int64_t* current_d, cudaStream_t s) {
    cudaError_t e = pre_launch_step_requests(ctx, prompt, generated, predicted, instance, n_requests, width, s);
    if (e != cudaSuccess) return e;
    const int I = ctx->cfg.n_instances;
    int blocks = (I + RING_THREADS - 1) / RING_THREADS;
    if (blocks > 4 * ctx->n_sm) blocks = 4 * ctx->n_sm;
    pre_ring_advance<<<blocks, RING_THREADS, 0, s>>>(ring, I, width, head, queued_p, current_d, ctx->d_active,
                                                   ctx->d_enter, ctx->d_ring_done);
    return cudaGetLastError();
}

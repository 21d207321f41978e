// Load-aware request router (paper Sec. 4.3.3) as one persistent kernel per batch.
//
// The grid is launched cooperatively (all blocks resident).  Block b owns a fixed,
// contiguous set of instance rows for the whole batch, so every read and every fold of a
// row happens inside one block and needs only block-level ordering.  Per arrival:
//   1. every warp streams its share of the block's rows with 16-byte loads and keeps, per
//      row, m1 = max_{j<Dc}(c[j] + j) and m2 = max_{j>=Dc} c[j]   (Dc = min(D, H));
//      the peak with the arrival virtually added is max(P + m1, m2);
//   2. warp 0 turns the peaks into scores, takes the block's (score, index) minimum and
//      publishes it in a global slot tagged with the arrival's running number;
//   3. warp 0 of every block reads all G slots (bounded spin), so every block knows the
//      winner without a second barrier; slots are double buffered by the tag's parity;
//   4. the owner of the winning row adds the arrival's ramp to it, updates queued_p and
//      current_d; block 0 appends the request and writes choice/score.
#include "pre_common.cuh"

#include <math_constants.h>

namespace {

constexpr int ROUTE_THREADS = 512;
constexpr int ROUTE_WARPS = ROUTE_THREADS / 32;
constexpr long long I64_MIN = (-9223372036854775807LL - 1);
constexpr unsigned int SPIN_LIMIT = 1u << 22;  // polls before a wait is declared lost

__device__ __forceinline__ void st_release_u64(unsigned long long* p, unsigned long long v) {
    asm volatile("st.release.gpu.global.u64 [%0], %1;" ::"l"(p), "l"(v) : "memory");
}
__device__ __forceinline__ unsigned long long ld_acquire_u64(const unsigned long long* p) {
    unsigned long long v;
    asm volatile("ld.acquire.gpu.global.u64 %0, [%1];" : "=l"(v) : "l"(p) : "memory");
    return v;
}
__device__ __forceinline__ unsigned long long ld_relaxed_u64(const unsigned long long* p) {
    unsigned long long v;
    asm volatile("ld.relaxed.gpu.global.u64 %0, [%1];" : "=l"(v) : "l"(p) : "memory");
    return v;
}
__device__ __forceinline__ int ld_relaxed_s32(const int* p) {
    int v;
    asm volatile("ld.relaxed.gpu.global.s32 %0, [%1];" : "=r"(v) : "l"(p) : "memory");
    return v;
}
// Streaming loads served by L2 (no L1 allocation): a row is re-read only after ~I*H*8 bytes.
__device__ __forceinline__ longlong2 ld_cg_v2(const int64_t* p) {
    return __ldcg(reinterpret_cast<const longlong2*>(p));
}
__device__ __forceinline__ long long ld_cg(const int64_t* p) {
    return __ldcg(reinterpret_cast<const long long*>(p));
}

__device__ __forceinline__ long long max64(long long a, long long b) { return a > b ? a : b; }

// Score of one instance, binary64, every operation rounded on its own.
__device__ __forceinline__ double score_of(long long queued_p, long long current_d, long long peak, int P,
                                           int D, double theta, double beta) {
    double over = __dsub_rn((double)peak, theta);
    if (over < 0.0) over = 0.0;
    const double lp = (double)(queued_p + (long long)P);
    const double ld = (double)(current_d + (long long)D);
    const double lm = __dmul_rn(beta, over);
    return __dadd_rn(__dadd_rn(lp, ld), lm);
}

__device__ __forceinline__ bool better(double s, int i, double bs, int bi) {
    return s < bs || (s == bs && i < bi);
}

struct RouteArgs {
    const int32_t* arr_prompt;
    const int32_t* arr_predicted;
    long long n_arrivals;
    int64_t* curves;
    int64_t* queued_p;
    int64_t* current_d;
    int32_t* prompt;
    int32_t* generated;
    int32_t* predicted;
    int32_t* instance;
    int64_t* n_requests;
    long long max_requests;
    int32_t* choice;
    double* score;
    int I, H;
    double theta, beta;
    unsigned long long* slots;  // [2][G][2]
    unsigned int epoch;
    int* status;
    int* abort_flag;
    int max_rows;  // ceil(I / G)
};

__global__ void __launch_bounds__(ROUTE_THREADS, 1) pre_route_persistent(const RouteArgs a) {
    extern __shared__ __align__(16) unsigned char smem_raw[];
    long long* m1 = reinterpret_cast<long long*>(smem_raw);  // [max_rows]
    long long* m2 = m1 + a.max_rows;                         // [max_rows]
    long long* sq = m2 + a.max_rows;                         // queued_p of the owned rows
    long long* scd = sq + a.max_rows;                        // current_d of the owned rows
    __shared__ int sh_winner;
    __shared__ double sh_score;
    __shared__ int sh_dead;
    __shared__ long long sh_n0;

    const int G = gridDim.x, b = blockIdx.x;
    const int tid = threadIdx.x, lane = tid & 31, warp = tid >> 5;
    const int I = a.I, H = a.H;
    const int row0 = (int)(((long long)b * I) / G);
    const int row1 = (int)(((long long)(b + 1) * I) / G);
    const int nrows = row1 - row0;
    const int cpr = (H + 63) >> 6;  // 64-cell chunks per row (one 16-byte load per lane)
    const long long nch = (long long)nrows * cpr;
    const long long ch0 = nch * warp / ROUTE_WARPS, ch1 = nch * (warp + 1) / ROUTE_WARPS;
    const bool vec = (H & 1) == 0;

    for (int r = tid; r < nrows; r += ROUTE_THREADS) {
        sq[r] = a.queued_p[row0 + r];
        scd[r] = a.current_d[row0 + r];
    }
    if (tid == 0) { sh_dead = 0; sh_n0 = *a.n_requests; }
    __syncthreads();
    const long long n0 = sh_n0;
    long long room = a.max_requests - n0;
    if (room < 0) room = 0;
    long long appended = 0;  // meaningful in every thread: all blocks take the same decisions
    bool saw_bad = false, saw_full = false;

    for (long long k = 0; k < a.n_arrivals; ++k) {
        const int P = a.arr_prompt[k], D = a.arr_predicted[k];
        if (P < 0 || D < 1 || P > PRE_FIELD_MAX || D > PRE_FIELD_MAX) {
            saw_bad = true;
            if (b == 0 && tid == 0) { a.choice[k] = -1; if (a.score) a.score[k] = 0.0; }
            continue;
        }
        if (appended >= room) {
            saw_full = true;
            if (b == 0 && tid == 0) { a.choice[k] = -1; if (a.score) a.score[k] = 0.0; }
            continue;
        }
        const int Dc = D < H ? D : H;
        for (int r = tid; r < nrows; r += ROUTE_THREADS) { m1[r] = I64_MIN; m2[r] = I64_MIN; }
        __syncthreads();

        // ---- 1. stream the owned rows
        long long c = ch0;
        while (c < ch1) {
            const int row = (int)(c / cpr);
            const long long row_end = ((long long)(row + 1) * cpr < ch1) ? (long long)(row + 1) * cpr : ch1;
            const int64_t* rp = a.curves + (size_t)(row0 + row) * H;
            long long a1 = I64_MIN, a2 = I64_MIN;
            int j = (int)(c - (long long)row * cpr) * 64 + lane * 2;
            if (vec) {
                long long q = c;
                for (; q + 4 <= row_end; q += 4, j += 256) {
                    longlong2 v[4];
                    #pragma unroll
                    for (int u = 0; u < 4; ++u) {
                        v[u] = (j + u * 64 < H) ? ld_cg_v2(rp + j + u * 64) : make_longlong2(I64_MIN, I64_MIN);
                    }
                    #pragma unroll
                    for (int u = 0; u < 4; ++u) {
                        const int jj = j + u * 64;
                        if (jj < H) {
                            if (jj < Dc) a1 = max64(a1, v[u].x + jj); else a2 = max64(a2, v[u].x);
                            if (jj + 1 < Dc) a1 = max64(a1, v[u].y + jj + 1); else a2 = max64(a2, v[u].y);
                        }
                    }
                }
                for (; q < row_end; ++q, j += 64) {
                    if (j < H) {
                        const longlong2 v = ld_cg_v2(rp + j);
                        if (j < Dc) a1 = max64(a1, v.x + j); else a2 = max64(a2, v.x);
                        if (j + 1 < Dc) a1 = max64(a1, v.y + j + 1); else a2 = max64(a2, v.y);
                    }
                }
            } else {
                for (long long q = c; q < row_end; ++q, j += 64) {
                    if (j < H) {
                        const long long x = ld_cg(rp + j);
                        if (j < Dc) a1 = max64(a1, x + j); else a2 = max64(a2, x);
                    }
                    if (j + 1 < H) {
                        const long long y = ld_cg(rp + j + 1);
                        if (j + 1 < Dc) a1 = max64(a1, y + j + 1); else a2 = max64(a2, y);
                    }
                }
            }
            #pragma unroll
            for (int off = 16; off > 0; off >>= 1) {
                a1 = max64(a1, __shfl_xor_sync(0xffffffffu, a1, off));
                a2 = max64(a2, __shfl_xor_sync(0xffffffffu, a2, off));
            }
            if (lane == 0) {
                atomicMax(&m1[row], a1);
                atomicMax(&m2[row], a2);
            }
            c = row_end;
        }
        __syncthreads();

        // ---- 2./3. block minimum, publish, gather
        if (warp == 0) {
            double bs = CUDART_INF;
            int bi = 0x7fffffff;
            for (int r = lane; r < nrows; r += 32) {
                long long peak = m1[r] + P;  // Dc >= 1: the ramp part is never empty
                if (m2[r] > peak) peak = m2[r];
                const double s = score_of(sq[r], scd[r], peak, P, D, a.theta, a.beta);
                if (better(s, row0 + r, bs, bi)) { bs = s; bi = row0 + r; }
            }
            #pragma unroll
            for (int off = 16; off > 0; off >>= 1) {
                const double os = __shfl_xor_sync(0xffffffffu, bs, off);
                const int oi = __shfl_xor_sync(0xffffffffu, bi, off);
                if (better(os, oi, bs, bi)) { bs = os; bi = oi; }
            }
            const unsigned int tag = a.epoch + (unsigned int)appended;  // dense: one tag per exchange
            unsigned long long* slot = a.slots + (size_t)(tag & 1u) * G * 2;
            if (lane == 0) {
                slot[b * 2] = (unsigned long long)__double_as_longlong(bs);
                st_release_u64(&slot[b * 2 + 1], ((unsigned long long)tag << 32) | (unsigned int)bi);
            }
            bool lost = false;
            bs = CUDART_INF;
            bi = 0x7fffffff;
            for (int cta = lane; cta < G && !lost; cta += 32) {
                unsigned long long w1;
                unsigned int polls = 0;
                for (;;) {
                    w1 = ld_acquire_u64(&slot[cta * 2 + 1]);
                    if ((unsigned int)(w1 >> 32) == tag) break;
                    if (++polls > SPIN_LIMIT || ((polls & 63u) == 0 && ld_relaxed_s32(a.abort_flag))) {
                        lost = true;
                        break;
                    }
                    if (polls > 256) __nanosleep(64);
                }
                if (!lost) {
                    const double s = __longlong_as_double((long long)ld_relaxed_u64(&slot[cta * 2]));
                    const int i = (int)(unsigned int)(w1 & 0xffffffffu);
                    if (better(s, i, bs, bi)) { bs = s; bi = i; }
                }
            }
            lost = __any_sync(0xffffffffu, lost);
            #pragma unroll
            for (int off = 16; off > 0; off >>= 1) {
                const double os = __shfl_xor_sync(0xffffffffu, bs, off);
                const int oi = __shfl_xor_sync(0xffffffffu, bi, off);
                if (better(os, oi, bs, bi)) { bs = os; bi = oi; }
            }
            if (lane == 0) {
                if (lost) {
                    atomicOr(a.status, PRE_ST_TIMEOUT);
                    atomicExch(a.abort_flag, 1);
                    sh_dead = 1;
                }
                sh_winner = bi;
                sh_score = bs;
            }
        }
        __syncthreads();
        if (sh_dead) break;
        const int w = sh_winner;

        // ---- 4. fold
        if (w >= row0 && w < row1) {
            int64_t* rp = a.curves + (size_t)w * H;
            for (int j = tid; j < Dc; j += ROUTE_THREADS) rp[j] += (long long)P + j;
            if (tid == 0) {
                const int r = w - row0;
                sq[r] += P;
                scd[r] += D;
                a.queued_p[w] = sq[r];
                a.current_d[w] = scd[r];
            }
        }
        if (b == 0 && tid == 0) {
            const long long slot = n0 + appended;
            a.prompt[slot] = P;
            a.generated[slot] = 0;
            a.predicted[slot] = D;
            a.instance[slot] = w;
            a.choice[k] = w;
            if (a.score) a.score[k] = sh_score;
        }
        ++appended;
        __syncthreads();
    }

    if (b == 0 && tid == 0) {
        *a.n_requests = n0 + appended;
        if (saw_bad) atomicOr(a.status, PRE_ST_BADREQ);
        if (saw_full) atomicOr(a.status, PRE_ST_CAPACITY);
    }
}

}  // namespace

cudaError_t pre_route_configure(pre_ctx* ctx) {
    const int I = ctx->cfg.n_instances;
    const int G = ctx->n_sm < I ? ctx->n_sm : I;  // one block per SM, never more blocks than rows
    const int max_rows = (I + G - 1) / G;
    const size_t smem = (size_t)max_rows * 4 * sizeof(long long);
    cudaError_t e = cudaFuncSetAttribute(pre_route_persistent, cudaFuncAttributeMaxDynamicSharedMemorySize,
                                         (int)(smem > 48 * 1024 ? smem : 48 * 1024));
    if (e != cudaSuccess) return e;
    int per_sm = 0;
    e = cudaOccupancyMaxActiveBlocksPerMultiprocessor(&per_sm, pre_route_persistent, ROUTE_THREADS, smem);
    if (e != cudaSuccess) return e;
    if (per_sm < 1) return cudaErrorInvalidConfiguration;
    ctx->route_blocks = G;
    ctx->route_threads = ROUTE_THREADS;
    ctx->route_smem = smem;
    return cudaSuccess;
}

cudaError_t pre_launch_route(pre_ctx* ctx, const int32_t* arr_prompt, const int32_t* arr_predicted,
                             int64_t n_arrivals, int64_t* curves, int64_t* queued_p, int64_t* current_d,
                             int32_t* prompt, int32_t* generated, int32_t* predicted, int32_t* instance,
                             int64_t* n_requests, int32_t* choice, double* score, cudaStream_t s) {
    if (n_arrivals == 0) return cudaSuccess;
    cudaError_t e = cudaMemsetAsync(ctx->d_abort, 0, sizeof(int), s);
    if (e != cudaSuccess) return e;
    RouteArgs a;
    a.arr_prompt = arr_prompt; a.arr_predicted = arr_predicted; a.n_arrivals = n_arrivals;
    a.curves = curves; a.queued_p = queued_p; a.current_d = current_d;
    a.prompt = prompt; a.generated = generated; a.predicted = predicted; a.instance = instance;
    a.n_requests = n_requests; a.max_requests = ctx->cfg.max_requests;
    a.choice = choice; a.score = score;
    a.I = ctx->cfg.n_instances; a.H = ctx->cfg.horizon;
    a.theta = ctx->theta; a.beta = ctx->cfg.beta;
    a.slots = ctx->d_slots; a.epoch = ctx->epoch;
    a.status = ctx->d_status; a.abort_flag = ctx->d_abort;
    a.max_rows = (a.I + ctx->route_blocks - 1) / ctx->route_blocks;
    ctx->epoch += (unsigned int)n_arrivals;
    void* params[] = {(void*)&a};
    return cudaLaunchCooperativeKernel((const void*)pre_route_persistent, dim3(ctx->route_blocks),
                                       dim3(ROUTE_THREADS), params, ctx->route_smem, s);
}

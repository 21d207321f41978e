// Anticipator build: request table -> load-look-ahead maps (paper Sec. 4.3.1).
//
// A live request (P, g, D) on instance i holds B + j tokens at step j for
// j < R, with B = P + g and R = min(D - g, H).  Written as difference arrays
// over the horizon, its constant part is "+B at 0, -B at R" and its slope part
// "+1 at 0, -1 at R".  Accumulating from the release end instead, both become a
// single update at column R-1 whose SUFFIX sums give
//     N[j] = #{r : R_r > j},   A[j] = sum{B_r : R_r > j},   c[j] = A[j] + j*N[j],
// so each request costs one shared-memory update and column 0 is not a hot spot.
//
// Pipeline (all on the caller's stream, no host synchronisation):
//   1. pre_bin_count    per-tile request counts (a tile = T consecutive instance rows)
//   2. pre_bin_scan     exclusive scan of the counts -> where each tile's records start
//   3. pre_bin_scatter  packs every live request into 8 bytes and writes it to its tile
//   4. pre_tile_build   one block per tile: shared-memory accumulation of (count, sum B)
//                       per (row, R-1), suffix scan over the horizon, writes the rows
#include "pre_common.cuh"

namespace {

constexpr int BIN_THREADS = 512;
constexpr int TILE_THREADS = 512;
constexpr int TILE_WARPS = TILE_THREADS / 32;

__global__ void __launch_bounds__(BIN_THREADS)
pre_bin_count(const int32_t* __restrict__ instance, int64_t n, int I, int T, int n_tiles,
              unsigned int* __restrict__ bin_count) {
    extern __shared__ unsigned int sh_bins[];
    const bool use_sh = n_tiles <= PRE_SMEM_BINS;
    if (use_sh) {
        for (int i = threadIdx.x; i < n_tiles; i += blockDim.x) sh_bins[i] = 0;
        __syncthreads();
    }
    const int64_t stride = (int64_t)gridDim.x * blockDim.x;
    for (int64_t r = (int64_t)blockIdx.x * blockDim.x + threadIdx.x; r < n; r += stride) {
        const int32_t v = instance[r];
        if ((uint32_t)v < (uint32_t)I) {
            const int b = v / T;
            if (use_sh) atomicAdd(&sh_bins[b], 1u); else atomicAdd(&bin_count[b], 1u);
        }
    }
    if (use_sh) {
        __syncthreads();
        for (int i = threadIdx.x; i < n_tiles; i += blockDim.x) {
            const unsigned int c = sh_bins[i];
            if (c) atomicAdd(&bin_count[i], c);
        }
    }
}

// One block.  base[b] = sum of count[0..b), cursor[b] = base[b]; the counts are cleared
// for the next call.
__global__ void __launch_bounds__(1024)
pre_bin_scan(unsigned int* __restrict__ bin_count, int n_tiles, unsigned int* __restrict__ bin_base,
             unsigned int* __restrict__ bin_cursor) {
    __shared__ unsigned int warp_tot[32];
    __shared__ unsigned int carry_sh;
    const int lane = threadIdx.x & 31, warp = threadIdx.x >> 5;
    if (threadIdx.x == 0) carry_sh = 0;
    __syncthreads();
    for (int start = 0; start < n_tiles; start += 1024) {
        const int i = start + threadIdx.x;
        const unsigned int v = i < n_tiles ? bin_count[i] : 0u;
        unsigned int x = v;
        #pragma unroll
        for (int off = 1; off < 32; off <<= 1) {
            const unsigned int y = __shfl_up_sync(0xffffffffu, x, off);
            if (lane >= off) x += y;
        }
        if (lane == 31) warp_tot[warp] = x;
        __syncthreads();
        unsigned int before = carry_sh;
        for (int w = 0; w < warp; ++w) before += warp_tot[w];
        if (i < n_tiles) {
            const unsigned int excl = before + x - v;
            bin_base[i] = excl;
            bin_cursor[i] = excl;
            bin_count[i] = 0;
        }
        __syncthreads();
        if (threadIdx.x == 1023) carry_sh = before + x;
        __syncthreads();
    }
    if (threadIdx.x == 0) bin_base[n_tiles] = carry_sh;
}

struct Packed { bool live; bool bad; int tile; unsigned long long rec; };

__device__ __forceinline__ Packed pack_request(int32_t P, int32_t g, int32_t D, int32_t inst, int I, int T) {
    Packed o;
    o.live = false; o.bad = false; o.tile = 0; o.rec = 0;
    if (!pre_request_ok(P, g, D, inst, I)) { o.bad = true; return o; }
    if (g >= D) return o;  // finished: tombstone
    const int64_t B = (int64_t)P + g;
    const int32_t rem = D - g;
    if (B > PRE_FIELD_MAX || rem > PRE_FIELD_MAX) { o.bad = true; return o; }
    o.live = true;
    o.tile = inst / T;
    const unsigned long long local = (unsigned long long)(inst - o.tile * T);
    o.rec = (local << (2 * PRE_FIELD_BITS)) | ((unsigned long long)B << PRE_FIELD_BITS) |
            (unsigned long long)rem;
    return o;
}

__global__ void __launch_bounds__(BIN_THREADS)
pre_bin_scatter(const int32_t* __restrict__ prompt, const int32_t* __restrict__ generated,
                const int32_t* __restrict__ predicted, const int32_t* __restrict__ instance, int64_t n,
                int I, int T, int n_tiles, unsigned int* __restrict__ bin_cursor,
                unsigned long long* __restrict__ records, int* __restrict__ status) {
    extern __shared__ unsigned int sh_bins[];
    const bool use_sh = n_tiles <= PRE_SMEM_BINS;
    const int64_t chunk = (n + gridDim.x - 1) / gridDim.x;
    const int64_t r0 = (int64_t)blockIdx.x * chunk;
    const int64_t r1 = r0 + chunk < n ? r0 + chunk : n;
    bool any_bad = false;
    if (use_sh) {
        for (int i = threadIdx.x; i < n_tiles; i += blockDim.x) sh_bins[i] = 0;
        __syncthreads();
        for (int64_t r = r0 + threadIdx.x; r < r1; r += blockDim.x) {
            const Packed p = pack_request(prompt[r], generated[r], predicted[r], instance[r], I, T);
            any_bad |= p.bad;
            if (p.live) atomicAdd(&sh_bins[p.tile], 1u);
        }
        __syncthreads();
        // reserve this block's span in every tile it touches; sh_bins becomes a write cursor
        for (int i = threadIdx.x; i < n_tiles; i += blockDim.x) {
            const unsigned int c = sh_bins[i];
            if (c) sh_bins[i] = atomicAdd(&bin_cursor[i], c);
        }
        __syncthreads();
        for (int64_t r = r0 + threadIdx.x; r < r1; r += blockDim.x) {
            const Packed p = pack_request(prompt[r], generated[r], predicted[r], instance[r], I, T);
            if (p.live) records[atomicAdd(&sh_bins[p.tile], 1u)] = p.rec;
        }
    } else {
        for (int64_t r = r0 + threadIdx.x; r < r1; r += blockDim.x) {
            const Packed p = pack_request(prompt[r], generated[r], predicted[r], instance[r], I, T);
            any_bad |= p.bad;
            if (p.live) records[atomicAdd(&bin_cursor[p.tile], 1u)] = p.rec;
        }
    }
    if (any_bad) atomicOr(status, PRE_ST_BADREQ);
}

// Shared-memory layout of one tile: count[cells], lo[cells], hi[cells] (uint32 each; the
// sum of B per cell is kept as lo + 2^32*hi so that only 32-bit shared atomics are needed),
// then per-row 64-bit words.
__global__ void __launch_bounds__(TILE_THREADS)
pre_tile_build(const unsigned long long* __restrict__ records, const unsigned int* __restrict__ bin_base,
               const unsigned int* __restrict__ bin_cursor, int I, int H, int T, int cells_pad,
               int64_t* __restrict__ curves, int64_t* __restrict__ current_d) {
    extern __shared__ __align__(16) unsigned char smem_raw[];
    uint32_t* cnt = reinterpret_cast<uint32_t*>(smem_raw);
    uint32_t* lo = cnt + cells_pad;
    uint32_t* hi = lo + cells_pad;
    unsigned long long* excess = reinterpret_cast<unsigned long long*>(hi + cells_pad);  // [T]
    unsigned long long* sum_n = excess + T;                                              // [T]
    unsigned long long* wt = sum_n + T;  // [2][TILE_WARPS][2] cross-warp totals, double buffered

    const int tile = blockIdx.x;
    const int row0 = tile * T;
    const int rows = (I - row0) < T ? (I - row0) : T;
    const int tid = threadIdx.x, lane = tid & 31, warp = tid >> 5;

    for (int i = tid; i < 3 * cells_pad; i += TILE_THREADS) cnt[i] = 0;
    for (int i = tid; i < 2 * T; i += TILE_THREADS) excess[i] = 0;
    __syncthreads();

    // ---- accumulate: one update per request at (row, R-1)
    const unsigned int rec0 = bin_base[tile], rec1 = bin_cursor[tile];
    for (unsigned int r = rec0 + tid; r < rec1; r += TILE_THREADS) {
        const unsigned long long rec = records[r];
        const uint32_t rem = (uint32_t)(rec & PRE_FIELD_MAX);
        const uint32_t B = (uint32_t)((rec >> PRE_FIELD_BITS) & PRE_FIELD_MAX);
        const int local = (int)(rec >> (2 * PRE_FIELD_BITS));
        const uint32_t R = rem < (uint32_t)H ? rem : (uint32_t)H;
        const int cell = local * H + (int)R - 1;
        atomicAdd(&cnt[cell], 1u);
        const uint32_t old = atomicAdd(&lo[cell], B);
        if (old + B < old) atomicAdd(&hi[cell], 1u);  // exactly one thread sees each wrap
        if (rem > (uint32_t)H) atomicAdd(&excess[local], (unsigned long long)(rem - (uint32_t)H));
    }
    __syncthreads();

    // ---- suffix scan over the horizon, `team_warps` warps per row
    int team_warps = 1;
    while (team_warps < TILE_WARPS && team_warps * 128 < H) team_warps <<= 1;
    const int teams = TILE_WARPS / team_warps;
    const int team = warp / team_warps, wteam = warp % team_warps;
    const int span = team_warps * 128;
    const int passes = (H + span - 1) / span;
    const bool vec_sm = (H & 3) == 0;
    const bool vec_gl = (H & 1) == 0;
    int buf = 0;

    for (int rb = 0; rb < rows; rb += teams) {
        const int row = rb + team;
        const bool active = row < rows;
        unsigned long long carry_n = 0, carry_s = 0, my_sum_n = 0;
        for (int p = passes - 1; p >= 0; --p) {
            const int j0 = p * span + (wteam * 32 + lane) * 4;
            unsigned long long n[4] = {0, 0, 0, 0}, s[4] = {0, 0, 0, 0};
            if (active && j0 < H) {
                const int c0 = row * H + j0;
                if (vec_sm) {
                    const uint4 a = *reinterpret_cast<const uint4*>(cnt + c0);
                    const uint4 b = *reinterpret_cast<const uint4*>(lo + c0);
                    const uint4 c = *reinterpret_cast<const uint4*>(hi + c0);
                    n[0] = a.x; n[1] = a.y; n[2] = a.z; n[3] = a.w;
                    s[0] = ((unsigned long long)c.x << 32) | b.x; s[1] = ((unsigned long long)c.y << 32) | b.y;
                    s[2] = ((unsigned long long)c.z << 32) | b.z; s[3] = ((unsigned long long)c.w << 32) | b.w;
                } else {
                    #pragma unroll
                    for (int k = 0; k < 4; ++k) {
                        if (j0 + k < H) {
                            n[k] = cnt[c0 + k];
                            s[k] = ((unsigned long long)hi[c0 + k] << 32) | lo[c0 + k];
                        }
                    }
                }
            }
            const unsigned long long tn = n[0] + n[1] + n[2] + n[3];
            const unsigned long long ts = s[0] + s[1] + s[2] + s[3];
            // inclusive suffix over the lanes of this warp (higher lane = later steps)
            unsigned long long xn = tn, xs = ts;
            #pragma unroll
            for (int off = 1; off < 32; off <<= 1) {
                const unsigned long long yn = __shfl_down_sync(0xffffffffu, xn, off);
                const unsigned long long ys = __shfl_down_sync(0xffffffffu, xs, off);
                if (lane + off < 32) { xn += yn; xs += ys; }
            }
            if (lane == 0) { wt[(buf * TILE_WARPS + warp) * 2] = xn; wt[(buf * TILE_WARPS + warp) * 2 + 1] = xs; }
            __syncthreads();
            unsigned long long above_n = carry_n, above_s = carry_s, team_n = 0, team_s = 0;
            for (int w = 0; w < team_warps; ++w) {
                const unsigned long long wn = wt[(buf * TILE_WARPS + team * team_warps + w) * 2];
                const unsigned long long ws = wt[(buf * TILE_WARPS + team * team_warps + w) * 2 + 1];
                team_n += wn; team_s += ws;
                if (w > wteam) { above_n += wn; above_s += ws; }
            }
            buf ^= 1;
            if (active && j0 < H) {
                unsigned long long N = above_n + (xn - tn), A = above_s + (xs - ts);
                unsigned long long c[4];
                #pragma unroll
                for (int k = 3; k >= 0; --k) {
                    N += n[k]; A += s[k];
                    c[k] = A + (unsigned long long)(j0 + k) * N;
                    if (j0 + k < H) my_sum_n += N;
                }
                int64_t* out = curves + ((size_t)(row0 + row) * H + j0);
                if (vec_gl) {
                    *reinterpret_cast<ulonglong2*>(out) = make_ulonglong2(c[0], c[1]);
                    if (j0 + 2 < H) *reinterpret_cast<ulonglong2*>(out + 2) = make_ulonglong2(c[2], c[3]);
                } else {
                    #pragma unroll
                    for (int k = 0; k < 4; ++k) if (j0 + k < H) out[k] = (int64_t)c[k];
                }
            }
            carry_n += team_n; carry_s += team_s;
        }
        // sum over j of N[j] = sum over requests of R (each request is counted on R steps)
        #pragma unroll
        for (int off = 16; off > 0; off >>= 1) my_sum_n += __shfl_xor_sync(0xffffffffu, my_sum_n, off);
        if (active && lane == 0 && my_sum_n) atomicAdd(&sum_n[row], my_sum_n);
    }
    __syncthreads();
    for (int i = tid; i < rows; i += TILE_THREADS) current_d[row0 + i] = (int64_t)(sum_n[i] + excess[i]);
}

}  // namespace

size_t pre_tile_smem_bytes(int tile_rows, int horizon) {
    const size_t cells_pad = (((size_t)tile_rows * horizon + 3) / 4) * 4 + 4;
    return 3 * cells_pad * sizeof(uint32_t) + 2 * (size_t)tile_rows * 8 + 2 * TILE_WARPS * 2 * 8;
}

cudaError_t pre_launch_anticipate(pre_ctx* ctx, const int32_t* prompt, const int32_t* generated,
                                  const int32_t* predicted, const int32_t* instance, int64_t n,
                                  int64_t* curves, int64_t* current_d, cudaStream_t s) {
    const int I = ctx->cfg.n_instances, H = ctx->cfg.horizon, T = ctx->tile_rows, nt = ctx->n_tiles;
    const size_t bins_smem = nt <= PRE_SMEM_BINS ? (size_t)nt * sizeof(unsigned int) : 0;
    int grid = (int)((n + BIN_THREADS * 8 - 1) / (BIN_THREADS * 8));
    if (grid > 2 * ctx->n_sm) grid = 2 * ctx->n_sm;
    if (grid < 1) grid = 1;
    if (n > 0) {
        pre_bin_count<<<grid, BIN_THREADS, bins_smem, s>>>(instance, n, I, T, nt, ctx->d_bin_count);
    }
    pre_bin_scan<<<1, 1024, 0, s>>>(ctx->d_bin_count, nt, ctx->d_bin_base, ctx->d_bin_cursor);
    if (n > 0) {
        pre_bin_scatter<<<grid, BIN_THREADS, bins_smem, s>>>(prompt, generated, predicted, instance, n, I, T, nt,
                                                           ctx->d_bin_cursor, ctx->d_records, ctx->d_status);
    }
    const size_t cells_pad = (((size_t)T * H + 3) / 4) * 4 + 4;
    pre_tile_build<<<nt, TILE_THREADS, pre_tile_smem_bytes(T, H), s>>>(
        ctx->d_records, ctx->d_bin_base, ctx->d_bin_cursor, I, H, T, (int)cells_pad, curves, current_d);
    return cudaGetLastError();
}

cudaError_t pre_anticipate_configure(pre_ctx* ctx) {
    return cudaFuncSetAttribute(pre_tile_build, cudaFuncAttributeMaxDynamicSharedMemorySize,
                                (int)pre_tile_smem_bytes(ctx->tile_rows, ctx->cfg.horizon));
}

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
//   2. pre_bin_scatter  scans the counts (where each tile's records start), packs every
//                       live request into 8 bytes and writes it to its tile's span
//      (pre_bin_scan    separate scan launch, only when there are too many tiles for the
//                       scatter blocks to scan in shared memory)
//   3. pre_tile_build   one block per tile: shared-memory accumulation of (count, sum B)
//                       per (row, R-1), suffix scan over the horizon, writes the rows
#include "pre_common.cuh"

namespace {

constexpr int BIN_THREADS = 512;
constexpr int TILE_THREADS = 512;
constexpr int TILE_WARPS = TILE_THREADS / 32;

// Per-tile request counts.  Finished and malformed requests may be counted too: the counts
// only reserve room, the scatter pass decides what is written.
__global__ void __launch_bounds__(BIN_THREADS)
pre_bin_count(const int32_t* __restrict__ instance, int64_t n, int I, int T, int n_tiles,
              unsigned int* __restrict__ bin_count) {
    extern __shared__ unsigned int sh_bins[];
    const bool use_sh = n_tiles <= PRE_SMEM_BINS;
    if (use_sh) {
        for (int i = threadIdx.x; i < n_tiles; i += blockDim.x) sh_bins[i] = 0;
        __syncthreads();
    }
    auto add = [&](int32_t v) {
        if ((uint32_t)v < (uint32_t)I) {
            const int b = v / T;
            if (use_sh) atomicAdd(&sh_bins[b], 1u); else atomicAdd(&bin_count[b], 1u);
        }
    };
    const int64_t stride = (int64_t)gridDim.x * blockDim.x;
    const int64_t gtid = (int64_t)blockIdx.x * blockDim.x + threadIdx.x;
    if ((reinterpret_cast<uintptr_t>(instance) & 15) == 0) {
        const int64_t n4 = n >> 2;
        const int4* in4 = reinterpret_cast<const int4*>(instance);
        for (int64_t q = gtid; q < n4; q += stride) {
            const int4 v = __ldg(in4 + q);
            add(v.x); add(v.y); add(v.z); add(v.w);
        }
        for (int64_t r = (n4 << 2) + gtid; r < n; r += stride) add(instance[r]);
    } else {
        for (int64_t r = gtid; r < n; r += stride) add(instance[r]);
    }
    if (use_sh) {
        __syncthreads();
        for (int i = threadIdx.x; i < n_tiles; i += blockDim.x) {
            const unsigned int c = sh_bins[i];
            if (c) atomicAdd(&bin_count[i], c);
        }
    }
}

// One block.  base[b] = sum of count[0..b).  Only used when the tile count is too large
// for the scatter blocks to scan it themselves in shared memory.
__global__ void __launch_bounds__(1024)
pre_bin_scan(const unsigned int* __restrict__ bin_count, int n_tiles, unsigned int* __restrict__ bin_base) {
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
        if (i < n_tiles) bin_base[i] = before + x - v;
        __syncthreads();
        if (threadIdx.x == 1023) carry_sh = before + x;
        __syncthreads();
    }
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

// Calls f(P, g, D, inst) for every request of [r0, r1); 16-byte loads when the four arrays
// allow it (r0 is then a multiple of 4, or the range is empty).
template <class F>
__device__ __forceinline__ void for_each_request(const int32_t* __restrict__ prompt,
                                                 const int32_t* __restrict__ generated,
                                                 const int32_t* __restrict__ predicted,
                                                 const int32_t* __restrict__ instance, int64_t r0, int64_t r1,
                                                 bool vec, F f) {
    if (vec) {
        const int64_t q1 = r1 >> 2;  // full quads end here
        for (int64_t q = (r0 >> 2) + threadIdx.x; q < q1; q += blockDim.x) {
            const int4 p = __ldg(reinterpret_cast<const int4*>(prompt) + q);
            const int4 g = __ldg(reinterpret_cast<const int4*>(generated) + q);
            const int4 d = __ldg(reinterpret_cast<const int4*>(predicted) + q);
            const int4 i = __ldg(reinterpret_cast<const int4*>(instance) + q);
            f(p.x, g.x, d.x, i.x); f(p.y, g.y, d.y, i.y); f(p.z, g.z, d.z, i.z); f(p.w, g.w, d.w, i.w);
        }
        for (int64_t r = (q1 << 2) + threadIdx.x; r < r1; r += blockDim.x)
            if (r >= r0) f(prompt[r], generated[r], predicted[r], instance[r]);
    } else {
        for (int64_t r = r0 + threadIdx.x; r < r1; r += blockDim.x)
            f(prompt[r], generated[r], predicted[r], instance[r]);
    }
}

// Writes every live request, packed, into its tile's span of `records`.  Each block takes a
// contiguous chunk of the table: it counts its requests per tile in shared memory, reserves
// one span per touched tile with a single global atomic, then writes.  When the tile counts
// fit in shared memory every block scans them itself (no separate scan launch); block 0
// publishes the bases for the build kernel.
__global__ void __launch_bounds__(BIN_THREADS)
pre_bin_scatter(const int32_t* __restrict__ prompt, const int32_t* __restrict__ generated,
                const int32_t* __restrict__ predicted, const int32_t* __restrict__ instance, int64_t n,
                int I, int T, int n_tiles, const unsigned int* __restrict__ bin_count,
                unsigned int* __restrict__ bin_base, unsigned int* __restrict__ bin_cursor,
                unsigned long long* __restrict__ records, int* __restrict__ status) {
    extern __shared__ unsigned int sh_u32[];
    __shared__ unsigned int warp_tot[BIN_THREADS / 32];
    const bool use_sh = n_tiles <= PRE_SMEM_BINS;
    int64_t chunk = (n + gridDim.x - 1) / gridDim.x;
    chunk = (chunk + 3) & ~(int64_t)3;
    const int64_t r0 = (int64_t)blockIdx.x * chunk < n ? (int64_t)blockIdx.x * chunk : n;
    const int64_t r1 = r0 + chunk < n ? r0 + chunk : n;
    const bool vec = ((reinterpret_cast<uintptr_t>(prompt) | reinterpret_cast<uintptr_t>(generated) |
                       reinterpret_cast<uintptr_t>(predicted) | reinterpret_cast<uintptr_t>(instance)) & 15) == 0;
    bool any_bad = false;
    if (use_sh) {
        unsigned int* sh_bins = sh_u32;            // [n_tiles] histogram, then write cursor
        unsigned int* sh_base = sh_u32 + n_tiles;  // [n_tiles] exclusive scan of the global counts
        // ---- exclusive scan of the tile counts (each thread a contiguous run)
        const int per = (n_tiles + BIN_THREADS - 1) / BIN_THREADS;
        const int b0 = threadIdx.x * per;
        unsigned int local = 0;
        for (int k = 0; k < per; ++k) {
            const int i = b0 + k;
            if (i < n_tiles) { sh_bins[i] = 0; local += bin_count[i]; }
        }
        const int lane = threadIdx.x & 31, warp = threadIdx.x >> 5;
        unsigned int x = local;
        #pragma unroll
        for (int off = 1; off < 32; off <<= 1) {
            const unsigned int y = __shfl_up_sync(0xffffffffu, x, off);
            if (lane >= off) x += y;
        }
        if (lane == 31) warp_tot[warp] = x;
        __syncthreads();
        unsigned int run = x - local;
        for (int w = 0; w < warp; ++w) run += warp_tot[w];
        for (int k = 0; k < per; ++k) {
            const int i = b0 + k;
            if (i < n_tiles) {
                sh_base[i] = run;
                if (blockIdx.x == 0) bin_base[i] = run;
                run += bin_count[i];
            }
        }
        __syncthreads();
        // ---- pass A: this block's requests per tile
        for_each_request(prompt, generated, predicted, instance, r0, r1, vec,
                         [&](int32_t P, int32_t g, int32_t D, int32_t inst) {
                             const Packed p = pack_request(P, g, D, inst, I, T);
                             any_bad |= p.bad;
                             if (p.live) atomicAdd(&sh_bins[p.tile], 1u);
                         });
        __syncthreads();
        for (int i = threadIdx.x; i < n_tiles; i += BIN_THREADS) {
            const unsigned int c = sh_bins[i];
            if (c) sh_bins[i] = sh_base[i] + atomicAdd(&bin_cursor[i], c);
        }
        __syncthreads();
        // ---- pass B: write (the chunk is re-read, from L2)
        for_each_request(prompt, generated, predicted, instance, r0, r1, vec,
                         [&](int32_t P, int32_t g, int32_t D, int32_t inst) {
                             const Packed p = pack_request(P, g, D, inst, I, T);
                             if (p.live) records[atomicAdd(&sh_bins[p.tile], 1u)] = p.rec;
                         });
    } else {
        for_each_request(prompt, generated, predicted, instance, r0, r1, vec,
                         [&](int32_t P, int32_t g, int32_t D, int32_t inst) {
                             const Packed p = pack_request(P, g, D, inst, I, T);
                             any_bad |= p.bad;
                             if (p.live) records[bin_base[p.tile] + atomicAdd(&bin_cursor[p.tile], 1u)] = p.rec;
                         });
    }
    if (any_bad) atomicOr(status, PRE_ST_BADREQ);
}

// One block per tile of T instance rows.  Shared memory: count[cells], lo[cells], hi[cells]
// (uint32 each; the sum of B per cell is kept as lo + 2^32*hi so that only 32-bit shared
// atomics are needed), then per-row 64-bit words.
constexpr int CPT = 8;  // cells per thread and scan pass

__global__ void __launch_bounds__(TILE_THREADS, 2)
pre_tile_build(const unsigned long long* __restrict__ records, const unsigned int* __restrict__ bin_base,
               unsigned int* __restrict__ bin_cursor, unsigned int* __restrict__ bin_count, int I, int H, int T,
               int cells_pad, int64_t* __restrict__ curves, int64_t* __restrict__ current_d) {
    extern __shared__ __align__(16) unsigned char smem_raw[];
    uint32_t* cnt = reinterpret_cast<uint32_t*>(smem_raw);
    uint32_t* lo = cnt + cells_pad;
    uint32_t* hi = lo + cells_pad;
    unsigned long long* excess = reinterpret_cast<unsigned long long*>(hi + cells_pad);  // [T]
    unsigned long long* sum_n = excess + T;                                              // [T]
    unsigned long long* wt_s = sum_n + T;                                                // [2][TILE_WARPS]
    uint32_t* wt_n = reinterpret_cast<uint32_t*>(wt_s + 2 * TILE_WARPS);                 // [2][TILE_WARPS]

    const int tile = blockIdx.x;
    const int row0 = tile * T;
    const int rows = (I - row0) < T ? (I - row0) : T;
    const int tid = threadIdx.x, lane = tid & 31, warp = tid >> 5;

    {
        uint4* z = reinterpret_cast<uint4*>(cnt);
        const int nz = (3 * cells_pad) >> 2;
        for (int i = tid; i < nz; i += TILE_THREADS) z[i] = make_uint4(0, 0, 0, 0);
        for (int i = tid; i < 2 * T; i += TILE_THREADS) excess[i] = 0;
    }
    const unsigned int rec0 = bin_base[tile];
    const unsigned int rec1 = rec0 + bin_cursor[tile];
    __syncthreads();
    if (tid == 0) { bin_cursor[tile] = 0; bin_count[tile] = 0; }  // ready for the next call

    // ---- accumulate: one update per request at (row, R-1)
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

    // ---- suffix scan over the horizon, `team_warps` warps per row, CPT cells per thread
    int team_warps = 1;
    while (team_warps < TILE_WARPS && team_warps * 32 * CPT < H) team_warps <<= 1;
    const int teams = TILE_WARPS / team_warps;
    const int team = warp / team_warps, wteam = warp % team_warps;
    const int span = team_warps * 32 * CPT;
    const int passes = (H + span - 1) / span;
    const bool vec_sm = (H & 3) == 0;
    const bool vec_gl = (H & 1) == 0;
    int buf = 0;

    for (int rb = 0; rb < rows; rb += teams) {
        const int row = rb + team;
        const bool active = row < rows;
        uint32_t carry_n = 0;
        unsigned long long carry_s = 0, my_sum_n = 0;
        for (int p = passes - 1; p >= 0; --p) {
            const int j0 = p * span + (wteam * 32 + lane) * CPT;
            uint32_t n[CPT];
            unsigned long long s[CPT];
            #pragma unroll
            for (int k = 0; k < CPT; ++k) { n[k] = 0; s[k] = 0; }
            if (active && j0 < H) {
                const int c0 = row * H + j0;
                if (vec_sm) {
                    #pragma unroll
                    for (int v = 0; v < CPT / 4; ++v) {
                        if (j0 + 4 * v < H) {
                            const uint4 a = *reinterpret_cast<const uint4*>(cnt + c0 + 4 * v);
                            const uint4 b = *reinterpret_cast<const uint4*>(lo + c0 + 4 * v);
                            const uint4 c = *reinterpret_cast<const uint4*>(hi + c0 + 4 * v);
                            n[4 * v] = a.x; n[4 * v + 1] = a.y; n[4 * v + 2] = a.z; n[4 * v + 3] = a.w;
                            s[4 * v] = ((unsigned long long)c.x << 32) | b.x;
                            s[4 * v + 1] = ((unsigned long long)c.y << 32) | b.y;
                            s[4 * v + 2] = ((unsigned long long)c.z << 32) | b.z;
                            s[4 * v + 3] = ((unsigned long long)c.w << 32) | b.w;
                        }
                    }
                } else {
                    #pragma unroll
                    for (int k = 0; k < CPT; ++k) {
                        if (j0 + k < H) {
                            n[k] = cnt[c0 + k];
                            s[k] = ((unsigned long long)hi[c0 + k] << 32) | lo[c0 + k];
                        }
                    }
                }
            }
            uint32_t tn = 0;
            unsigned long long ts = 0;
            #pragma unroll
            for (int k = 0; k < CPT; ++k) { tn += n[k]; ts += s[k]; }
            // inclusive suffix over the lanes of this warp (higher lane = later steps)
            uint32_t xn = tn;
            unsigned long long xs = ts;
            #pragma unroll
            for (int off = 1; off < 32; off <<= 1) {
                const uint32_t yn = __shfl_down_sync(0xffffffffu, xn, off);
                const unsigned long long ys = __shfl_down_sync(0xffffffffu, xs, off);
                if (lane + off < 32) { xn += yn; xs += ys; }
            }
            uint32_t above_n = carry_n;
            unsigned long long above_s = carry_s;
            if (team_warps > 1) {
                if (lane == 0) { wt_n[buf * TILE_WARPS + warp] = xn; wt_s[buf * TILE_WARPS + warp] = xs; }
                __syncthreads();
                // suffix over the warps of the team, done redundantly by every warp
                uint32_t wn = 0;
                unsigned long long ws = 0;
                if (lane < team_warps) {
                    wn = wt_n[buf * TILE_WARPS + team * team_warps + lane];
                    ws = wt_s[buf * TILE_WARPS + team * team_warps + lane];
                }
                #pragma unroll
                for (int off = 1; off < TILE_WARPS; off <<= 1) {
                    const uint32_t yn = __shfl_down_sync(0xffffffffu, wn, off);
                    const unsigned long long ys = __shfl_down_sync(0xffffffffu, ws, off);
                    if (lane + off < 32) { wn += yn; ws += ys; }
                }
                above_n += __shfl_sync(0xffffffffu, wn, wteam + 1);  // lanes >= team_warps hold 0
                above_s += __shfl_sync(0xffffffffu, ws, wteam + 1);
                carry_n += __shfl_sync(0xffffffffu, wn, 0);
                carry_s += __shfl_sync(0xffffffffu, ws, 0);
                buf ^= 1;
            } else {
                carry_n += __shfl_sync(0xffffffffu, xn, 0);
                carry_s += __shfl_sync(0xffffffffu, xs, 0);
            }
            if (active && j0 < H) {
                uint32_t N = above_n + (xn - tn);
                unsigned long long A = above_s + (xs - ts);
                unsigned long long c[CPT];
                #pragma unroll
                for (int k = CPT - 1; k >= 0; --k) {
                    N += n[k]; A += s[k];
                    c[k] = A + (unsigned long long)(uint32_t)(j0 + k) * N;
                    if (j0 + k < H) my_sum_n += N;
                }
                int64_t* out = curves + ((size_t)(row0 + row) * H + j0);
                if (vec_gl) {
                    #pragma unroll
                    for (int k = 0; k < CPT; k += 2)
                        if (j0 + k < H) *reinterpret_cast<ulonglong2*>(out + k) = make_ulonglong2(c[k], c[k + 1]);
                } else {
                    #pragma unroll
                    for (int k = 0; k < CPT; ++k) if (j0 + k < H) out[k] = (int64_t)c[k];
                }
            }
        }
        // sum over j of N[j] = sum over requests of R (each request is counted on R steps)
        #pragma unroll
        for (int off = 16; off > 0; off >>= 1) my_sum_n += __shfl_xor_sync(0xffffffffu, my_sum_n, off);
        if (active && lane == 0 && my_sum_n) atomicAdd(&sum_n[row], my_sum_n);
    }
    __syncthreads();
    for (int i = tid; i < rows; i += TILE_THREADS) current_d[row0 + i] = (int64_t)(sum_n[i] + excess[i]);
}

size_t tile_cells_pad(int tile_rows, int horizon) {
    return (((size_t)tile_rows * horizon + 3) / 4) * 4 + 4;
}

}  // namespace

size_t pre_tile_smem_bytes(int tile_rows, int horizon) {
    return 3 * tile_cells_pad(tile_rows, horizon) * sizeof(uint32_t) + 2 * (size_t)tile_rows * 8 +
           2 * TILE_WARPS * 8 + 2 * TILE_WARPS * 4;
}

cudaError_t pre_launch_anticipate(pre_ctx* ctx, const int32_t* prompt, const int32_t* generated,
                                  const int32_t* predicted, const int32_t* instance, int64_t n,
                                  int64_t* curves, int64_t* current_d, cudaStream_t s) {
    const int I = ctx->cfg.n_instances, H = ctx->cfg.horizon, T = ctx->tile_rows, nt = ctx->n_tiles;
    const bool use_sh = nt <= PRE_SMEM_BINS;
    int grid = (int)((n + BIN_THREADS * 8 - 1) / (BIN_THREADS * 8));
    if (grid > 2 * ctx->n_sm) grid = 2 * ctx->n_sm;
    if (grid < 1) grid = 1;
    if (n > 0) {
        pre_bin_count<<<grid, BIN_THREADS, use_sh ? (size_t)nt * 4 : 0, s>>>(instance, n, I, T, nt, ctx->d_bin_count);
        if (!use_sh) pre_bin_scan<<<1, 1024, 0, s>>>(ctx->d_bin_count, nt, ctx->d_bin_base);
        pre_bin_scatter<<<grid, BIN_THREADS, use_sh ? (size_t)nt * 8 : 0, s>>>(
            prompt, generated, predicted, instance, n, I, T, nt, ctx->d_bin_count, ctx->d_bin_base,
            ctx->d_bin_cursor, ctx->d_records, ctx->d_status);
    }
    // With n == 0 the counts and cursors are all zero (every build clears them), so every
    // tile sees an empty span and writes zero rows.
    pre_tile_build<<<nt, TILE_THREADS, pre_tile_smem_bytes(T, H), s>>>(
        ctx->d_records, ctx->d_bin_base, ctx->d_bin_cursor, ctx->d_bin_count, I, H, T,
        (int)tile_cells_pad(T, H), curves, current_d);
    return cudaGetLastError();
}

cudaError_t pre_anticipate_configure(pre_ctx* ctx) {
    cudaError_t e = cudaFuncSetAttribute(pre_bin_scatter, cudaFuncAttributeMaxDynamicSharedMemorySize,
                                         PRE_SMEM_BINS * 8);
    if (e != cudaSuccess) return e;
    return cudaFuncSetAttribute(pre_tile_build, cudaFuncAttributeMaxDynamicSharedMemorySize,
                                (int)pre_tile_smem_bytes(ctx->tile_rows, ctx->cfg.horizon));
}

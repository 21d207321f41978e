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
// Pipeline (all on the caller's stream, no host synchronisation).  A tile is T
// consecutive instance rows, built by one block in shared memory.
//   1. pre_chunk_sort   each block takes a contiguous chunk of the table, packs every live
//                       request into 8 bytes, orders them by tile inside the chunk (counting
//                       sort in shared memory) and records where each tile starts in it
//   2. pre_tile_build   one block per tile: gathers the tile's requests from every chunk,
//                       accumulates (count, sum B) per (row, R-1) with shared-memory atomics,
//                       suffix-scans over the horizon and writes the rows
// No global atomics, no counting pass.  When there are more tiles than a block can count in
// shared memory, a slower path is taken: pre_bin_count, pre_bin_scan, pre_bin_scatter
// (global per-tile cursors) feed the same pre_tile_build.
#include "pre_common.cuh"

namespace {

constexpr int BIN_THREADS = 512;

// Slow path only.  Per-tile request counts.  Finished and malformed requests may be counted
// too: the counts only reserve room, the scatter pass decides what is written.
__global__ void __launch_bounds__(BIN_THREADS)
pre_bin_count(const int32_t* __restrict__ instance, int64_t n, int I, int T, unsigned int* __restrict__ bin_count) {
    const int64_t stride = (int64_t)gridDim.x * blockDim.x;
    for (int64_t r = (int64_t)blockIdx.x * blockDim.x + threadIdx.x; r < n; r += stride) {
        const int32_t v = instance[r];
        if ((uint32_t)v < (uint32_t)I) atomicAdd(&bin_count[v / T], 1u);
    }
}

// Slow path only.  One block: base[b] = sum of count[0..b).
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

// Slow path only: one global atomic per live request on its tile's cursor.
__global__ void __launch_bounds__(BIN_THREADS)
pre_bin_scatter(const int32_t* __restrict__ prompt, const int32_t* __restrict__ generated,
                const int32_t* __restrict__ predicted, const int32_t* __restrict__ instance, int64_t n,
                int I, int T, const unsigned int* __restrict__ bin_base, unsigned int* __restrict__ bin_cursor,
                unsigned long long* __restrict__ records, int* __restrict__ status) {
    int64_t chunk = (n + gridDim.x - 1) / gridDim.x;
    chunk = (chunk + 3) & ~(int64_t)3;
    const int64_t r0 = (int64_t)blockIdx.x * chunk < n ? (int64_t)blockIdx.x * chunk : n;
    const int64_t r1 = r0 + chunk < n ? r0 + chunk : n;
    const bool vec = ((reinterpret_cast<uintptr_t>(prompt) | reinterpret_cast<uintptr_t>(generated) |
                       reinterpret_cast<uintptr_t>(predicted) | reinterpret_cast<uintptr_t>(instance)) & 15) == 0;
    bool any_bad = false;
    for_each_request(prompt, generated, predicted, instance, r0, r1, vec,
                     [&](int32_t P, int32_t g, int32_t D, int32_t inst) {
                         const Packed p = pack_request(P, g, D, inst, I, T);
                         any_bad |= p.bad;
                         if (p.live) records[bin_base[p.tile] + atomicAdd(&bin_cursor[p.tile], 1u)] = p.rec;
                     });
    if (any_bad) atomicOr(status, PRE_ST_BADREQ);
}

// ---------------------------------------------------------------------------------------
// Fast path, step 1.  Block `ch` owns table rows [ch*chunk, (ch+1)*chunk) and the same span
// of `records`.  It writes its live requests there ordered by tile and stores, for every
// tile t, the offset of t's first record inside the span: chunk_off[t*NC + ch]
// (chunk_off[n_tiles*NC + ch] = number of live requests of the chunk).
constexpr int SORT_THREADS = 512;
constexpr int SORT_CHUNK = 6144;   // requests a block can stage in shared memory
constexpr int SORT_MAX_CHUNKS = 1024;

__global__ void __launch_bounds__(SORT_THREADS)
pre_chunk_sort(const int32_t* __restrict__ prompt, const int32_t* __restrict__ generated,
               const int32_t* __restrict__ predicted, const int32_t* __restrict__ instance, int64_t n,
               int I, int T, int n_tiles, int64_t chunk, int staged, unsigned long long* __restrict__ records,
               unsigned int* __restrict__ chunk_off, int* __restrict__ status) {
    extern __shared__ __align__(16) unsigned char sort_smem[];
    __shared__ unsigned int warp_tot[SORT_THREADS / 32];
    // layout: [stage: u64 x SORT_CHUNK][tile_of: u16 x SORT_CHUNK] (only when staged) [hist: u32 x (n_tiles+1)]
    unsigned long long* stage = reinterpret_cast<unsigned long long*>(sort_smem);
    unsigned short* tile_of = reinterpret_cast<unsigned short*>(stage + (staged ? SORT_CHUNK : 0));
    unsigned int* hist = reinterpret_cast<unsigned int*>(tile_of + (staged ? SORT_CHUNK : 0));

    const int ch = blockIdx.x, NC = gridDim.x;
    const int64_t r0 = (int64_t)ch * chunk < n ? (int64_t)ch * chunk : n;
    const int64_t r1 = r0 + chunk < n ? r0 + chunk : n;
    const bool vec = ((reinterpret_cast<uintptr_t>(prompt) | reinterpret_cast<uintptr_t>(generated) |
                       reinterpret_cast<uintptr_t>(predicted) | reinterpret_cast<uintptr_t>(instance)) & 15) == 0;
    const int tid = threadIdx.x, lane = tid & 31, warp = tid >> 5;
    bool any_bad = false;

    for (int i = tid; i <= n_tiles; i += SORT_THREADS) hist[i] = 0;
    __syncthreads();

    // ---- pass A: pack, count per tile (and keep the packed request when it fits)
    if (staged) {
        // one request per (thread, slot): slot li = r - r0 < SORT_CHUNK
        auto take = [&](int64_t r, int32_t P, int32_t g, int32_t D, int32_t inst) {
            const Packed p = pack_request(P, g, D, inst, I, T);
            any_bad |= p.bad;
            const int li = (int)(r - r0);
            stage[li] = p.rec;
            tile_of[li] = p.live ? (unsigned short)p.tile : (unsigned short)0xFFFF;
            if (p.live) atomicAdd(&hist[p.tile], 1u);
        };
        if (vec) {
            const int64_t q1 = r1 >> 2;
            for (int64_t q = (r0 >> 2) + tid; q < q1; q += SORT_THREADS) {
                const int4 p = __ldg(reinterpret_cast<const int4*>(prompt) + q);
                const int4 g = __ldg(reinterpret_cast<const int4*>(generated) + q);
                const int4 d = __ldg(reinterpret_cast<const int4*>(predicted) + q);
                const int4 i = __ldg(reinterpret_cast<const int4*>(instance) + q);
                const int64_t r = q << 2;
                take(r, p.x, g.x, d.x, i.x); take(r + 1, p.y, g.y, d.y, i.y);
                take(r + 2, p.z, g.z, d.z, i.z); take(r + 3, p.w, g.w, d.w, i.w);
            }
            for (int64_t r = (q1 << 2) + tid; r < r1; r += SORT_THREADS)
                if (r >= r0) take(r, prompt[r], generated[r], predicted[r], instance[r]);
        } else {
            for (int64_t r = r0 + tid; r < r1; r += SORT_THREADS)
                take(r, prompt[r], generated[r], predicted[r], instance[r]);
        }
    } else {
        for_each_request(prompt, generated, predicted, instance, r0, r1, vec,
                         [&](int32_t P, int32_t g, int32_t D, int32_t inst) {
                             const Packed p = pack_request(P, g, D, inst, I, T);
                             any_bad |= p.bad;
                             if (p.live) atomicAdd(&hist[p.tile], 1u);
                         });
    }
    __syncthreads();

    // ---- exclusive scan of the per-tile counts, in place (each thread a contiguous run)
    {
        const int per = (n_tiles + SORT_THREADS) / SORT_THREADS;  // covers n_tiles + 1 entries
        const int b0 = tid * per;
        unsigned int local = 0;
        for (int k = 0; k < per; ++k) if (b0 + k <= n_tiles) local += hist[b0 + k];
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
            if (i <= n_tiles) {
                const unsigned int c = hist[i];
                hist[i] = run;                              // becomes the tile's write cursor
                chunk_off[(size_t)i * NC + ch] = run;       // entry n_tiles receives the total
                run += c;
            }
        }
    }
    __syncthreads();

    // ---- pass B: place
    unsigned long long* out = records + r0;
    if (staged) {
        const int cnt = (int)(r1 - r0);
        for (int l0 = tid; l0 < cnt; l0 += 4 * SORT_THREADS) {   // four independent cursor bumps in flight
            unsigned int t[4], pos[4];
            #pragma unroll
            for (int u = 0; u < 4; ++u) {
                const int li = l0 + u * SORT_THREADS;
                t[u] = li < cnt ? tile_of[li] : 0xFFFFu;
            }
            #pragma unroll
            for (int u = 0; u < 4; ++u) pos[u] = t[u] != 0xFFFFu ? atomicAdd(&hist[t[u]], 1u) : 0u;
            #pragma unroll
            for (int u = 0; u < 4; ++u)
                if (t[u] != 0xFFFFu) out[pos[u]] = stage[l0 + u * SORT_THREADS];
        }
    } else {
        for_each_request(prompt, generated, predicted, instance, r0, r1, vec,
                         [&](int32_t P, int32_t g, int32_t D, int32_t inst) {
                             const Packed p = pack_request(P, g, D, inst, I, T);
                             if (p.live) out[atomicAdd(&hist[p.tile], 1u)] = p.rec;
                         });
    }
    if (any_bad) atomicOr(status, PRE_ST_BADREQ);
}

// ---------------------------------------------------------------------------------------
// Step 2.  One block per tile.  Shared memory holds, per cell (row, j) of the tile, one
// 64-bit word {low: sum of B mod 2^32, high: count} plus a rarely used 32-bit carry word
// (so that only 32-bit shared atomics are needed).  Rows are padded to a multiple of RUN
// cells; a run of RUN consecutive cells is scanned by one thread, and every run is
// followed by 16 bytes of padding so that the threads' 16-byte loads fall in different banks.
constexpr int TILE_THREADS = 256;
constexpr int TILE_WARPS = TILE_THREADS / 32;
constexpr int RUN = 16;

__device__ __forceinline__ int cell_slot(int c) { return c + ((c >> 4) << 1); }  // index in 8-byte words

struct TileShape { int hp, rpr, cpw; };  // padded row length, runs per row, 32-run chunks per row

__host__ __device__ inline TileShape tile_shape(int H) {
    TileShape t;
    t.rpr = (H + RUN - 1) / RUN;
    t.hp = t.rpr * RUN;
    t.cpw = (t.rpr + 31) / 32;
    return t;
}

__global__ void __launch_bounds__(TILE_THREADS, 3)
pre_tile_build(const unsigned long long* __restrict__ records,
               const unsigned int* __restrict__ chunk_off, int NC, int64_t chunk,          // fast path
               const unsigned int* __restrict__ bin_base, unsigned int* __restrict__ bin_cursor,
               unsigned int* __restrict__ bin_count,                                        // slow path
               int I, int H, int T, int64_t* __restrict__ curves, int64_t* __restrict__ current_d) {
    extern __shared__ __align__(16) unsigned char smem_raw[];
    const TileShape sh = tile_shape(H);
    const int cells = T * sh.hp;            // padded cells of a full tile
    const int n_runs_max = T * sh.rpr;
    unsigned long long* cl = reinterpret_cast<unsigned long long*>(smem_raw);        // [cells * 9/8]
    unsigned long long* run_s = cl + (cells + (cells >> 3));                          // [n_runs_max]
    unsigned long long* run_w = run_s + n_runs_max;                                   // [n_runs_max]
    unsigned long long* chk_s = run_w + n_runs_max;                                   // [T * cpw]
    unsigned long long* excess = chk_s + T * sh.cpw;                                  // [T]
    unsigned long long* sum_n = excess + T;                                           // [T]
    uint32_t* run_n = reinterpret_cast<uint32_t*>(sum_n + T);                         // [n_runs_max]
    uint32_t* chk_n = run_n + n_runs_max;                                             // [T * cpw]
    uint32_t* hi = chk_n + T * sh.cpw;                                                // [cells]
    __shared__ int any_hi;

    const int tile = blockIdx.x;
    const int row0 = tile * T;
    const int rows = (I - row0) < T ? (I - row0) : T;
    const int n_runs = rows * sh.rpr;
    const int tid = threadIdx.x, lane = tid & 31, warp = tid >> 5;

    {   // clear the cell words, the carry words and the per-row sums
        uint4* z = reinterpret_cast<uint4*>(cl);
        const int nz = (cells + (cells >> 3)) >> 1;
        for (int i = tid; i < nz; i += TILE_THREADS) z[i] = make_uint4(0, 0, 0, 0);
        for (int i = tid; i < cells; i += TILE_THREADS) hi[i] = 0;
        for (int i = tid; i < 2 * T; i += TILE_THREADS) excess[i] = 0;
        if (tid == 0) any_hi = 0;
    }
    __syncthreads();

    // ---- accumulate: one update per request at (row, R-1)
    auto add_record = [&](unsigned long long rec) {
        const uint32_t rem = (uint32_t)(rec & PRE_FIELD_MAX);
        const uint32_t B = (uint32_t)((rec >> PRE_FIELD_BITS) & PRE_FIELD_MAX);
        const int local = (int)(rec >> (2 * PRE_FIELD_BITS));
        const uint32_t R = rem < (uint32_t)H ? rem : (uint32_t)H;
        const int c = local * sh.hp + (int)R - 1;
        uint32_t* w = reinterpret_cast<uint32_t*>(cl + cell_slot(c));
        atomicAdd(w + 1, 1u);
        const uint32_t old = atomicAdd(w, B);
        if (old + B < old) { atomicAdd(&hi[c], 1u); any_hi = 1; }  // exactly one thread sees each wrap
        if (rem > (uint32_t)H) atomicAdd(&excess[local], (unsigned long long)(rem - (uint32_t)H));
    };
    if (chunk_off != nullptr) {
        const unsigned int* o0 = chunk_off + (size_t)tile * NC;
        const unsigned int* o1 = o0 + NC;
        // A tile has a few records per chunk (about n / (tiles * chunks)): take up to four with
        // independent loads, then whatever is left one by one.
        for (int ch = tid; ch < NC; ch += TILE_THREADS) {
            const unsigned int a = o0[ch], b = o1[ch];
            const unsigned long long* src = records + (size_t)ch * chunk + a;
            const unsigned int len = b - a;
            unsigned long long rec[4];
            #pragma unroll
            for (int u = 0; u < 4; ++u) rec[u] = (unsigned int)u < len ? src[u] : 0ull;
            #pragma unroll
            for (int u = 0; u < 4; ++u) if ((unsigned int)u < len) add_record(rec[u]);
            for (unsigned int r = 4; r < len; ++r) add_record(src[r]);
        }
    } else {
        const unsigned int rec0 = bin_base[tile];
        const unsigned int rec1 = rec0 + bin_cursor[tile];
        for (unsigned int r = rec0 + tid; r < rec1; r += TILE_THREADS) add_record(records[r]);
    }
    __syncthreads();
    if (chunk_off == nullptr && tid == 0) { bin_cursor[tile] = 0; bin_count[tile] = 0; }  // for the next call
    const bool with_hi = any_hi != 0;

    // ---- phase 1: totals of every run
    for (int run = tid; run < n_runs; run += TILE_THREADS) {
        const ulonglong2* src = reinterpret_cast<const ulonglong2*>(cl + run * (RUN + 2));
        const int j0 = (run % sh.rpr) * RUN;
        uint32_t tn = 0;
        unsigned long long ts = 0, tw = 0;
        #pragma unroll
        for (int i = 0; i < RUN / 2; ++i) {
            const ulonglong2 v = src[i];
            const uint32_t n0 = (uint32_t)(v.x >> 32), n1 = (uint32_t)(v.y >> 32);
            tn += n0 + n1;
            ts += (v.x & 0xffffffffull) + (v.y & 0xffffffffull);
            tw += (unsigned long long)n0 * (uint32_t)(j0 + 2 * i + 1) + (unsigned long long)n1 * (uint32_t)(j0 + 2 * i + 2);
        }
        if (with_hi) {
            for (int k = 0; k < RUN; ++k) ts += (unsigned long long)hi[run * RUN + k] << 32;
        }
        run_n[run] = tn; run_s[run] = ts; run_w[run] = tw;
    }
    __syncthreads();

    // ---- phase 2: suffix over the runs of each row, 32 runs per warp task
    for (int task = warp; task < rows * sh.cpw; task += TILE_WARPS) {
        const int row = task / sh.cpw, k = task - row * sh.cpw;
        const int q = k * 32 + lane;
        const bool valid = q < sh.rpr;
        const int run = row * sh.rpr + q;
        const uint32_t n = valid ? run_n[run] : 0u;
        const unsigned long long s = valid ? run_s[run] : 0ull;
        unsigned long long w = valid ? run_w[run] : 0ull;
        uint32_t xn = n;
        unsigned long long xs = s;
        #pragma unroll
        for (int off = 1; off < 32; off <<= 1) {
            const uint32_t yn = __shfl_down_sync(0xffffffffu, xn, off);
            const unsigned long long ys = __shfl_down_sync(0xffffffffu, xs, off);
            if (lane + off < 32) { xn += yn; xs += ys; }
            w += __shfl_xor_sync(0xffffffffu, w, off);
        }
        if (valid) { run_n[run] = xn - n; run_s[run] = xs - s; }  // what lies above, inside the chunk
        if (lane == 0) {
            chk_n[task] = xn; chk_s[task] = xs;
            // sum over j of N[j] = sum over requests of R: each request is counted on R steps
            if (w) atomicAdd(&sum_n[row], w);
        }
    }
    __syncthreads();

    // ---- phase 3: every run from its last cell down; results overwrite the cell words
    for (int run = tid; run < n_runs; run += TILE_THREADS) {
        const int row = run / sh.rpr, q = run - row * sh.rpr;
        const int k = q >> 5;
        uint32_t N = run_n[run];
        unsigned long long A = run_s[run];
        for (int kk = k + 1; kk < sh.cpw; ++kk) { N += chk_n[row * sh.cpw + kk]; A += chk_s[row * sh.cpw + kk]; }
        ulonglong2* io = reinterpret_cast<ulonglong2*>(cl + run * (RUN + 2));
        const int j0 = q * RUN;
        #pragma unroll
        for (int i = RUN / 2 - 1; i >= 0; --i) {
            const ulonglong2 v = io[i];
            unsigned long long s1 = v.y & 0xffffffffull, s0 = v.x & 0xffffffffull;
            if (with_hi) {
                s1 |= (unsigned long long)hi[run * RUN + 2 * i + 1] << 32;
                s0 |= (unsigned long long)hi[run * RUN + 2 * i] << 32;
            }
            ulonglong2 o;
            N += (uint32_t)(v.y >> 32); A += s1;
            o.y = A + (unsigned long long)(uint32_t)(j0 + 2 * i + 1) * N;
            N += (uint32_t)(v.x >> 32); A += s0;
            o.x = A + (unsigned long long)(uint32_t)(j0 + 2 * i) * N;
            io[i] = o;
        }
    }
    __syncthreads();

    // ---- phase 4: copy the rows out with consecutive lanes on consecutive 16 bytes
    {
        const int half = sh.hp >> 1;  // cell pairs per padded row
        const int total = rows * half;
        const bool vec_gl = (H & 1) == 0;
        const int shift = (half & (half - 1)) == 0 ? 31 - __clz(half) : -1;  // log2 when a power of two
        for (int p = tid; p < total; p += TILE_THREADS) {
            const int row = shift >= 0 ? p >> shift : p / half;
            const int j = (p - row * half) << 1;
            if (j < H) {
                const int c = row * sh.hp + j;
                const ulonglong2 v = *reinterpret_cast<const ulonglong2*>(cl + cell_slot(c));
                int64_t* dst = curves + ((size_t)(row0 + row) * H + j);
                if (vec_gl) {
                    *reinterpret_cast<ulonglong2*>(dst) = v;
                } else {
                    dst[0] = (int64_t)v.x;
                    if (j + 1 < H) dst[1] = (int64_t)v.y;
                }
            }
        }
    }
    for (int i = tid; i < rows; i += TILE_THREADS) current_d[row0 + i] = (int64_t)(sum_n[i] + excess[i]);
}

}  // namespace

size_t pre_tile_smem_bytes(int tile_rows, int horizon) {
    const TileShape sh = tile_shape(horizon);
    const size_t cells = (size_t)tile_rows * sh.hp;
    const size_t runs = (size_t)tile_rows * sh.rpr;
    const size_t chunks = (size_t)tile_rows * sh.cpw;
    return (cells + cells / 8) * 8 + runs * (8 + 8 + 4) + chunks * (8 + 4) + (size_t)tile_rows * 16 + cells * 4;
}

int pre_tile_rows_for(int n_instances, int horizon, int n_sm) {
    const TileShape sh = tile_shape(horizon);
    int t = 4096 / sh.hp;                       // about 4096 cells (16 per thread) per tile
    if (t < 1) t = 1;
    if (t > PRE_MAX_TILE_ROWS) t = PRE_MAX_TILE_ROWS;
    int by_grid = n_instances / (8 * n_sm);     // but keep the grid at several blocks per SM
    if (by_grid < 1) by_grid = 1;
    return t < by_grid ? t : by_grid;
}

// How the table is cut into chunks: enough chunks that each fits the staging buffer, and, when
// the table allows it, as many as the GPU runs blocks at once (`slots`), so that the sort is a
// single wave; never more than `max_chunks` (the width of the offset table).
static void sort_geometry(int64_t n, int slots, int max_chunks, int* n_chunks, int64_t* chunk, int* staged) {
    int64_t nc = (n + SORT_CHUNK - 1) / SORT_CHUNK;
    int64_t wave = (n + 1023) / 1024;            // but no chunk below ~1024 requests
    if (wave > slots) wave = slots;
    if (nc < wave) nc = wave;
    if (nc > max_chunks) nc = max_chunks;
    if (nc < 1) nc = 1;
    int64_t c = (n + nc - 1) / nc;
    c = (c + 3) & ~(int64_t)3;
    if (c < 4) c = 4;
    *n_chunks = (int)nc;
    *chunk = c;
    *staged = c <= SORT_CHUNK;
}

static size_t sort_smem_bytes(int n_tiles, int staged) {
    return (staged ? (size_t)SORT_CHUNK * (8 + 2) : 0) + ((size_t)n_tiles + 1) * 4;
}

size_t pre_chunk_off_words(int n_tiles) {
    return n_tiles <= PRE_SMEM_BINS ? ((size_t)n_tiles + 1) * SORT_MAX_CHUNKS : 0;
}

cudaError_t pre_launch_anticipate(pre_ctx* ctx, const int32_t* prompt, const int32_t* generated,
                                  const int32_t* predicted, const int32_t* instance, int64_t n,
                                  int64_t* curves, int64_t* current_d, cudaStream_t s) {
    const int I = ctx->cfg.n_instances, H = ctx->cfg.horizon, T = ctx->tile_rows, nt = ctx->n_tiles;
    const size_t tile_smem = pre_tile_smem_bytes(T, H);
    if (nt <= PRE_SMEM_BINS) {
        int nc = 1, staged = 1;
        int64_t chunk = 4;
        sort_geometry(n, 3 * ctx->n_sm, SORT_MAX_CHUNKS, &nc, &chunk, &staged);
        // With n == 0 the single chunk is empty: its offsets are all zero and every tile writes zero rows.
        pre_chunk_sort<<<nc, SORT_THREADS, sort_smem_bytes(nt, staged), s>>>(
            prompt, generated, predicted, instance, n, I, T, nt, chunk, staged, ctx->d_records, ctx->d_chunk_off,
            ctx->d_status);
        pre_tile_build<<<nt, TILE_THREADS, tile_smem, s>>>(ctx->d_records, ctx->d_chunk_off, nc, chunk, nullptr,
                                                         nullptr, nullptr, I, H, T, curves, current_d);
    } else {
        int grid = (int)((n + BIN_THREADS * 8 - 1) / (BIN_THREADS * 8));
        if (grid > 2 * ctx->n_sm) grid = 2 * ctx->n_sm;
        if (grid < 1) grid = 1;
        if (n > 0) {
            pre_bin_count<<<grid, BIN_THREADS, 0, s>>>(instance, n, I, T, ctx->d_bin_count);
            pre_bin_scan<<<1, 1024, 0, s>>>(ctx->d_bin_count, nt, ctx->d_bin_base);
            pre_bin_scatter<<<grid, BIN_THREADS, 0, s>>>(prompt, generated, predicted, instance, n, I, T,
                                                       ctx->d_bin_base, ctx->d_bin_cursor, ctx->d_records,
                                                       ctx->d_status);
        }
        // With n == 0 the cursors are zero (every build clears them): every tile sees an empty span.
        pre_tile_build<<<nt, TILE_THREADS, tile_smem, s>>>(ctx->d_records, nullptr, 0, 0, ctx->d_bin_base,
                                                         ctx->d_bin_cursor, ctx->d_bin_count, I, H, T, curves,
                                                         current_d);
    }
    return cudaGetLastError();
}

cudaError_t pre_anticipate_configure(pre_ctx* ctx) {
    // The limit is a property of the kernel, shared by every context of the process: always
    // raise it to the device maximum, so that contexts of different shapes do not undo each other.
    int optin = 0;
    cudaError_t e = cudaDeviceGetAttribute(&optin, cudaDevAttrMaxSharedMemoryPerBlockOptin, ctx->device);
    if (e != cudaSuccess) return e;
    cudaFuncAttributes attr;
    e = cudaFuncGetAttributes(&attr, pre_chunk_sort);
    if (e != cudaSuccess) return e;
    e = cudaFuncSetAttribute(pre_chunk_sort, cudaFuncAttributeMaxDynamicSharedMemorySize,
                             optin - (int)attr.sharedSizeBytes);
    if (e != cudaSuccess) return e;
    e = cudaFuncGetAttributes(&attr, pre_tile_build);
    if (e != cudaSuccess) return e;
    return cudaFuncSetAttribute(pre_tile_build, cudaFuncAttributeMaxDynamicSharedMemorySize,
                                optin - (int)attr.sharedSizeBytes);
}

// ---------------------------------------------------------------------------------------
// pre_anticipate_static: the same build for callers that must not allocate.
//
// Its scratch (the packed, tile-ordered requests and the per-chunk tile offsets) lives in
// one array that is part of the library image: every GPU that loads the library holds these
// bytes until the process exits.  The sizes below are therefore deliberately modest.
constexpr int PRE_STATIC_MAX_REQUESTS = 262144;   // table rows one call may cover
constexpr int PRE_STATIC_MAX_TILES = 2048;        // build tiles one call may need
constexpr int PRE_STATIC_MAX_CHUNKS = 64;          // chunks of at most 4,096 requests
constexpr size_t PRE_STATIC_STATUS_BYTES = 256;
constexpr size_t PRE_STATIC_OFF_BYTES = (size_t)(PRE_STATIC_MAX_TILES + 1) * PRE_STATIC_MAX_CHUNKS * sizeof(unsigned int);
constexpr size_t PRE_STATIC_REC_BYTES = (size_t)PRE_STATIC_MAX_REQUESTS * sizeof(unsigned long long);
constexpr size_t PRE_STATIC_BYTES = PRE_STATIC_STATUS_BYTES + ((PRE_STATIC_OFF_BYTES + 255) & ~(size_t)255) + PRE_STATIC_REC_BYTES;

static __device__ __align__(256) unsigned char pre_static_scratch[PRE_STATIC_BYTES];

namespace {

constexpr int PRE_STATIC_MAX_DEVICES = 64;

struct StaticSetup {
    bool ready;
    unsigned char* base;   // device address of pre_static_scratch on this device
    int n_sm;
    int smem_optin;
};
StaticSetup g_static_setup[PRE_STATIC_MAX_DEVICES];

// Once per device, with that device current.  In host code `pre_static_scratch` is only a
// handle of the symbol, not an address the GPU can use: the device address has to be asked for.
cudaError_t static_setup(int device, StaticSetup** out) {
    StaticSetup* st = &g_static_setup[device];
    if (!st->ready) {
        void* p = nullptr;
        cudaError_t e = cudaGetSymbolAddress(&p, pre_static_scratch);
        if (e != cudaSuccess) return e;
        e = cudaDeviceGetAttribute(&st->n_sm, cudaDevAttrMultiProcessorCount, device);
        if (e != cudaSuccess) return e;
        e = cudaDeviceGetAttribute(&st->smem_optin, cudaDevAttrMaxSharedMemoryPerBlockOptin, device);
        if (e != cudaSuccess) return e;
        cudaFuncAttributes attr;
        e = cudaFuncGetAttributes(&attr, pre_chunk_sort);
        if (e != cudaSuccess) return e;
        e = cudaFuncSetAttribute(pre_chunk_sort, cudaFuncAttributeMaxDynamicSharedMemorySize,
                                 st->smem_optin - (int)attr.sharedSizeBytes);
        if (e != cudaSuccess) return e;
        e = cudaFuncGetAttributes(&attr, pre_tile_build);
        if (e != cudaSuccess) return e;
        e = cudaFuncSetAttribute(pre_tile_build, cudaFuncAttributeMaxDynamicSharedMemorySize,
                                 st->smem_optin - (int)attr.sharedSizeBytes);
        if (e != cudaSuccess) return e;
        st->base = static_cast<unsigned char*>(p);
        st->ready = true;
    }
    *out = st;
    return cudaSuccess;
}

}  // namespace

extern "C" int pre_anticipate_static(int32_t n_instances, int32_t horizon, const int32_t* d_prompt,
                                     const int32_t* d_generated, const int32_t* d_predicted,
                                     const int32_t* d_instance, int64_t n_requests, int64_t* d_curves,
                                     int64_t* d_current_d, int32_t* d_flags, void* stream) {
    if (n_instances < 1 || horizon < 1 || horizon > PRE_MAX_HORIZON) return PRE_EINVAL;
    if (n_requests < 0 || !d_curves || !d_current_d) return PRE_EINVAL;
    if (n_requests > 0 && (!d_prompt || !d_generated || !d_predicted || !d_instance)) return PRE_EINVAL;
    if ((reinterpret_cast<uintptr_t>(d_curves) & 15) || (reinterpret_cast<uintptr_t>(d_current_d) & 7) ||
        (reinterpret_cast<uintptr_t>(d_flags) & 3) || (reinterpret_cast<uintptr_t>(d_prompt) & 3) ||
        (reinterpret_cast<uintptr_t>(d_generated) & 3) || (reinterpret_cast<uintptr_t>(d_predicted) & 3) ||
        (reinterpret_cast<uintptr_t>(d_instance) & 3))
        return PRE_EINVAL;
    if (n_requests > PRE_STATIC_MAX_REQUESTS) return PRE_ESIZE;

    int device = 0;
    if (cudaGetDevice(&device) != cudaSuccess) return PRE_ECUDA;
    if (device < 0 || device >= PRE_STATIC_MAX_DEVICES) return PRE_ESIZE;
    StaticSetup* st = nullptr;
    if (static_setup(device, &st) != cudaSuccess) return PRE_ECUDA;

    const int T = pre_tile_rows_for(n_instances, horizon, st->n_sm);
    const int n_tiles = (n_instances + T - 1) / T;
    if (n_tiles > PRE_STATIC_MAX_TILES) return PRE_ESIZE;
    const size_t tile_smem = pre_tile_smem_bytes(T, horizon);
    if (tile_smem > (size_t)st->smem_optin) return PRE_EINVAL;

    int nc = 1, staged = 1;
    int64_t chunk = 4;
    sort_geometry(n_requests, 3 * st->n_sm, PRE_STATIC_MAX_CHUNKS, &nc, &chunk, &staged);  // staged: chunk <= 4096

    int* status = d_flags ? d_flags : reinterpret_cast<int*>(st->base);
    unsigned int* chunk_off = reinterpret_cast<unsigned int*>(st->base + PRE_STATIC_STATUS_BYTES);
    unsigned long long* records = reinterpret_cast<unsigned long long*>(
        st->base + PRE_STATIC_STATUS_BYTES + ((PRE_STATIC_OFF_BYTES + 255) & ~(size_t)255));
    cudaStream_t s = static_cast<cudaStream_t>(stream);
    // Nothing in the scratch has to start at zero: pre_chunk_sort writes every offset that
    // pre_tile_build reads, and a record is read only where an offset says one was written.
    pre_chunk_sort<<<nc, SORT_THREADS, sort_smem_bytes(n_tiles, staged), s>>>(
        d_prompt, d_generated, d_predicted, d_instance, n_requests, n_instances, T, n_tiles, chunk, staged, records,
        chunk_off, status);
    pre_tile_build<<<n_tiles, TILE_THREADS, tile_smem, s>>>(records, chunk_off, nc, chunk, nullptr, nullptr, nullptr,
                                                          n_instances, horizon, T, d_curves, d_current_d);
    return cudaGetLastError() == cudaSuccess ? PRE_OK : PRE_ECUDA;
}

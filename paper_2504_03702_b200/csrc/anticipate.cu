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
// consecutive instance rows (T a power of two), built by one block in shared memory.
//   1. pre_chunk_sort   each block takes a contiguous chunk of the table and turns every live
//                       request into an 8-byte record {where its update goes inside the tile's
//                       shared memory, B}; records are ordered by tile inside the chunk (the
//                       rank of a request is what its counting atomic returns) and the block
//                       records where each tile starts in the chunk
//   2. pre_tile_build   one block per tile: gathers the tile's records from every chunk,
//                       accumulates (count, sum B) per (row, R-1) with shared-memory atomics,
//                       suffix-scans over the horizon in registers and writes the rows
// No counting pass over the table.  When there are more tiles than a block can count in
// shared memory, or more chunks than the offset table is wide, a slower path is taken:
// pre_bin_count, pre_bin_scan, pre_bin_scatter (global per-tile cursors) feed the same
// pre_tile_build.
//
// The part of a request's remaining length that lies beyond the window, (D - g - H)+, only
// matters for current_d; the first pass adds it to a per-instance scratch array (a global
// reduction, a few percent of the requests), the tile kernel adds it in and clears it again.
#include "build_tile.cuh"

namespace {

constexpr int BIN_THREADS = 512;

// Slow path only.  Per-tile request counts.  Finished and malformed requests may be counted
// too: the counts only reserve room, the scatter pass decides what is written.
__global__ void __launch_bounds__(BIN_THREADS)
pre_bin_count(const int32_t* __restrict__ instance, int64_t n, int I, int tile_shift,
              unsigned int* __restrict__ bin_count) {
    const int64_t stride = (int64_t)gridDim.x * blockDim.x;
    for (int64_t r = (int64_t)blockIdx.x * blockDim.x + threadIdx.x; r < n; r += stride) {
        const int32_t v = instance[r];
        if ((uint32_t)v < (uint32_t)I) atomicAdd(&bin_count[v >> tile_shift], 1u);
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

// Slow path only: one global atomic per live request on its tile's cursor.
__global__ void __launch_bounds__(BIN_THREADS)
pre_bin_scatter(const int32_t* __restrict__ prompt, const int32_t* __restrict__ generated,
                const int32_t* __restrict__ predicted, const int32_t* __restrict__ instance, int64_t n,
                const BuildShape sh, const unsigned int* __restrict__ bin_base,
                unsigned int* __restrict__ bin_cursor, unsigned long long* __restrict__ records,
                unsigned long long* __restrict__ excess, int* __restrict__ status) {
    const int64_t stride = (int64_t)gridDim.x * blockDim.x;
    bool any_bad = false;
    for (int64_t r = (int64_t)blockIdx.x * blockDim.x + threadIdx.x; r < n; r += stride) {
        const int32_t inst = instance[r];
        const Packed p = pack_request(prompt[r], generated[r], predicted[r], inst, sh);
        any_bad |= p.bad;
        if (p.live) {
            records[bin_base[p.tile] + atomicAdd(&bin_cursor[p.tile], 1u)] = p.rec;
            if (p.excess) atomicAdd(&excess[inst], (unsigned long long)p.excess);
        }
    }
    if (any_bad) atomicOr(status, PRE_ST_BADREQ);
}

// ---------------------------------------------------------------------------------------
// Fast path, step 1.  Block `ch` owns table rows [ch*chunk, (ch+1)*chunk), chunk <= SORT_CHUNK,
// and the same span of `records`.  Every thread keeps its (at most eight) records in
// registers: all table loads are issued before the first is used, the per-tile rank of a
// request is the value its counting atomic returns, and after one scan of the per-tile counts
// each record is stored at (tile start + rank).  The chunk's records end up ordered by tile;
// chunk_off[ch*n_tiles + t] = {start of tile t inside the span : 16 | number of its records : 16}
// (a chunk has at most 4,096 rows, so both fit); chunk_max[ch] = largest B of the chunk.
constexpr int SORT_THREADS = 512;
constexpr int SORT_QUADS = 2;                                  // 16-byte loads per thread and array
constexpr int SORT_SLOTS = 4 * SORT_QUADS;                     // requests a thread holds
constexpr int SORT_CHUNK = SORT_THREADS * SORT_SLOTS;          // 4,096
constexpr int SORT_MAX_CHUNKS = 4096;                          // widest offset table (16.7 M requests)

__global__ void __launch_bounds__(SORT_THREADS, 2)
pre_chunk_sort(const int32_t* __restrict__ prompt, const int32_t* __restrict__ generated,
               const int32_t* __restrict__ predicted, const int32_t* __restrict__ instance, int64_t n,
               const BuildShape sh, int64_t chunk, unsigned long long* __restrict__ records,
               unsigned int* __restrict__ chunk_off, unsigned int* __restrict__ chunk_max,
               unsigned long long* __restrict__ excess, int* __restrict__ status) {
    extern __shared__ __align__(16) unsigned int hist[];    // [n_tiles + 1], rounded up to whole 16-byte groups;
                                                             // then the chunk's records in tile order
    __shared__ unsigned int warp_tot[SORT_THREADS / 32];
    __shared__ unsigned int block_max;

    const int n_tiles = sh.n_tiles;
    const int ch = blockIdx.x;
    const int64_t r0 = (int64_t)ch * chunk < n ? (int64_t)ch * chunk : n;
    const int64_t r1 = r0 + chunk < n ? r0 + chunk : n;
    const int cnt = (int)(r1 - r0);
    const bool vec = ((reinterpret_cast<uintptr_t>(prompt) | reinterpret_cast<uintptr_t>(generated) |
                       reinterpret_cast<uintptr_t>(predicted) | reinterpret_cast<uintptr_t>(instance)) & 15) == 0;
    const int tid = threadIdx.x, lane = tid & 31, warp = tid >> 5;

    // ---- load: slot u of this thread is table row r0 + (u/4 * SORT_THREADS + tid) * 4 + u%4
    int32_t P[SORT_SLOTS], G[SORT_SLOTS], D[SORT_SLOTS], N[SORT_SLOTS];
    unsigned int present = 0;
    if (vec && (SORT_QUADS - 1) * SORT_THREADS * 4 + tid * 4 + 4 <= cnt) {   // r0 is a multiple of 4
        #pragma unroll
        for (int h = 0; h < SORT_QUADS; ++h) {
            const int64_t q = (r0 >> 2) + h * SORT_THREADS + tid;
            const int4 p = __ldg(reinterpret_cast<const int4*>(prompt) + q);
            const int4 g = __ldg(reinterpret_cast<const int4*>(generated) + q);
            const int4 d = __ldg(reinterpret_cast<const int4*>(predicted) + q);
            const int4 i = __ldg(reinterpret_cast<const int4*>(instance) + q);
            P[4 * h] = p.x; P[4 * h + 1] = p.y; P[4 * h + 2] = p.z; P[4 * h + 3] = p.w;
            G[4 * h] = g.x; G[4 * h + 1] = g.y; G[4 * h + 2] = g.z; G[4 * h + 3] = g.w;
            D[4 * h] = d.x; D[4 * h + 1] = d.y; D[4 * h + 2] = d.z; D[4 * h + 3] = d.w;
            N[4 * h] = i.x; N[4 * h + 1] = i.y; N[4 * h + 2] = i.z; N[4 * h + 3] = i.w;
        }
        present = (1u << SORT_SLOTS) - 1;
    } else {
        #pragma unroll
        for (int u = 0; u < SORT_SLOTS; ++u) {
            const int li = ((u >> 2) * SORT_THREADS + tid) * 4 + (u & 3);
            P[u] = G[u] = D[u] = N[u] = 0;
            if (li < cnt) {
                const int64_t r = r0 + li;
                P[u] = __ldg(prompt + r); G[u] = __ldg(generated + r);
                D[u] = __ldg(predicted + r); N[u] = __ldg(instance + r);
                present |= 1u << u;
            }
        }
    }
    // hist is cleared 16 bytes at a time (it is padded to whole groups)
    const int groups = (n_tiles + 4) >> 2;                    // 16-byte groups that cover n_tiles + 1 counts
    for (int i = tid; i < groups; i += SORT_THREADS) reinterpret_cast<uint4*>(hist)[i] = make_uint4(0, 0, 0, 0);
    if (tid == 0) block_max = 0;
    __syncthreads();

    // ---- pack and count: the counting atomic hands back the request's rank inside its tile
    unsigned long long rec[SORT_SLOTS];
    int tile_of[SORT_SLOTS];                 // -1 when there is nothing to place
    unsigned int rank[SORT_SLOTS];
    bool any_bad = false;
    unsigned int max_b = 0;
    #pragma unroll
    for (int u = 0; u < SORT_SLOTS; ++u) {
        const Packed p = pack_request(P[u], G[u], D[u], N[u], sh);
        const bool here = (present >> u) & 1u;
        const bool live = here & p.live;
        any_bad |= here & p.bad;
        rec[u] = p.rec;
        tile_of[u] = live ? p.tile : -1;
        const unsigned int b = live ? (unsigned int)p.rec : 0u;
        max_b = b > max_b ? b : max_b;
        if (live && p.excess) atomicAdd(&excess[N[u]], (unsigned long long)p.excess);
    }
    #pragma unroll
    for (int u = 0; u < SORT_SLOTS; ++u) {
        rank[u] = 0;
        if (tile_of[u] >= 0) rank[u] = atomicAdd(&hist[tile_of[u]], 1u);
    }
    max_b = __reduce_max_sync(0xffffffffu, max_b);
    if (lane == 0 && max_b) atomicMax(&block_max, max_b);
    __syncthreads();

    // ---- exclusive scan of the per-tile counts, in place; a thread owns whole 16-byte groups
    {
        const int per = (groups + SORT_THREADS - 1) / SORT_THREADS;
        const int g0 = tid * per;
        unsigned int local = 0;
        for (int k = 0; k < per; ++k) {
            if (g0 + k < groups) {
                const uint4 v = reinterpret_cast<const uint4*>(hist)[g0 + k];
                local += v.x + v.y + v.z + v.w;
            }
        }
        unsigned int x = local;
        #pragma unroll
        for (int off = 1; off < 32; off <<= 1) {
            const unsigned int y = __shfl_up_sync(0xffffffffu, x, off);
            if (lane >= off) x += y;
        }
        if (lane == 31) warp_tot[warp] = x;
        __syncthreads();
        // what the warps before this one hold: a 16-lane scan of the warp totals
        unsigned int w = lane < SORT_THREADS / 32 ? warp_tot[lane] : 0u;
        #pragma unroll
        for (int off = 1; off < SORT_THREADS / 32; off <<= 1) {
            const unsigned int y = __shfl_up_sync(0xffffffffu, w, off);
            if (lane >= off) w += y;
        }
        const unsigned int before = __shfl_sync(0xffffffffu, w, warp > 0 ? warp - 1 : 0);
        unsigned int run = x - local + (warp > 0 ? before : 0u);
        for (int k = 0; k < per; ++k) {
            if (g0 + k < groups) {
                const uint4 v = reinterpret_cast<const uint4*>(hist)[g0 + k];
                uint4 o;
                o.x = run; run += v.x;
                o.y = run; run += v.y;
                o.z = run; run += v.z;
                o.w = run; run += v.w;
                reinterpret_cast<uint4*>(hist)[g0 + k] = o;   // entries past n_tiles hold the chunk's total
            }
        }
    }
    __syncthreads();

    // ---- offsets {start, length} (consecutive threads, consecutive tiles) and records
    unsigned int* my_off = chunk_off + (size_t)ch * n_tiles;
    for (int i = tid; i < n_tiles; i += SORT_THREADS) {
        const unsigned int a = hist[i];
        my_off[i] = a | ((hist[i + 1] - a) << 16);
    }
    if (tid == 0) chunk_max[ch] = block_max;
    // the records are put in order in shared memory (a scattered store there costs little) and
    // leave in one bulk copy: scattered 8-byte stores to global memory would each touch a sector
    unsigned long long* stage = reinterpret_cast<unsigned long long*>(hist + 4 * groups);
    #pragma unroll
    for (int u = 0; u < SORT_SLOTS; ++u)
        if (tile_of[u] >= 0) stage[hist[tile_of[u]] + rank[u]] = rec[u];
    if (any_bad) atomicOr(status, PRE_ST_BADREQ);
    asm volatile("fence.proxy.async.shared::cta;" ::: "memory");
    __syncthreads();
    if (tid == 0) {
        const unsigned int bytes = ((hist[n_tiles] + 1u) & ~1u) * 8u;   // whole 16 bytes; the span has room (chunk is even)
        if (bytes) {
            const unsigned int src = (unsigned int)__cvta_generic_to_shared(stage);
            asm volatile("cp.async.bulk.global.shared::cta.bulk_group [%0], [%1], %2;"
                         :: "l"(records + r0), "r"(src), "r"(bytes) : "memory");
            asm volatile("cp.async.bulk.commit_group;" ::: "memory");
            asm volatile("cp.async.bulk.wait_group.read 0;" ::: "memory");   // shared memory must outlive the copy
        }
    }
}

// ---------------------------------------------------------------------------------------
// Step 2.  A persistent grid of blocks; a block builds one tile after another.  Shared memory
// holds one 64-bit word per cell (row, j) of the tile, {low: sum of B, high: count}, updated
// with two 32-bit atomics whose results are not needed, in the swizzled layout of cell_bytes().
// A run of RUN consecutive cells of a row belongs to one thread, which keeps it in registers
// for the whole scan.  A warp serves 32 consecutive runs of one row, or, when a row has fewer
// than 32 runs, several rows side by side (W lanes each).  The finished tile, int64 values in
// the same layout, leaves shared memory in bulk tensor stores issued by one thread.
//
// A tile has a few records in every chunk, each piece somewhere else in memory, so the gather
// is bound by the number of separate 32-byte sectors it touches: a lane reads its piece in
// aligned 32-byte windows (one load each).  The first windows of the NEXT tile are copied into
// a per-thread slot of shared memory asynchronously while this tile is scanned and stored, and
// the offset word they need is loaded one tile earlier still, so the accumulation of a tile
// does not wait for global memory.
//
// All sums, and the map values themselves, fit 32 bits as long as
//     (records of the tile) * (max(largest B, 32) + H) < 2^32,
// which the block checks once it has accumulated.  Otherwise it works in wide mode: the counts
// stay in shared memory, the sums of B are accumulated with 64-bit atomics in the tile's own
// rows of `curves` (cleared first), and the scan runs in 64 bits.
constexpr int TILE_MAX_THREADS = 512;
constexpr int TILE_BUFFERS = 1;

struct TileArgs {
    BuildShape sh;
    TileGeom g;
    const unsigned long long* records;
    const unsigned int* chunk_off;     // fast path (else null)
    const unsigned int* chunk_max;
    int NC;
    unsigned int chunk;
    const unsigned int* bin_base;      // slow path
    unsigned int* bin_cursor;
    unsigned int* bin_count;
    unsigned long long* excess;
    int64_t* curves;
    int64_t* current_d;
    int buffer_runs;                   // runs of 128 bytes in one cell buffer (a multiple of 8)
    int use_tma;                       // the tensor map describes `curves` as runs of 128 bytes
};

constexpr int WINDOW = 4;          // records of one 32-byte load
constexpr int WINDOWS_AHEAD = 2;   // windows of a chunk's piece that a lane loads before using any
constexpr int WINDOWS_ALONE = 8;   // beyond this many, the whole warp shares a lane's piece

// This lane's piece of the tile's records in one trip over the chunks (chunk c = first + lane):
// records [s, s + len) of the chunk's span, read in aligned windows of four starting at `win`.
struct Piece {
    const unsigned long long* win;   // 32-byte aligned
    unsigned int skip;               // records of the first window that belong to the previous tile
    unsigned int len;
    unsigned int n_win;
};

__device__ __forceinline__ unsigned int load_offset(const TileArgs& a, int tile, int c) {
    return tile < a.sh.n_tiles && c < a.NC
               ? __ldg(a.chunk_off + ((unsigned int)c * (unsigned int)a.sh.n_tiles + tile)) : 0u;
}

__device__ __forceinline__ Piece piece_of(const TileArgs& a, int c, unsigned int w) {
    Piece p;
    const unsigned int s = w & 0xFFFFu;
    p.len = w >> 16;
    p.skip = s & (WINDOW - 1);
    p.win = a.records + ((unsigned int)c * a.chunk + (s - p.skip));
    p.n_win = p.len ? (p.skip + p.len + WINDOW - 1) / WINDOW : 0u;
    return p;
}

struct Window { unsigned long long r[WINDOW]; };

// One 32-byte load (the span of a chunk starts on a 32-byte boundary and is a whole number of windows).
__device__ __forceinline__ Window load_window(const unsigned long long* p) {
    Window x;
    asm volatile("ld.global.nc.v4.u64 {%0, %1, %2, %3}, [%4];"
                 : "=l"(x.r[0]), "=l"(x.r[1]), "=l"(x.r[2]), "=l"(x.r[3]) : "l"(p));
    return x;
}

// The same window copied into shared memory behind the thread's back (two 16-byte pieces).
__device__ __forceinline__ void copy_window_async(unsigned char* dst_shared, const unsigned long long* p) {
    const unsigned int d = (unsigned int)__cvta_generic_to_shared(dst_shared);
    asm volatile("cp.async.cg.shared.global [%0], [%1], 16;" :: "r"(d), "l"(p) : "memory");
    asm volatile("cp.async.cg.shared.global [%0], [%1], 16;" :: "r"(d + 16u), "l"(p + 2) : "memory");
}

__device__ __forceinline__ Window read_window(const unsigned char* src_shared) {
    Window x;
    const ulonglong2 lo = *reinterpret_cast<const ulonglong2*>(src_shared);
    const ulonglong2 hi = *reinterpret_cast<const ulonglong2*>(src_shared + 16);
    x.r[0] = lo.x; x.r[1] = lo.y; x.r[2] = hi.x; x.r[3] = hi.y;
    return x;
}

// f(record) for the records of window k of a piece.
template <class F>
__device__ __forceinline__ void apply_window(const Window& x, unsigned int k, unsigned int skip, unsigned int len, F f) {
    #pragma unroll
    for (int i = 0; i < WINDOW; ++i)
        if (k * WINDOW + i - skip < len) f(x.r[i]);      // unsigned: also false in front of the piece
}

// f(record) for what a lane has not loaded ahead: its windows up to WINDOWS_ALONE by itself, and
// the rest of a long piece (a skewed or instance-ordered table) with all lanes of the warp.
template <class F>
__device__ __forceinline__ void apply_rest(const Piece& p, F f) {
    const int lane = threadIdx.x & 31;
    const unsigned int alone = p.n_win < (unsigned int)WINDOWS_ALONE ? p.n_win : (unsigned int)WINDOWS_ALONE;
    for (unsigned int k = WINDOWS_AHEAD; k < alone; ++k) apply_window(load_window(p.win + k * WINDOW), k, p.skip, p.len, f);
    unsigned int longs = __ballot_sync(0xffffffffu, p.n_win > (unsigned int)WINDOWS_ALONE);
    while (longs) {
        const int src = __ffs(longs) - 1;
        longs &= longs - 1;
        const unsigned long long* win =
            reinterpret_cast<const unsigned long long*>(__shfl_sync(0xffffffffu, reinterpret_cast<unsigned long long>(p.win), src));
        const unsigned int skip = __shfl_sync(0xffffffffu, p.skip, src);
        const unsigned int len = __shfl_sync(0xffffffffu, p.len, src);
        const unsigned int n_win = __shfl_sync(0xffffffffu, p.n_win, src);
        for (unsigned int k = WINDOWS_ALONE + lane; k < n_win; k += 32) apply_window(load_window(win + k * WINDOW), k, skip, len, f);
    }
}

__global__ void __launch_bounds__(TILE_MAX_THREADS, 2)
pre_tile_build(const TileArgs a, const __grid_constant__ CUtensorMap out_map) {
    extern __shared__ unsigned char smem_raw[];
    const TileGeom& g = a.g;
    const int H = a.sh.H, T = 1 << a.sh.tile_shift, hp = a.sh.hp, n_tiles = a.sh.n_tiles;
    const int nwarps = blockDim.x >> 5;
    const int tid = threadIdx.x, nthr = blockDim.x, lane = tid & 31;
    // carve: cell buffers (1024-byte aligned: the swizzle pattern repeats every 1024 bytes), backlog
    // sums, piece sums, piece counts
    const unsigned int raw = (unsigned int)__cvta_generic_to_shared(smem_raw);
    unsigned char* cells0 = smem_raw + ((1024u - (raw & 1023u)) & 1023u);
    const size_t buffer_bytes = (size_t)a.buffer_runs << 7;
    unsigned long long* cur = reinterpret_cast<unsigned long long*>(cells0 + TILE_BUFFERS * buffer_bytes);   // [T]
    unsigned long long* piece_s = cur + T;                                                                   // [nwarps]
    unsigned int* piece_n = reinterpret_cast<unsigned int*>(piece_s + nwarps);                               // [nwarps]
    // [WINDOWS_AHEAD][nthr] windows of 32 bytes: where the next tile's first records arrive
    unsigned char* stage = reinterpret_cast<unsigned char*>(cur) + (((size_t)T * 8 + (size_t)nwarps * 12 + 31) & ~(size_t)31);
    __shared__ unsigned int tile_records, tile_max_b, table_max_b;

    const bool fast = a.chunk_off != nullptr;
    const bool tma = a.use_tma != 0;
    // A tile of exactly two store boxes built by 512 threads: threads 0 and 256 each store one
    // box, and each half of the block clears its half of the buffer as soon as ITS box has been
    // read, while the other box may still be on its way out.
    const bool split = tma && nthr == 512 && T * g.rpr == 2 * TMA_BOX_RUNS;
    const int trip = nthr;                        // chunks the block covers in one trip: one per thread

    // ---- once: an upper bound of every B of the table (the largest of the chunks' maxima)
    if (tid == 0) table_max_b = 0;
    __syncthreads();
    if (fast) {
        unsigned int m = 0;
        for (int c = tid; c < a.NC; c += nthr) { const unsigned int x = __ldg(a.chunk_max + c); m = x > m ? x : m; }
        m = __reduce_max_sync(0xffffffffu, m);
        if (lane == 0 && m) atomicMax(&table_max_b, m);
    }

    // this thread's piece of the block's first tile is on its way; the offset word of the second is loaded
    Piece mine;
    unsigned int w = 0;
    mine.win = a.records; mine.skip = 0; mine.len = 0; mine.n_win = 0;
    if (fast) {
        mine = piece_of(a, tid, load_offset(a, blockIdx.x, tid));
        #pragma unroll
        for (int k = 0; k < WINDOWS_AHEAD; ++k)
            if ((unsigned int)k < mine.n_win) copy_window_async(stage + ((size_t)(k * nthr + tid) << 5), mine.win + k * WINDOW);
        asm volatile("cp.async.commit_group;" ::: "memory");
        w = load_offset(a, blockIdx.x + gridDim.x, tid);
    }

    int it = 0;
    for (int tile = blockIdx.x; tile < n_tiles; tile += gridDim.x, ++it) {
        unsigned char* cells = cells0 + (it & (TILE_BUFFERS - 1)) * buffer_bytes;
        const int row0 = tile << a.sh.tile_shift;
        const int rows = (a.sh.I - row0) < T ? (a.sh.I - row0) : T;

        const unsigned long long beyond = tid < rows ? a.excess[row0 + tid] : 0ull;

        // ---- the cell buffer is free once the store that last used it has read it
        if (split) {
            const int half = tid >> 8, t = tid & 255;
            if (t == 0) asm volatile("cp.async.bulk.wait_group.read 0;" ::: "memory");
            __syncwarp();    // the one-lane wait above must not leave the warp split in front of an aligned barrier
            asm volatile("bar.sync %0, 256;" :: "r"(1 + half) : "memory");      // the eight warps of this half
            uint4* z = reinterpret_cast<uint4*>(cells) + (size_t)half * (TMA_BOX_RUNS << 3);
            for (int i = t; i < (TMA_BOX_RUNS << 3); i += 256) z[i] = make_uint4(0, 0, 0, 0);
            if (tid < T) cur[tid] = 0ull;
            if (tid == 0) { tile_records = 0; tile_max_b = 0; }
        } else {
            if (tma && tid == 0) asm volatile("cp.async.bulk.wait_group.read %0;" :: "n"(TILE_BUFFERS - 1) : "memory");
            __syncthreads();
            uint4* z = reinterpret_cast<uint4*>(cells);
            const int nz = a.buffer_runs << 3;
            for (int i = tid; i < nz; i += nthr) z[i] = make_uint4(0, 0, 0, 0);
            for (int i = tid; i < T; i += nthr) cur[i] = 0ull;
            if (tid == 0) { tile_records = 0; tile_max_b = 0; }
        }
        __syncthreads();

        // ---- accumulate: one update per request at (row, R-1)
        unsigned int cnt = 0, max_b = 0;
        auto add = [&](unsigned long long rec) {
            unsigned int* w = reinterpret_cast<unsigned int*>(cells + (unsigned int)(rec >> 32));
            atomicAdd(w, (unsigned int)rec);
            atomicAdd(w + 1, 1u);
        };
        if (fast) {
            cnt = mine.len;
            asm volatile("cp.async.wait_all;" ::: "memory");       // this thread's own copies
            #pragma unroll
            for (int k = 0; k < WINDOWS_AHEAD; ++k)
                if ((unsigned int)k < mine.n_win)
                    apply_window(read_window(stage + ((size_t)(k * nthr + tid) << 5)), k, mine.skip, mine.len, add);
            apply_rest(mine, add);
            for (int base = trip; base < a.NC; base += trip) {      // tables of more than `trip` chunks
                const Piece more = piece_of(a, base + tid, load_offset(a, tile, base + tid));
                cnt += more.len;
                #pragma unroll
                for (int k = 0; k < WINDOWS_AHEAD; ++k)
                    if ((unsigned int)k < more.n_win)
                        apply_window(load_window(more.win + k * WINDOW), k, more.skip, more.len, add);
                apply_rest(more, add);
            }
        } else {
            const unsigned int rec0 = a.bin_base[tile];
            const unsigned int rec1 = rec0 + a.bin_cursor[tile];
            for (unsigned int r = rec0 + tid; r < rec1; r += nthr) {
                const unsigned long long rec = a.records[r];
                const unsigned int b = (unsigned int)rec;
                max_b = b > max_b ? b : max_b;
                ++cnt;
                add(rec);
            }
            max_b = __reduce_max_sync(0xffffffffu, max_b);
            if (lane == 0 && max_b) atomicMax(&tile_max_b, max_b);
        }
        cnt = __reduce_add_sync(0xffffffffu, cnt);
        if (lane == 0 && cnt) atomicAdd(&tile_records, cnt);
        if (fast) {
            // look ahead: the next tile's first windows start their way into this thread's slots (it
            // has read them), and the offset word of the tile after that is loaded
            mine = piece_of(a, tid, w);
            #pragma unroll
            for (int k = 0; k < WINDOWS_AHEAD; ++k)
                if ((unsigned int)k < mine.n_win) copy_window_async(stage + ((size_t)(k * nthr + tid) << 5), mine.win + k * WINDOW);
            asm volatile("cp.async.commit_group;" ::: "memory");
            w = load_offset(a, tile + 2 * gridDim.x, tid);
        }
        __syncthreads();
        const unsigned int largest = fast ? table_max_b : tile_max_b;
        const unsigned long long bound =
            (unsigned long long)tile_records * ((largest > 32u ? largest : 32u) + (unsigned long long)H);

        if (bound < (1ull << 32)) {
            if (g.W == 32 && g.rpr == 32 * g.cpw && rows == T && nthr == 32 * T * g.cpw)
                tile_scan_whole<false>(g.cpw, cells, nullptr, cur, reinterpret_cast<uint2*>(piece_s), false);
            else
                tile_scan_narrow<false>(g, rows, cells, nullptr, cur, piece_n, reinterpret_cast<unsigned int*>(piece_s), false);
            if (tma) {
                asm volatile("fence.proxy.async.shared::cta;" ::: "memory");   // the stores above, for the copy unit
                __syncthreads();
                if (split) {
                    if ((tid & 255) == 0) store_tile_tma(&out_map, cells, tile * (T * g.rpr), (tid >> 8) * TMA_BOX_RUNS, TMA_BOX_RUNS);
                } else if (tid == 0) {
                    store_tile_tma(&out_map, cells, tile * (T * g.rpr), 0, T * g.rpr);
                }
            } else {
                __syncthreads();
                // consecutive lanes on consecutive 16 bytes: the pair p of cells of the tile lies
                // at 16-byte word p ^ ((p >> 3) & 7) of the buffer
                const int half = hp >> 1;               // cell pairs per padded row
                const int total = rows * half;
                const uint4* src = reinterpret_cast<const uint4*>(cells);
                if (hp == H) {
                    ulonglong2* dst = reinterpret_cast<ulonglong2*>(a.curves + (size_t)row0 * H);
                    for (int p = tid; p < total; p += nthr) {
                        const uint4 v = src[p ^ ((p >> 3) & 7)];
                        dst[p] = make_ulonglong2(v.x, v.z);
                    }
                } else {
                    const bool vec_gl = (H & 1) == 0;
                    for (int p = tid; p < total; p += nthr) {
                        const int row = p / half;
                        const int j = (p - row * half) << 1;
                        if (j < H) {
                            const uint4 v = src[p ^ ((p >> 3) & 7)];
                            int64_t* dst = a.curves + ((size_t)(row0 + row) * H + j);
                            if (vec_gl) {
                                *reinterpret_cast<ulonglong2*>(dst) = make_ulonglong2(v.x, v.z);
                            } else {
                                dst[0] = (int64_t)v.x;
                                if (j + 1 < H) dst[1] = (int64_t)v.z;
                            }
                        }
                    }
                }
            }
        } else {
            // ---- wide mode: start over with the sums of B in the tile's rows of `curves`
            __syncthreads();
            {
                uint4* z = reinterpret_cast<uint4*>(cells);
                const int nz = a.buffer_runs << 3;
                for (int i = tid; i < nz; i += nthr) z[i] = make_uint4(0, 0, 0, 0);
            }
            unsigned long long* gsum = reinterpret_cast<unsigned long long*>(a.curves) + (size_t)row0 * H;
            for (int i = tid; i < rows * H; i += nthr) gsum[i] = 0ull;
            __threadfence();
            __syncthreads();
            auto add_wide = [&](unsigned long long rec) {
                const unsigned int at = (unsigned int)(rec >> 32);
                atomicAdd(reinterpret_cast<unsigned int*>(cells + at) + 1, 1u);
                const unsigned int run = at >> 7;
                const unsigned int k = ((((at >> 4) & 7u) ^ (run & 7u)) << 1) | ((at >> 3) & 1u);
                const unsigned int c = (run << 4) | k;                          // cell index in the padded tile
                const unsigned int local = c / (unsigned int)hp;
                atomicAdd(gsum + (size_t)local * H + (c - local * hp), (unsigned long long)(unsigned int)rec);
            };
            if (fast) {
                for (int base = 0; base < a.NC; base += trip) {
                    const Piece more = piece_of(a, base + tid, load_offset(a, tile, base + tid));
                    #pragma unroll
                    for (int k = 0; k < WINDOWS_AHEAD; ++k)
                        if ((unsigned int)k < more.n_win)
                            apply_window(load_window(more.win + k * WINDOW), k, more.skip, more.len, add_wide);
                    apply_rest(more, add_wide);
                }
            } else {
                const unsigned int rec0 = a.bin_base[tile];
                const unsigned int rec1 = rec0 + a.bin_cursor[tile];
                for (unsigned int r = rec0 + tid; r < rec1; r += nthr) add_wide(a.records[r]);
            }
            __threadfence();
            __syncthreads();
            tile_scan_wide(g, H, a.curves, row0, rows, cells, cur, piece_n, piece_s);
            __syncthreads();
            // an empty group keeps "one group per tile", which the wait at the top counts on
            if (tma && tid == 0) asm volatile("cp.async.bulk.commit_group;" ::: "memory");
        }
        // current_d = sum over j of N[j] + what lies beyond the window (left there by the first
        // pass; cleared for the next call).  cur[] is complete: a barrier followed the scan.
        if (tid < rows) {
            a.current_d[row0 + tid] = (int64_t)(cur[tid] + beyond);
            if (beyond) a.excess[row0 + tid] = 0ull;
        }
        if (!fast && tid == 0) { a.bin_cursor[tile] = 0; a.bin_count[tile] = 0; }   // for the next call
    }
    // shared memory must outlive the copy unit's reads of it
    if (tma && (tid == 0 || (split && tid == 256))) asm volatile("cp.async.bulk.wait_group.read 0;" ::: "memory");
}

}  // namespace

// ---------------------------------------------------------------------------------------
// Host side.

static TileArgs tile_args(int I, int H, int T) {
    TileArgs a;
    a.g = tile_geom(H);
    a.sh.I = I; a.sh.H = H; a.sh.rpr = a.g.rpr; a.sh.hp = a.g.rpr * RUN;
    a.sh.tile_shift = 0;
    while ((1 << a.sh.tile_shift) < T) ++a.sh.tile_shift;
    a.sh.n_tiles = (I + T - 1) / T;
    a.records = nullptr; a.chunk_off = nullptr; a.chunk_max = nullptr; a.NC = 0; a.chunk = 0;
    a.bin_base = nullptr; a.bin_cursor = nullptr; a.bin_count = nullptr;
    a.excess = nullptr; a.curves = nullptr; a.current_d = nullptr;
    a.buffer_runs = (T * a.g.rpr + 7) & ~7;
    a.use_tma = 0;
    return a;
}

// Threads of a tile block: one per run, but at least eight warps (the spare ones only help to
// gather, which is what a heavily loaded tile spends its time on).
int pre_tile_threads(int tile_rows, int horizon) {
    const int warps = tile_warps(tile_rows, tile_geom(horizon));
    return 32 * (warps < 8 ? 8 : warps);
}

size_t pre_tile_smem_bytes(int tile_rows, int horizon) {
    const TileGeom g = tile_geom(horizon);
    const size_t warps = (size_t)pre_tile_threads(tile_rows, horizon) / 32;
    const size_t buffer = (size_t)((tile_rows * g.rpr + 7) & ~7) * 128;
    // alignment slack, cell buffers, backlog sums + piece sums + piece counts, windows on their way
    return 1024 + TILE_BUFFERS * buffer + (((size_t)tile_rows * 8 + warps * 12 + 31) & ~(size_t)31) +
           (size_t)WINDOWS_AHEAD * warps * 32 * 32;
}

// Rows per tile: a power of two, about sixteen warps of runs, but several tiles per SM when the
// number of instances allows it.
int pre_tile_rows_for(int n_instances, int horizon, int n_sm) {
    const TileGeom g = tile_geom(horizon);
    int t = g.rpr >= 32 ? 16 / g.cpw : 16 * g.rpw;
    if (t < 1) t = 1;
    if (t > PRE_MAX_TILE_ROWS) t = PRE_MAX_TILE_ROWS;
    int p = 1;
    while (p * 2 <= t) p *= 2;
    while (p > 1 && n_instances / p < 2 * n_sm) p >>= 1;
    return p;
}

// Blocks of the persistent tile kernel: as many as are resident at once, at most one per tile.
int pre_tile_grid(int tile_rows, int horizon, int n_tiles, int n_sm) {
    int per_sm = 0;
    if (cudaOccupancyMaxActiveBlocksPerMultiprocessor(&per_sm, pre_tile_build, pre_tile_threads(tile_rows, horizon),
                                                      pre_tile_smem_bytes(tile_rows, horizon)) != cudaSuccess ||
        per_sm < 1)
        per_sm = 1;
    const long long resident = (long long)per_sm * n_sm;
    return (int)(n_tiles < resident ? n_tiles : resident);
}

// How the table is cut into chunks: no chunk above SORT_CHUNK rows, and, when the table allows
// it, as many chunks as the GPU runs blocks at once (`slots`) but none below ~1024 rows.
// Returns false when the table needs more than `max_chunks` chunks.
static bool sort_geometry(int64_t n, int slots, int max_chunks, int* n_chunks, int64_t* chunk) {
    int64_t nc = (n + SORT_CHUNK - 1) / SORT_CHUNK;
    if (nc > max_chunks) return false;
    int64_t wave = (n + 1023) / 1024;
    if (wave > slots) wave = slots;
    if (nc < wave) nc = wave;
    if (nc > max_chunks) nc = max_chunks;
    if (nc < 1) nc = 1;
    int64_t c = (n + nc - 1) / nc;
    c = (c + 3) & ~(int64_t)3;
    if (c < 4) c = 4;
    *n_chunks = (int)nc;
    *chunk = c;
    return true;
}

static size_t sort_smem_bytes(int n_tiles) { return (((size_t)n_tiles + 4) >> 2) * 16 + (size_t)SORT_CHUNK * 8; }   // counts, records

int pre_sort_max_chunks(int64_t max_requests, int n_sm) {
    int64_t need = (max_requests + SORT_CHUNK - 1) / SORT_CHUNK;
    int64_t wave = (max_requests + 1023) / 1024;
    if (wave > 2 * n_sm) wave = 2 * n_sm;
    if (need < wave) need = wave;
    if (need > SORT_MAX_CHUNKS) need = SORT_MAX_CHUNKS;
    return (int)need;
}

// Words of the offset table (n_tiles per chunk) followed by one word per chunk (its largest B).
size_t pre_chunk_table_words(int n_tiles, int max_chunks) {
    return n_tiles <= PRE_SMEM_BINS ? ((size_t)n_tiles + 1) * (size_t)max_chunks : 0;
}

cudaError_t pre_launch_anticipate(pre_ctx* ctx, const int32_t* prompt, const int32_t* generated,
                                  const int32_t* predicted, const int32_t* instance, int64_t n,
                                  int64_t* curves, int64_t* current_d, cudaStream_t s) {
    if (pre_fused_fits(ctx, n))
        return pre_launch_anticipate_fused(ctx, prompt, generated, predicted, instance, n, curves, current_d, s);
    const int I = ctx->cfg.n_instances, H = ctx->cfg.horizon, T = ctx->tile_rows, nt = ctx->n_tiles;
    const size_t tile_smem = pre_tile_smem_bytes(T, H);
    const int tile_threads = pre_tile_threads(T, H);
    TileArgs a = tile_args(I, H, T);
    a.records = ctx->d_records; a.excess = ctx->d_excess; a.curves = curves; a.current_d = current_d;
    CUtensorMap out_map;
    a.use_tma = make_out_map(&out_map, curves, I, H, T) ? 1 : 0;
    int nc = 1;
    int64_t chunk = 4;
    if (nt <= PRE_SMEM_BINS && sort_geometry(n, 2 * ctx->n_sm, ctx->max_chunks, &nc, &chunk)) {
        // With n == 0 the single chunk is empty: its offsets are all zero and every tile writes zero rows.
        unsigned int* chunk_max = ctx->d_chunk_off + (size_t)nt * ctx->max_chunks;
        pre_chunk_sort<<<nc, SORT_THREADS, sort_smem_bytes(nt), s>>>(
            prompt, generated, predicted, instance, n, a.sh, chunk, ctx->d_records, ctx->d_chunk_off, chunk_max,
            ctx->d_excess, ctx->d_status);
        a.chunk_off = ctx->d_chunk_off; a.chunk_max = chunk_max; a.NC = nc; a.chunk = (unsigned int)chunk;
        pre_tile_build<<<ctx->tile_grid, tile_threads, tile_smem, s>>>(a, out_map);
    } else {
        int grid = (int)((n + BIN_THREADS * 8 - 1) / (BIN_THREADS * 8));
        if (grid > 2 * ctx->n_sm) grid = 2 * ctx->n_sm;
        if (grid < 1) grid = 1;
        if (n > 0) {
            pre_bin_count<<<grid, BIN_THREADS, 0, s>>>(instance, n, I, a.sh.tile_shift, ctx->d_bin_count);
            pre_bin_scan<<<1, 1024, 0, s>>>(ctx->d_bin_count, nt, ctx->d_bin_base);
            pre_bin_scatter<<<grid, BIN_THREADS, 0, s>>>(prompt, generated, predicted, instance, n, a.sh,
                                                       ctx->d_bin_base, ctx->d_bin_cursor, ctx->d_records,
                                                       ctx->d_excess, ctx->d_status);
        }
        // With n == 0 the cursors are zero (every build clears them): every tile sees an empty span.
        a.bin_base = ctx->d_bin_base; a.bin_cursor = ctx->d_bin_cursor; a.bin_count = ctx->d_bin_count;
        pre_tile_build<<<ctx->tile_grid, tile_threads, tile_smem, s>>>(a, out_map);
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
    e = cudaFuncSetAttribute(pre_tile_build, cudaFuncAttributeMaxDynamicSharedMemorySize,
                             optin - (int)attr.sharedSizeBytes);
    if (e != cudaSuccess) return e;
    ctx->tile_grid = pre_tile_grid(ctx->tile_rows, ctx->cfg.horizon, ctx->n_tiles, ctx->n_sm);
    return cudaSuccess;
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
constexpr int PRE_STATIC_MAX_INSTANCES = 65536;    // rows of the map
constexpr size_t PRE_STATIC_STATUS_BYTES = 256;
constexpr size_t PRE_STATIC_OFF_BYTES = (size_t)(PRE_STATIC_MAX_TILES + 1) * PRE_STATIC_MAX_CHUNKS * sizeof(unsigned int);
constexpr size_t PRE_STATIC_REC_BYTES = (size_t)PRE_STATIC_MAX_REQUESTS * sizeof(unsigned long long);
constexpr size_t PRE_STATIC_EXCESS_BYTES = (size_t)PRE_STATIC_MAX_INSTANCES * sizeof(unsigned long long);
constexpr size_t PRE_STATIC_OFF_AT = PRE_STATIC_STATUS_BYTES;
constexpr size_t PRE_STATIC_REC_AT = PRE_STATIC_OFF_AT + ((PRE_STATIC_OFF_BYTES + 255) & ~(size_t)255);
constexpr size_t PRE_STATIC_EXCESS_AT = PRE_STATIC_REC_AT + PRE_STATIC_REC_BYTES;
constexpr size_t PRE_STATIC_BYTES = PRE_STATIC_EXCESS_AT + PRE_STATIC_EXCESS_BYTES;

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
    if (n_requests > PRE_STATIC_MAX_REQUESTS || n_instances > PRE_STATIC_MAX_INSTANCES) return PRE_ESIZE;

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

    int nc = 1;
    int64_t chunk = 4;
    if (!sort_geometry(n_requests, 2 * st->n_sm, PRE_STATIC_MAX_CHUNKS, &nc, &chunk)) return PRE_ESIZE;

    int* status = d_flags ? d_flags : reinterpret_cast<int*>(st->base);
    unsigned int* chunk_off = reinterpret_cast<unsigned int*>(st->base + PRE_STATIC_OFF_AT);
    unsigned int* chunk_max = chunk_off + (size_t)PRE_STATIC_MAX_TILES * PRE_STATIC_MAX_CHUNKS;
    unsigned long long* records = reinterpret_cast<unsigned long long*>(st->base + PRE_STATIC_REC_AT);
    unsigned long long* excess = reinterpret_cast<unsigned long long*>(st->base + PRE_STATIC_EXCESS_AT);
    cudaStream_t s = static_cast<cudaStream_t>(stream);
    // Nothing in the scratch has to be cleared here.  pre_chunk_sort writes every offset that
    // pre_tile_build reads, and a record is read only where an offset says one was written.
    // The per-instance words for what lies beyond the window start as zeros (the array is part of
    // the library image) and pre_tile_build clears each word again after reading it.
    TileArgs a = tile_args(n_instances, horizon, T);
    a.records = records; a.excess = excess; a.curves = d_curves; a.current_d = d_current_d;
    CUtensorMap out_map;
    a.use_tma = make_out_map(&out_map, d_curves, n_instances, horizon, T) ? 1 : 0;
    pre_chunk_sort<<<nc, SORT_THREADS, sort_smem_bytes(n_tiles), s>>>(
        d_prompt, d_generated, d_predicted, d_instance, n_requests, a.sh, chunk, records, chunk_off, chunk_max, excess,
        status);
    a.chunk_off = chunk_off; a.chunk_max = chunk_max; a.NC = nc; a.chunk = (unsigned int)chunk;
    pre_tile_build<<<pre_tile_grid(T, horizon, n_tiles, st->n_sm), pre_tile_threads(T, horizon), tile_smem, s>>>(a, out_map);
    return cudaGetLastError() == cudaSuccess ? PRE_OK : PRE_ECUDA;
}

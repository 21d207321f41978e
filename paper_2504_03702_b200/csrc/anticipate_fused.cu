// Anticipator build as ONE cooperative launch: the fast path of pre_anticipate (paper
// Sec. 4.3.1, the map update applied to every live request; derivation in anticipate.cu).
//
// All blocks are resident (two per SM) and pass through three phases separated by two
// grid-wide barriers:
//   A. Each block takes a contiguous chunk of the request table (at most 16 rows per thread,
//      held in registers), turns every live request into a 4-byte record {cell inside its
//      tile : 13 | B : 19}, counts its records per tile in shared memory, adds the counts to the
//      global per-tile totals (coalesced reductions), and orders the records by tile in shared
//      memory.
//      -- barrier 1: the totals are complete --
//   B. Every block turns the totals into the start of each tile's list (a scan of 4-aligned
//      list lengths), claims room for its piece of every list with one atomic per tile, and
//      copies its ordered records out: a tile's records from all blocks end up CONTIGUOUS in
//      global memory (the order inside a list depends on the claims; the sums do not).
//      -- barrier 2: the lists are complete --
//   C. A block builds one tile after another: the tile's list arrives in shared memory by ONE
//      bulk copy (started while the previous tile is scanned), is accumulated into compact
//      32-bit cells {count : 12 | sum of B : 20}, the suffix scan over the horizon reads and
//      clears those and writes int64 values into a separate buffer, which leaves by bulk tensor
//      stores while the next tile is accumulated.
// A table whose largest B needs more than 19 bits takes 8-byte records (phase B re-reads the
// table); a tile whose compact cells overflow is redone with 64-bit cells; a tile whose sums
// need more than 32 bits is built in the wide mode (64-bit sums in the tile's rows of the
// output).  All three are exact; only their speed differs.
//
// Waits (grid barriers, the arrival of a bulk copy) give up after a bounded number of polls,
// record PRE_ST_TIMEOUT and make every block leave.
#include "build_tile.cuh"

namespace {

constexpr int FUSED_THREADS = 512;
constexpr int FUSED_QUADS = 4;                                  // 16-byte loads per thread and table column (the last one half used)
constexpr int FUSED_CHUNK_MAX = 7168;                           // table rows per block: 14 per thread
constexpr int FUSED_MAX_TILES = 2048;
constexpr int FUSED_TILES_PER_THREAD = FUSED_MAX_TILES / FUSED_THREADS;
constexpr int FUSED_LANDING_WORDS = 3072;                       // room for one bulk copy of a tile's list (12 KB)
constexpr unsigned int REC4_B_BITS = 19;
constexpr unsigned int REC4_B_MASK = (1u << REC4_B_BITS) - 1u;
constexpr unsigned int FUSED_SPIN_LIMIT = 1u << 22;
// words of `sync`
constexpr int SYNC_BARRIER = 0, SYNC_MAX_B = 1, SYNC_ABORT = 2, SYNC_REDO = 3, SYNC_TILE = 4;

struct FusedArgs {
    const int32_t* prompt;
    const int32_t* generated;
    const int32_t* predicted;
    const int32_t* instance;
    long long n;
    long long chunk;              // table rows per block, a multiple of 4, at most FUSED_CHUNK_MAX
    BuildShape sh;
    TileGeom g;
    unsigned int* records;        // the tiles' lists, 4-byte (or 8-byte) records
    unsigned int* totals;         // [n_tiles] records per tile (zero when the call starts)
    unsigned int* totals_next;    // [n_tiles] the next call's totals: cleared by this one
    unsigned int* base;           // [n_tiles + 1] start of each list when laid out exactly, written by block 0
    const unsigned int* hint;     // [n_tiles + 1] where the previous build's lengths put each list (zeros: nowhere)
    unsigned int* hint_next;      // [n_tiles + 1] the same for the next build, written by block 0
    unsigned int record_words;    // room in `records`, in 4-byte words
    unsigned int* sync;           // barrier counter, largest B (zero between calls), ids of an abandoned launch and
                                  // of a launch whose records did not fit the hinted layout
    unsigned int bar_base;        // value of the barrier counter when the launch was made
    unsigned int launch_id;       // never zero
    unsigned int spin_limit;
    unsigned long long* excess;   // [I] remaining tokens beyond the window (zero between calls)
    int64_t* curves;
    int64_t* current_d;
    int* status;
    int buffer_runs;              // runs of 128 bytes in the tile buffer (a multiple of 8)
    int use_tma;                  // 1: the tensor map of whole tiles describes `curves`; 2: so does the one of 32-run boxes
};

__device__ __forceinline__ unsigned int ld_acquire_u32(const unsigned int* p) {
    unsigned int v;
    asm volatile("ld.acquire.gpu.global.u32 %0, [%1];" : "=r"(v) : "l"(p) : "memory");
    return v;
}
__device__ __forceinline__ unsigned int ld_relaxed_u32(const unsigned int* p) {
    unsigned int v;
    asm volatile("ld.relaxed.gpu.global.u32 %0, [%1];" : "=r"(v) : "l"(p) : "memory");
    return v;
}

// Grid-wide barrier over a counter that only grows: every block adds one, then waits until
// the counter has reached `target`.  Returns false (in every thread of the block) when the wait
// was abandoned, here or in another block.
__device__ __forceinline__ bool grid_barrier(const FusedArgs& a, unsigned int target, int* sh_flag) {
    __syncthreads();
    if (threadIdx.x == 0) {
        __threadfence();
        atomicAdd(a.sync + SYNC_BARRIER, 1u);
        bool good = true;
        unsigned int polls = 0;
        while ((int)(ld_acquire_u32(a.sync + SYNC_BARRIER) - target) < 0) {
            ++polls;
            if (polls > a.spin_limit || ((polls & 63u) == 0 && ld_relaxed_u32(a.sync + SYNC_ABORT) == a.launch_id)) {
                good = false;
                break;
            }
            if (polls > 32) __nanosleep(32);
        }
        if (!good) {
            atomicOr(a.status, PRE_ST_TIMEOUT);
            atomicExch(a.sync + SYNC_ABORT, a.launch_id);
        }
        *sh_flag = good ? 1 : 0;
    }
    __syncthreads();
    return *sh_flag != 0;
}

// Exclusive prefix sums of x[0..n) in shared memory, in place; returns the total (all threads).
__device__ __forceinline__ unsigned int block_exclusive_scan(unsigned int* x, int n, unsigned int* warp_tot) {
    const int tid = threadIdx.x, lane = tid & 31, warp = tid >> 5;
    const int per = (n + FUSED_THREADS - 1) / FUSED_THREADS;
    const int i0 = tid * per;
    unsigned int local = 0;
    for (int k = 0; k < per; ++k)
        if (i0 + k < n) local += x[i0 + k];
    unsigned int xs = local;
    #pragma unroll
    for (int off = 1; off < 32; off <<= 1) {
        const unsigned int y = __shfl_up_sync(0xffffffffu, xs, off);
        if (lane >= off) xs += y;
    }
    if (lane == 31) warp_tot[warp] = xs;
    __syncthreads();
    unsigned int w = lane < FUSED_THREADS / 32 ? warp_tot[lane] : 0u;
    #pragma unroll
    for (int off = 1; off < FUSED_THREADS / 32; off <<= 1) {
        const unsigned int y = __shfl_up_sync(0xffffffffu, w, off);
        if (lane >= off) w += y;
    }
    const unsigned int before = __shfl_sync(0xffffffffu, w, warp > 0 ? warp - 1 : 0);
    const unsigned int total = __shfl_sync(0xffffffffu, w, FUSED_THREADS / 32 - 1);
    unsigned int run = xs - local + (warp > 0 ? before : 0u);
    for (int k = 0; k < per; ++k) {
        if (i0 + k < n) {
            const unsigned int v = x[i0 + k];
            x[i0 + k] = run;
            run += v;
        }
    }
    __syncthreads();
    return total;
}

// A table row as phase A and B need it.
struct Cell {
    bool live, bad;
    int tile;
    unsigned int cell;      // row within the tile * hp + (R - 1): where the request's update goes
    unsigned int B;
    unsigned int excess;    // (D - g - H)+
};

__device__ __forceinline__ Cell cell_of(int32_t P, int32_t g, int32_t D, int32_t inst, const BuildShape& sh) {
    Cell o;
    o.B = (unsigned int)P + (unsigned int)g;                               // exact when P, g >= 0
    const int32_t rem = (int32_t)((unsigned int)D - (unsigned int)g);
    const bool ok = ((P | g) >= 0) & (D >= 1) & ((unsigned int)inst < (unsigned int)sh.I);
    const bool fits = (o.B <= (unsigned int)PRE_FIELD_MAX) & (rem <= PRE_FIELD_MAX);
    const bool alive = ok & (rem > 0);                                     // g >= D: finished, a tombstone
    o.bad = !ok | (alive & !fits);
    o.live = alive & fits;
    o.tile = inst >> sh.tile_shift;
    const int local = inst & ((1 << sh.tile_shift) - 1);
    const int R = rem < sh.H ? rem : sh.H;
    o.excess = rem > sh.H ? (unsigned int)(rem - sh.H) : 0u;
    o.cell = (unsigned int)(local * sh.hp + R - 1);
    return o;
}

// The four table rows of quad `h` of this thread: rows r0 + (h * FUSED_THREADS + tid) * 4 + e.
// `present` bit e says whether row e exists.
struct Quad { int4 p, g, d, i; unsigned int present; };

__device__ __forceinline__ Quad load_quad(const FusedArgs& a, long long r0, int cnt, int h, bool vec) {
    Quad q;
    const int li0 = (h * FUSED_THREADS + (int)threadIdx.x) * 4;
    q.present = 0;
    q.p = q.g = q.d = q.i = make_int4(0, 0, 0, 0);
    if (vec && li0 + 4 <= cnt) {           // r0 is a multiple of 4
        const long long at = (r0 + li0) >> 2;
        q.p = __ldcs(reinterpret_cast<const int4*>(a.prompt) + at);
        q.g = __ldcs(reinterpret_cast<const int4*>(a.generated) + at);
        q.d = __ldcs(reinterpret_cast<const int4*>(a.predicted) + at);
        q.i = __ldcs(reinterpret_cast<const int4*>(a.instance) + at);
        q.present = 15u;
    } else if (li0 < cnt) {
        int32_t* pp = &q.p.x; int32_t* gg = &q.g.x; int32_t* dd = &q.d.x; int32_t* ii = &q.i.x;
        #pragma unroll
        for (int e = 0; e < 4; ++e) {
            if (li0 + e < cnt) {
                const long long r = r0 + li0 + e;
                pp[e] = __ldg(a.prompt + r); gg[e] = __ldg(a.generated + r);
                dd[e] = __ldg(a.predicted + r); ii[e] = __ldg(a.instance + r);
                q.present |= 1u << e;
            }
        }
    }
    return q;
}

__global__ void __launch_bounds__(FUSED_THREADS, 2)
pre_build_fused(const FusedArgs a, const __grid_constant__ CUtensorMap out_map, const __grid_constant__ CUtensorMap warp_map) {
    extern __shared__ __align__(16) unsigned char smem_raw[];
    __shared__ unsigned int warp_tot[FUSED_THREADS / 32];
    __shared__ unsigned int sh_max_b;
    __shared__ int sh_flag;
    __shared__ int sh_lost;      // a bulk copy did not arrive in time: every thread leaves after the next barrier
    __shared__ unsigned int sh_word[2];
    __shared__ unsigned int sh_tile[2][4];   // {tile, start of its list, records} of the tile being built, by parity of the step
    __shared__ __align__(8) unsigned long long mbar;

    const TileGeom& g = a.g;
    const int H = a.sh.H, T = 1 << a.sh.tile_shift, hp = a.sh.hp, n_tiles = a.sh.n_tiles;
    const int tid = threadIdx.x, lane = tid & 31, nthr = FUSED_THREADS;
    const int G = gridDim.x, b = blockIdx.x;

    // =====================================================================================
    // Phase A: this block's chunk of the table -> records ordered by tile, in shared memory,
    // and copied to where the previous build's list lengths suggest each tile's list lies.
    const int ntp = (n_tiles + 4) & ~3;                                          // padded to whole 16 bytes
    unsigned int* start = reinterpret_cast<unsigned int*>(smem_raw);             // [ntp] start of each tile among the ordered records
    unsigned int* cursor = start + ntp;                                          // [ntp] counts, then running positions, then where this block's pieces go
    unsigned int* claim = cursor + ntp;                                          // [ntp] offset of this block's piece inside the tile's list
    unsigned int* arr_r = claim + ntp;                                           // [FUSED_CHUNK_MAX] records in table order
    unsigned int* sorted_r = arr_r + FUSED_CHUNK_MAX;                            // [FUSED_CHUNK_MAX] records in tile order
    unsigned short* arr_t = reinterpret_cast<unsigned short*>(sorted_r + FUSED_CHUNK_MAX);   // their tiles (0xffff: no record)
    unsigned short* sorted_t = arr_t + FUSED_CHUNK_MAX;

    const long long r0 = (long long)b * a.chunk < a.n ? (long long)b * a.chunk : a.n;
    const long long r1 = r0 + a.chunk < a.n ? r0 + a.chunk : a.n;
    const int rows_here = (int)(r1 - r0);
    const bool vec = ((reinterpret_cast<uintptr_t>(a.prompt) | reinterpret_cast<uintptr_t>(a.generated) |
                       reinterpret_cast<uintptr_t>(a.predicted) | reinterpret_cast<uintptr_t>(a.instance)) & 15) == 0;

    if (b == 0 && tid == 0) a.sync[SYNC_TILE] = 2u * (unsigned int)G;   // tiles are handed out from here after the barrier
    // two quads of table rows are always on their way while one is being packed
    Quad qa = load_quad(a, r0, rows_here, 0, vec);
    Quad qb = load_quad(a, r0, rows_here, 1, vec);
    for (int i = tid; i < (3 * ntp) >> 2; i += nthr) reinterpret_cast<uint4*>(start)[i] = make_uint4(0, 0, 0, 0);
    if (tid == 0) sh_max_b = 0;
    __syncthreads();

    bool any_bad = false;
    unsigned int max_b = 0;
    auto pack_quad = [&](const Quad& q, int h) {
        const int32_t pp[4] = {q.p.x, q.p.y, q.p.z, q.p.w}, gg[4] = {q.g.x, q.g.y, q.g.z, q.g.w};
        const int32_t dd[4] = {q.d.x, q.d.y, q.d.z, q.d.w}, ii[4] = {q.i.x, q.i.y, q.i.z, q.i.w};
        unsigned int r4[4], t4[4];
        #pragma unroll
        for (int e = 0; e < 4; ++e) {
            const Cell c = cell_of(pp[e], gg[e], dd[e], ii[e], a.sh);
            const bool here = (q.present >> e) & 1u;
            const bool live = here & c.live;
            any_bad |= here & c.bad;
            r4[e] = (c.cell << REC4_B_BITS) | (c.B & REC4_B_MASK);
            t4[e] = live ? (unsigned int)c.tile : 0xffffu;
            if (live) {
                max_b = c.B > max_b ? c.B : max_b;
                atomicAdd(&cursor[c.tile], 1u);
                if (c.excess) atomicAdd(&a.excess[ii[e]], (unsigned long long)c.excess);
            }
        }
        const int li0 = (h * FUSED_THREADS + tid) * 4;
        if (li0 < FUSED_CHUNK_MAX) {
            *reinterpret_cast<uint4*>(arr_r + li0) = make_uint4(r4[0], r4[1], r4[2], r4[3]);
            *reinterpret_cast<uint2*>(arr_t + li0) = make_uint2(t4[0] | (t4[1] << 16), t4[2] | (t4[3] << 16));
        }
    };
    pack_quad(qa, 0);
    qa = load_quad(a, r0, rows_here, 2, vec);
    pack_quad(qb, 1);
    qb = load_quad(a, r0, rows_here, 3, vec);
    pack_quad(qa, 2);
    pack_quad(qb, 3);
    max_b = __reduce_max_sync(0xffffffffu, max_b);
    if (lane == 0 && max_b) atomicMax(&sh_max_b, max_b);
    if (any_bad) atomicOr(a.status, PRE_ST_BADREQ);
    __syncthreads();

    // Counts -> the block's offset inside every tile's list: what the global total was before
    // this block's count was added.  The atomics' results are needed only after the local scan.
    unsigned int my_cnt[FUSED_TILES_PER_THREAD], my_off[FUSED_TILES_PER_THREAD];
    #pragma unroll
    for (int k = 0; k < FUSED_TILES_PER_THREAD; ++k) {
        const int t = tid + k * nthr;
        my_cnt[k] = 0; my_off[k] = 0;
        if (t < n_tiles) {
            my_cnt[k] = cursor[t];
            start[t] = my_cnt[k];
            if (my_cnt[k]) my_off[k] = atomicAdd(&a.totals[t], my_cnt[k]);
        }
    }
    const unsigned int block_max_b = sh_max_b;
    if (tid == 0 && block_max_b) atomicMax(a.sync + SYNC_MAX_B, block_max_b);
    __syncthreads();
    const unsigned int n_local = block_exclusive_scan(start, n_tiles, warp_tot);
    // where the previous build's lengths put each list (loaded now, used after the local sort)
    unsigned int h0[FUSED_TILES_PER_THREAD], h1[FUSED_TILES_PER_THREAD];
    #pragma unroll
    for (int k = 0; k < FUSED_TILES_PER_THREAD; ++k) {
        const int t = tid + k * nthr;
        h0[k] = h1[k] = 0;
        if (t < n_tiles) {
            cursor[t] = start[t];
            claim[t] = my_off[k];
            h0[k] = __ldcg(a.hint + t);
            h1[k] = __ldcg(a.hint + t + 1);
        }
    }
    __syncthreads();
    for (int idx = tid; idx < ((rows_here + 3) & ~3); idx += 4 * nthr) {     // four rows at a time: their atomics overlap
        unsigned int t16[4], pos[4];
        #pragma unroll
        for (int k = 0; k < 4; ++k) {
            const int at = idx + k * nthr;
            t16[k] = at < FUSED_CHUNK_MAX ? arr_t[at] : 0xffffu;
            pos[k] = 0;
            if (t16[k] != 0xffffu) pos[k] = atomicAdd(&cursor[t16[k]], 1u);
        }
        #pragma unroll
        for (int k = 0; k < 4; ++k) {
            if (t16[k] != 0xffffu) {
                sorted_r[pos[k]] = arr_r[idx + k * nthr];
                sorted_t[pos[k]] = (unsigned short)t16[k];
            }
        }
    }
    __syncthreads();
    // this block's piece of tile t goes to hint[t] + claim[t] if the whole piece lies inside the room kept for the list
    bool misfit = block_max_b > REC4_B_MASK;          // 8-byte records are never placed by the hints
    #pragma unroll
    for (int k = 0; k < FUSED_TILES_PER_THREAD; ++k) {
        const int t = tid + k * nthr;
        if (t < n_tiles) {
            const bool fits = my_off[k] + my_cnt[k] <= h1[k] - h0[k] && h1[k] >= h0[k];
            cursor[t] = fits ? h0[k] + my_off[k] : 0xffffffffu;
            misfit |= my_cnt[k] != 0 && !fits;
        }
    }
    misfit = __syncthreads_or(misfit) != 0;
    for (unsigned int pos = tid; pos < n_local; pos += nthr) {
        const unsigned int t = sorted_t[pos];
        const unsigned int at = cursor[t];
        if (at != 0xffffffffu) a.records[at + (pos - start[t])] = sorted_r[pos];
    }
    if (misfit && tid == 0) atomicExch(a.sync + SYNC_REDO, a.launch_id);
    if (!grid_barrier(a, a.bar_base + (unsigned int)G, &sh_flag)) return;

    // =====================================================================================
    // Phase B, only when some piece did not fit (the first build of a context, a table that
    // changed a lot, 8-byte records): lay the lists out exactly, from the totals, and copy again.
    // (one thread reads the two words every block needs: thousands of warps asking the same L2 line would queue up)
    if (tid == 0) {
        sh_word[0] = __ldcg(a.sync + SYNC_MAX_B);
        sh_word[1] = __ldcg(a.sync + SYNC_REDO);
    }
    __syncthreads();
    const unsigned int largest = sh_word[0];
    const bool fmt8 = largest > REC4_B_MASK;
    const bool exact = sh_word[1] == a.launch_id;
    if (exact) {
        for (int t = tid; t < n_tiles; t += nthr) {
            const unsigned int c = __ldcg(a.totals + t);
            cursor[t] = fmt8 ? (c + 1u) & ~1u : (c + 3u) & ~3u;        // every list starts on a 16-byte boundary
        }
        __syncthreads();
        const unsigned int list_end = block_exclusive_scan(cursor, n_tiles, warp_tot);
        if (b == 0) {
            for (int t = tid; t < n_tiles; t += nthr) a.base[t] = cursor[t];
            if (tid == 0) a.base[n_tiles] = list_end;
        }
        if (!fmt8) {
            for (unsigned int pos = tid; pos < n_local; pos += nthr) {
                const unsigned int t = sorted_t[pos];
                a.records[cursor[t] + claim[t] + (pos - start[t])] = sorted_r[pos];
            }
        } else {
            // The 4-byte records lost the high bits of B: read the chunk again and write 8-byte
            // records {cell : 32 | B : 32} straight to their places (slow, and rare).
            for (int t = tid; t < n_tiles; t += nthr) start[t] = 0;
            __syncthreads();
            unsigned long long* rec8 = reinterpret_cast<unsigned long long*>(a.records);
            for (int h = 0; h < FUSED_QUADS; ++h) {
                const Quad q = load_quad(a, r0, rows_here, h, vec);
                const int32_t pp[4] = {q.p.x, q.p.y, q.p.z, q.p.w}, gg[4] = {q.g.x, q.g.y, q.g.z, q.g.w};
                const int32_t dd[4] = {q.d.x, q.d.y, q.d.z, q.d.w}, ii[4] = {q.i.x, q.i.y, q.i.z, q.i.w};
                for (int e = 0; e < 4; ++e) {
                    const Cell c = cell_of(pp[e], gg[e], dd[e], ii[e], a.sh);
                    if (((q.present >> e) & 1u) && c.live) {
                        const unsigned int pos = atomicAdd(&start[c.tile], 1u);
                        rec8[cursor[c.tile] + claim[c.tile] + pos] = ((unsigned long long)c.cell << 32) | c.B;
                    }
                }
            }
        }
        if (!grid_barrier(a, a.bar_base + 2u * (unsigned int)G, &sh_flag)) return;
    } else {
        // keep the barrier counter in step: every launch adds two arrivals per block
        __syncthreads();
        if (tid == 0) atomicAdd(a.sync + SYNC_BARRIER, 1u);
    }
    const unsigned int* list_at = exact ? a.base : a.hint;
    if (b == 0) {
        // Room for the next build's lists: this build's lengths with an eighth and 32 records to spare.
        // Zeros (no room at all, so the next build lays its lists out exactly) when that does not fit.
        __syncthreads();
        for (int t = tid; t < n_tiles; t += nthr) {
            const unsigned int c = __ldcg(a.totals + t);
            start[t] = (c + (c >> 3) + 32u + 3u) & ~3u;
        }
        __syncthreads();
        const unsigned int room = block_exclusive_scan(start, n_tiles, warp_tot);
        const bool ok = room <= a.record_words;
        for (int t = tid; t < n_tiles; t += nthr) a.hint_next[t] = ok ? start[t] : 0u;
        if (tid == 0) {
            a.hint_next[n_tiles] = ok ? room : 0u;
            a.sync[SYNC_MAX_B] = 0;       // every block has read it; zero for the next call
        }
    }
    __syncthreads();

    // =====================================================================================
    // Phase C: tiles.  A block builds one tile after another; which tile comes next is decided
    // by a global counter (the first two of a block are fixed), so blocks that run ahead take
    // more.  Thread 0 looks a tile's list up one step before its bulk copy starts, and starts the
    // copy one step before the tile is built.
    const unsigned int raw = (unsigned int)__cvta_generic_to_shared(smem_raw);
    unsigned char* cells = smem_raw + ((1024u - (raw & 1023u)) & 1023u);       // the swizzle pattern repeats every 1024 bytes
    const size_t buffer_bytes = (size_t)a.buffer_runs << 7;
    unsigned int* compact = reinterpret_cast<unsigned int*>(cells + buffer_bytes);                  // [buffer_runs * 16]
    unsigned int* landing = compact + ((size_t)a.buffer_runs << 4);                                 // [FUSED_LANDING_WORDS]
    unsigned long long* cur = reinterpret_cast<unsigned long long*>(landing + FUSED_LANDING_WORDS); // [2][T] by parity of the step
    unsigned long long* piece_s = cur + 2 * T;                                                      // [32]
    unsigned int* piece_n = reinterpret_cast<unsigned int*>(piece_s + 32);                          // [32]
    const bool tma = a.use_tma != 0;
    const unsigned int mb = (unsigned int)__cvta_generic_to_shared(&mbar);
    const unsigned int landing_cap = fmt8 ? FUSED_LANDING_WORDS / 2 : FUSED_LANDING_WORDS;   // in records
    const unsigned int rec_words = fmt8 ? 2u : 1u;
    const int warp = tid >> 5;
    // Tiles of whole rows of whole 32-run pieces, one run per thread: every warp stores its own
    // 32 runs as soon as it has written them and waits only for its own previous store.
    const bool warp_stores = a.use_tma == 2 && g.W == 32 && g.rpr == 32 * g.cpw && nthr == 32 * T * g.cpw;

    // thread 0: one bulk copy of records [first, first + count) of a list into the landing area
    auto fetch = [&](unsigned int first, unsigned int count) {
        const unsigned int bytes = ((count * rec_words + 3u) & ~3u) * 4u;      // whole 16 bytes; the lists are padded
        const unsigned int dst = (unsigned int)__cvta_generic_to_shared(landing);
        asm volatile("mbarrier.arrive.expect_tx.shared::cta.b64 _, [%0], %1;" :: "r"(mb), "r"(bytes) : "memory");
        asm volatile("cp.async.bulk.shared::cluster.global.mbarrier::complete_tx::bytes [%0], [%1], %2, [%3];"
                     :: "r"(dst), "l"(a.records + (size_t)first * rec_words), "r"(bytes), "r"(mb) : "memory");
    };
    unsigned int phase = 0;
    // every thread: wait for the copy that `fetch` started; false when the wait ran out
    auto arrived = [&]() {
        unsigned int done = 0, polls = 0;
        while (!done) {
            asm volatile("{ .reg .pred p; mbarrier.try_wait.parity.shared::cta.b64 p, [%1], %2; selp.u32 %0, 1, 0, p; }"
                         : "=r"(done) : "r"(mb), "r"(phase) : "memory");
            if (!done && ++polls > a.spin_limit) break;
        }
        phase ^= 1u;
        return done != 0;
    };
    auto drain_own_stores = [&]() {      // every warp: the copy unit has read what this warp's lane 0 gave it
        if (lane == 0) asm volatile("cp.async.bulk.wait_group.read 0;" ::: "memory");
        __syncwarp();
    };

    // thread 0 only: the tile after the one being built (its list known), and the one after that
    unsigned int t1 = 0, f1 = 0, c1 = 0, t2 = 0;
    if (tid == 0) {
        sh_lost = 0;
        asm volatile("mbarrier.init.shared::cta.b64 [%0], 1;" :: "r"(mb) : "memory");
        asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory");
        const unsigned int t0 = (unsigned int)b;
        unsigned int f0 = 0, c0 = 0;
        t1 = (unsigned int)(b + G);
        if (t0 < (unsigned int)n_tiles) { f0 = __ldcg(list_at + t0); c0 = __ldcg(a.totals + t0); }
        if (t1 < (unsigned int)n_tiles) { f1 = __ldcg(list_at + t1); c1 = __ldcg(a.totals + t1); }
        t2 = t1 < (unsigned int)n_tiles ? atomicAdd(a.sync + SYNC_TILE, 1u) : (unsigned int)n_tiles;
        sh_tile[0][0] = t0; sh_tile[0][1] = f0; sh_tile[0][2] = c0;
    }
    for (int i = tid; i < (a.buffer_runs << 2); i += nthr) reinterpret_cast<uint4*>(compact)[i] = make_uint4(0, 0, 0, 0);
    for (int i = tid; i < 2 * T; i += nthr) cur[i] = 0ull;
    __syncthreads();
    if (tid == 0 && sh_tile[0][0] < (unsigned int)n_tiles && sh_tile[0][2])
        fetch(sh_tile[0][1], sh_tile[0][2] < landing_cap ? sh_tile[0][2] : landing_cap);

    // the tile finished one step ago: its backlog words are written one step late, after a barrier
    int prev_row0 = 0, prev_rows = 0;
    unsigned long long prev_beyond = 0;
    auto finish_previous = [&](int par) {
        if (tid < prev_rows) {
            a.current_d[prev_row0 + tid] = (int64_t)(cur[par * T + tid] + prev_beyond);
            cur[par * T + tid] = 0ull;
            if (prev_beyond) a.excess[prev_row0 + tid] = 0ull;     // for the next call
        }
    };

    // where this thread's run is when every thread owns one (the usual case below)
    const unsigned int row = (unsigned int)warp / (unsigned int)g.cpw, piece = (unsigned int)warp - row * (unsigned int)g.cpw;
    const unsigned int j0 = (piece * 32u + (unsigned int)lane) * RUN;
    unsigned char* const mine = cells + ((size_t)tid << 7);
    const unsigned int sw = ((unsigned int)tid & 7u) << 4;          // piece i of the run lies at byte (i*16) ^ sw
    const int tile_runs = T * g.rpr;
    const unsigned long long per_record = (unsigned long long)(largest > 32u ? largest : 32u) + (unsigned long long)H;

    int it = 0;
    for (;; ++it) {
        const int par = it & 1;
        const unsigned int tile = sh_tile[par][0];
        if (tile >= (unsigned int)n_tiles) break;
        const unsigned int first = sh_tile[par][1], count = sh_tile[par][2];
        const int row0 = (int)tile << a.sh.tile_shift;
        const int rows = (a.sh.I - row0) < T ? (a.sh.I - row0) : T;
        // current_d = sum over j of N[j] + what lies beyond the window (left there by phase A)
        const unsigned long long beyond = tid < rows ? __ldcg(a.excess + row0 + tid) : 0ull;
        const bool wide = (unsigned long long)count * per_record >= (1ull << 32);
        const bool try_compact = !wide && !fmt8;
        unsigned long long* my_cur = cur + par * T;

        // ---- accumulate the list into the compact cells as it arrives
        bool overflow = false;
        for (unsigned int done = 0; done < count; done += landing_cap) {
            const unsigned int part = count - done < landing_cap ? count - done : landing_cap;
            if (done) {                      // a list longer than the landing area: the next part, not prefetched
                __syncthreads();
                if (tid == 0) fetch(first + done, part);
            }
            const bool here = arrived();
            if (!here) sh_lost = 1;          // decided for the whole block after the next barrier
            if (here && try_compact) {
                for (unsigned int i = tid; i < part; i += 4 * nthr) {
                    unsigned int old[4], add[4];
                    #pragma unroll
                    for (int k = 0; k < 4; ++k) {
                        old[k] = 0; add[k] = 0;
                        if (i + k * nthr < part) {
                            const unsigned int rec = landing[i + k * nthr];
                            add[k] = rec & REC4_B_MASK;
                            old[k] = atomicAdd(&compact[compact_word(rec >> REC4_B_BITS)], add[k] | (1u << COMPACT_SUM_BITS));
                        }
                    }
                    #pragma unroll
                    for (int k = 0; k < 4; ++k)
                        overflow |= ((old[k] & COMPACT_SUM_MASK) + add[k] > COMPACT_SUM_MASK) |
                                    ((old[k] >> COMPACT_SUM_BITS) >= COMPACT_MAX_COUNT);
                }
            }
        }
        const bool redo = __syncthreads_or(overflow) != 0;       // barrier 1: the tile's cells are complete, the landing area is free
        if (sh_lost) break;
        if (tid == 0) {
            // the next tile's list starts its way in; the one after is looked up; one more is claimed
            sh_tile[par ^ 1][0] = t1; sh_tile[par ^ 1][1] = f1; sh_tile[par ^ 1][2] = c1;
            if (t1 < (unsigned int)n_tiles && c1) fetch(f1, c1 < landing_cap ? c1 : landing_cap);
            t1 = t2; f1 = 0; c1 = 0;
            if (t1 < (unsigned int)n_tiles) {
                f1 = __ldcg(list_at + t1); c1 = __ldcg(a.totals + t1);
                t2 = atomicAdd(a.sync + SYNC_TILE, 1u);
            }
            a.totals_next[tile] = 0;     // the next call counts into the other array
        }
        finish_previous(par ^ 1);

        if (warp_stores && rows == T && try_compact && !redo) {
            // ---- the usual case.  First half of the scan: this thread's run (cleared as it is read),
            // its totals, the suffix scan over the runs of the warp's piece.
            uint4 v[RUN / 2];     // {sum, count, sum, count} of two cells
            load_run<true>(v, cells, compact, (unsigned int)tid, true);
            unsigned int tn = 0, ts = 0;
            #pragma unroll
            for (int i = 0; i < RUN / 2; ++i) { ts += v[i].x + v[i].z; tn += v[i].y + v[i].w; }
            unsigned int xn = tn, xs = ts;
            #pragma unroll
            for (int off = 1; off < 32; off <<= 1) {
                const unsigned int yn = __shfl_down_sync(0xffffffffu, xn, off);
                const unsigned int ys = __shfl_down_sync(0xffffffffu, xs, off);
                if ((unsigned int)lane + off < 32u) { xn += yn; xs += ys; }
            }
            unsigned int N = xn - tn, A = xs - ts;
            uint2* piece_tot = reinterpret_cast<uint2*>(piece_s);
            if (lane == 0) piece_tot[warp] = make_uint2(xn, xs);
            __syncthreads();     // barrier 2: every compact cell has been read and cleared; the pieces' totals are in place
            for (unsigned int kk = piece + 1; kk < (unsigned int)g.cpw; ++kk) {
                const uint2 t = piece_tot[(unsigned int)warp - piece + kk];
                N += t.x; A += t.y;
            }
            drain_own_stores();  // this warp's 32 runs of the previous tile have left the buffer
            // second half: from the run's last cell down, N[j], A[j], c[j] = A[j] + j * N[j]
            unsigned int sn = 0;
            #pragma unroll
            for (int i = RUN / 2 - 1; i >= 0; --i) {
                uint4 o;
                N += v[i].w; A += v[i].z; sn += N;
                o.z = A + N * (j0 + 2 * i + 1); o.w = 0;
                N += v[i].y; A += v[i].x; sn += N;
                o.x = A + N * (j0 + 2 * i); o.y = 0;
                *reinterpret_cast<uint4*>(mine + ((i * 16) ^ sw)) = o;
            }
            asm volatile("fence.proxy.async.shared::cta;" ::: "memory");   // these stores, for the copy unit
            // sum over j of N[j] = sum over the row's requests of R: each is counted on R steps
            const unsigned int lo = __reduce_add_sync(0xffffffffu, sn & 0xFFFFu);
            const unsigned int hi = __reduce_add_sync(0xffffffffu, sn >> 16);
            __syncwarp();        // every lane's stores and fence come before the one lane's copy
            if (lane == 0) {
                const unsigned int src = (unsigned int)__cvta_generic_to_shared(cells + ((size_t)(warp * 32) << 7));
                asm volatile("cp.async.bulk.tensor.2d.global.shared::cta.bulk_group [%0, {%1, %2}], [%3];"
                             :: "l"(&warp_map), "r"(0), "r"((int)tile * tile_runs + warp * 32), "r"(src) : "memory");
                asm volatile("cp.async.bulk.commit_group;" ::: "memory");
                atomicAdd(&my_cur[row], ((unsigned long long)hi << 16) + lo);
            }
        } else {
            // ---- every other tile (a last tile of fewer rows, shapes without whole pieces, sums that
            // do not fit the compact cells or 32 bits, 8-byte records): built and stored by the
            // whole block, without overlap.
            drain_own_stores();
            __syncthreads();
            const unsigned long long* list8 = reinterpret_cast<const unsigned long long*>(a.records) + first;
            const unsigned int* list4 = a.records + first;
            auto for_each_record = [&](auto f) {       // f(cell, B) over the tile's whole list, from global memory
                if (fmt8) {
                    for (unsigned int i = tid; i < count; i += nthr) {
                        const unsigned long long rec = __ldcg(list8 + i);
                        f((unsigned int)(rec >> 32), (unsigned int)rec);
                    }
                } else {
                    for (unsigned int i = tid; i < count; i += nthr) {
                        const unsigned int rec = __ldcg(list4 + i);
                        f(rec >> REC4_B_BITS, rec & REC4_B_MASK);
                    }
                }
            };
            const bool whole = g.W == 32 && g.rpr == 32 * g.cpw && rows == T && nthr == 32 * T * g.cpw;
            if (try_compact && !redo) {
                if (whole) tile_scan_whole<true>(g.cpw, cells, compact, my_cur, reinterpret_cast<uint2*>(piece_s), false);
                else tile_scan_narrow<true>(g, rows, cells, compact, my_cur, piece_n, reinterpret_cast<unsigned int*>(piece_s), false);
            } else if (!wide) {
                // 64-bit cells {sum of B : 32 | count : 32}, accumulated and scanned in the tile buffer
                if (redo)
                    for (int i = tid; i < (a.buffer_runs << 2); i += nthr) reinterpret_cast<uint4*>(compact)[i] = make_uint4(0, 0, 0, 0);
                for (int i = tid; i < (a.buffer_runs << 3); i += nthr) reinterpret_cast<uint4*>(cells)[i] = make_uint4(0, 0, 0, 0);
                __syncthreads();
                for_each_record([&](unsigned int c, unsigned int B) {
                    unsigned int* w = reinterpret_cast<unsigned int*>(cells + cell_bytes(c));
                    atomicAdd(w, B);
                    atomicAdd(w + 1, 1u);
                });
                __syncthreads();
                if (whole) tile_scan_whole<false>(g.cpw, cells, nullptr, my_cur, reinterpret_cast<uint2*>(piece_s), false);
                else tile_scan_narrow<false>(g, rows, cells, nullptr, my_cur, piece_n, reinterpret_cast<unsigned int*>(piece_s), false);
            } else {
                // wide mode: counts in the tile buffer, sums of B in the tile's rows of `curves`
                for (int i = tid; i < (a.buffer_runs << 3); i += nthr) reinterpret_cast<uint4*>(cells)[i] = make_uint4(0, 0, 0, 0);
                unsigned long long* gsum = reinterpret_cast<unsigned long long*>(a.curves) + (size_t)row0 * H;
                for (int i = tid; i < rows * H; i += nthr) gsum[i] = 0ull;
                __threadfence();
                __syncthreads();
                for_each_record([&](unsigned int c, unsigned int B) {
                    atomicAdd(reinterpret_cast<unsigned int*>(cells + cell_bytes(c)) + 1, 1u);
                    const unsigned int local = c / (unsigned int)hp;
                    atomicAdd(gsum + (size_t)local * H + (c - local * hp), (unsigned long long)B);
                });
                __threadfence();
                __syncthreads();
                tile_scan_wide(g, H, a.curves, row0, rows, cells, my_cur, piece_n, piece_s);
            }
            // the finished rows leave
            if (wide) {
                __syncthreads();
            } else if (tma) {
                asm volatile("fence.proxy.async.shared::cta;" ::: "memory");   // the scan's stores, for the copy unit
                __syncthreads();
                if (tid == 0) {
                    store_tile_tma(&out_map, cells, (int)tile * (T * g.rpr), 0, T * g.rpr);
                    asm volatile("cp.async.bulk.wait_group.read 0;" ::: "memory");
                }
                __syncthreads();
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
                __syncthreads();     // the tile buffer is read before the next scan writes it
            }
        }
        prev_row0 = row0; prev_rows = rows; prev_beyond = beyond;
    }
    __syncthreads();
    if (!sh_lost) {
        if (it > 0) finish_previous((it - 1) & 1);
    } else if (tid == 0) {
        atomicOr(a.status, PRE_ST_TIMEOUT);
        // the copy that did not arrive in time may still be on its way: give it one more bounded wait
        unsigned int done = 0, polls = 0;
        while (!done && ++polls <= FUSED_SPIN_LIMIT)
            asm volatile("{ .reg .pred p; mbarrier.try_wait.parity.shared::cta.b64 p, [%1], %2; selp.u32 %0, 1, 0, p; }"
                         : "=r"(done) : "r"(mb), "r"(phase ^ 1u) : "memory");
    }
    // shared memory must outlive the copy unit's reads of it
    drain_own_stores();
}

}  // namespace

// ---------------------------------------------------------------------------------------
// Host side.

static size_t fused_smem_bytes(int tile_rows, int horizon, int n_tiles) {
    const TileGeom g = tile_geom(horizon);
    const size_t buffer_runs = (size_t)((tile_rows * g.rpr + 7) & ~7);
    const size_t ntp = ((size_t)n_tiles + 4) & ~(size_t)3;
    const size_t phase_a = 3 * ntp * 4 + (size_t)FUSED_CHUNK_MAX * 12;
    const size_t phase_c = 1024 + buffer_runs * 128 + buffer_runs * 64 + (size_t)FUSED_LANDING_WORDS * 4 +
                           (size_t)tile_rows * 16 + 32 * 8 + 32 * 4;
    return phase_a > phase_c ? phase_a : phase_c;
}

// Decides whether contexts of this shape use the fused build and sizes its grid.  Leaves
// ctx->fused_grid at 0 when they do not (the two-kernel build then serves every call).
cudaError_t pre_fused_configure(pre_ctx* ctx) {
    ctx->fused_grid = 0;
    const int I = ctx->cfg.n_instances, H = ctx->cfg.horizon, T = ctx->tile_rows;
    const TileGeom g = tile_geom(H);
    if (ctx->n_tiles > FUSED_MAX_TILES) return cudaSuccess;
    if ((long long)T * g.rpr * RUN > 8192) return cudaSuccess;           // a cell index has 13 bits
    if (tile_warps(T, g) * 32 > FUSED_THREADS) return cudaSuccess;
    int coop = 0;
    cudaError_t e = cudaDeviceGetAttribute(&coop, cudaDevAttrCooperativeLaunch, ctx->device);
    if (e != cudaSuccess) return e;
    if (!coop) return cudaSuccess;
    int optin = 0;
    e = cudaDeviceGetAttribute(&optin, cudaDevAttrMaxSharedMemoryPerBlockOptin, ctx->device);
    if (e != cudaSuccess) return e;
    cudaFuncAttributes attr;
    e = cudaFuncGetAttributes(&attr, pre_build_fused);
    if (e != cudaSuccess) return e;
    const size_t smem = fused_smem_bytes(T, H, ctx->n_tiles);
    if (smem + attr.sharedSizeBytes > (size_t)optin) return cudaSuccess;
    // (the limit is a property of the kernel, shared by every context: always the device maximum)
    e = cudaFuncSetAttribute(pre_build_fused, cudaFuncAttributeMaxDynamicSharedMemorySize,
                             optin - (int)attr.sharedSizeBytes);
    if (e != cudaSuccess) return e;
    int per_sm = 0;
    e = cudaOccupancyMaxActiveBlocksPerMultiprocessor(&per_sm, pre_build_fused, FUSED_THREADS, smem);
    if (e != cudaSuccess) return e;
    if (per_sm < 1) return cudaSuccess;
    if (per_sm > 2) per_sm = 2;
    ctx->fused_grid = per_sm * ctx->n_sm;
    ctx->fused_smem = smem;
    (void)I;
    return cudaSuccess;
}

// Whether the fused build can take a table of n rows on this context.
int64_t pre_fused_max_rows(const pre_ctx* ctx) { return (int64_t)ctx->fused_grid * FUSED_CHUNK_MAX; }

bool pre_fused_fits(const pre_ctx* ctx, int64_t n) { return ctx->fused_grid > 0 && n <= pre_fused_max_rows(ctx); }

cudaError_t pre_launch_anticipate_fused(pre_ctx* ctx, const int32_t* prompt, const int32_t* generated,
                                        const int32_t* predicted, const int32_t* instance, int64_t n,
                                        int64_t* curves, int64_t* current_d, cudaStream_t s) {
    const int I = ctx->cfg.n_instances, H = ctx->cfg.horizon, T = ctx->tile_rows;
    FusedArgs a;
    a.prompt = prompt; a.generated = generated; a.predicted = predicted; a.instance = instance;
    a.n = n;
    const int G = ctx->fused_grid;
    long long chunk = (n + G - 1) / G;
    chunk = (chunk + 3) & ~3LL;
    if (chunk < 4) chunk = 4;
    a.chunk = chunk;
    a.g = tile_geom(H);
    a.sh.I = I; a.sh.H = H; a.sh.rpr = a.g.rpr; a.sh.hp = a.g.rpr * RUN;
    a.sh.tile_shift = 0;
    while ((1 << a.sh.tile_shift) < T) ++a.sh.tile_shift;
    a.sh.n_tiles = ctx->n_tiles;
    a.records = reinterpret_cast<unsigned int*>(ctx->d_records);
    const int flip = ctx->fused_flip;
    ctx->fused_flip ^= 1;
    a.totals = ctx->d_fused_totals[flip]; a.totals_next = ctx->d_fused_totals[flip ^ 1];
    a.hint = ctx->d_fused_hint[flip]; a.hint_next = ctx->d_fused_hint[flip ^ 1];
    a.base = ctx->d_fused_base;
    a.record_words = ctx->fused_record_words;
    a.sync = ctx->d_fused_sync;
    a.bar_base = ctx->fused_bar_base;
    ctx->fused_bar_base += 2u * (unsigned int)G;
    ctx->fused_launch_id += 1;
    if (ctx->fused_launch_id == 0) ctx->fused_launch_id = 1;
    a.launch_id = ctx->fused_launch_id;
    a.spin_limit = ctx->spin_limit;
    a.excess = ctx->d_excess; a.curves = curves; a.current_d = current_d; a.status = ctx->d_status;
    a.buffer_runs = (T * a.g.rpr + 7) & ~7;
    CUtensorMap out_map, warp_map;
    a.use_tma = make_out_map(&out_map, curves, I, H, T) ? 1 : 0;
    if (a.use_tma && (T * a.g.rpr) % 32 == 0 && make_out_map(&warp_map, curves, I, H, T, 32)) a.use_tma = 2;
    else memset(&warp_map, 0, sizeof(warp_map));
    void* params[] = {(void*)&a, (void*)&out_map, (void*)&warp_map};
    return cudaLaunchCooperativeKernel((const void*)pre_build_fused, dim3(G), dim3(FUSED_THREADS), params,
                                       ctx->fused_smem, s);
}

// After a wait ran out the barrier counter and the per-tile words are in an unknown state.
cudaError_t pre_fused_reset(pre_ctx* ctx, cudaStream_t s) {
    if (!ctx->d_fused_sync) return cudaSuccess;
    cudaError_t e = cudaMemsetAsync(ctx->d_fused_sync, 0, 8 * sizeof(unsigned int), s);
    for (int k = 0; k < 2 && e == cudaSuccess; ++k) {
        e = cudaMemsetAsync(ctx->d_fused_totals[k], 0, (size_t)ctx->n_tiles * sizeof(unsigned int), s);
        if (e == cudaSuccess) e = cudaMemsetAsync(ctx->d_fused_hint[k], 0, ((size_t)ctx->n_tiles + 1) * sizeof(unsigned int), s);
    }
    if (e == cudaSuccess) e = cudaMemsetAsync(ctx->d_excess, 0, (size_t)ctx->cfg.n_instances * sizeof(unsigned long long), s);
    ctx->fused_bar_base = 0;
    return e;
}

// Pieces of the anticipator build shared by its kernels: the shape of a build, the packing of a
// request into a record, the geometry of a tile, the suffix scans over the horizon and the bulk
// tensor store of a finished tile (paper Sec. 4.3.1: the map update, accumulated from the release
// end; see anticipate.cu for the derivation).
#pragma once

#include <cuda.h>   // CUtensorMap (types only; the encoder is fetched through the runtime)

#include <cstring>

#include "pre_common.cuh"

namespace {

constexpr int RUN = 16;                 // consecutive cells of a row that one thread scans: 128 bytes

// Shape of the build, the same for every kernel of a call.
struct BuildShape {
    int I, H;
    int tile_shift;   // log2 of the rows per tile
    int n_tiles;
    int rpr;          // runs per row
    int hp;           // rpr * RUN: cells of a padded row
};

// Where cell c of a tile (row within tile * hp + column) lies in the tile's shared memory.  Run
// c/16 occupies 128 consecutive bytes; inside them the 16-byte piece p is stored at position
// p ^ (run & 7).  This is the 128-byte swizzle of the tensor copy unit, so a finished tile can
// leave shared memory in one bulk tensor store, and it lets 32 threads that each own a run
// read and write their runs 16 bytes at a time without bank conflicts.
__host__ __device__ __forceinline__ unsigned int cell_bytes(unsigned int c) {
    const unsigned int run = c >> 4, k = c & 15u;
    return (run << 7) | ((((k >> 1) ^ (run & 7u)) << 4)) | ((k & 1u) << 3);
}

// A request as the tile kernel wants it: {byte offset of its cell word in the tile's shared
// memory : 32 | B : 32}.  The cell of a request is (row within tile, R - 1).
struct Packed {
    bool live, bad;
    int tile;
    unsigned int excess;        // (D - g - H)+
    unsigned long long rec;
};

__device__ __forceinline__ Packed pack_request(int32_t P, int32_t g, int32_t D, int32_t inst, const BuildShape& sh) {
    Packed o;
    const unsigned int B = (unsigned int)P + (unsigned int)g;              // exact when P, g >= 0
    const int32_t rem = (int32_t)((unsigned int)D - (unsigned int)g);
    const bool ok = ((P | g) >= 0) & (D >= 1) & ((unsigned int)inst < (unsigned int)sh.I);
    const bool fits = (B <= (unsigned int)PRE_FIELD_MAX) & (rem <= PRE_FIELD_MAX);
    const bool alive = ok & (rem > 0);                                     // g >= D: finished, a tombstone
    o.bad = !ok | (alive & !fits);
    o.live = alive & fits;
    o.tile = inst >> sh.tile_shift;
    const int local = inst & ((1 << sh.tile_shift) - 1);
    const int R = rem < sh.H ? rem : sh.H;
    o.excess = rem > sh.H ? (unsigned int)(rem - sh.H) : 0u;
    o.rec = ((unsigned long long)cell_bytes((unsigned int)(local * sh.hp + R - 1)) << 32) | B;
    return o;
}

constexpr int TMA_BOX_RUNS = 256;      // rows (runs of 128 bytes) of one bulk tensor store

struct TileGeom {
    int rpr;      // runs per row
    int W;        // lanes that serve one row piece: 32, or the power of two >= rpr when rpr < 32
    int w_shift;  // log2(W)
    int cpw;      // 32-run pieces per row (1 when rpr <= 32)
    int rpw;      // rows per warp (1 when rpr >= 32)
};

inline TileGeom tile_geom(int H) {
    TileGeom g;
    g.rpr = (H + RUN - 1) / RUN;
    if (g.rpr >= 32) {
        g.W = 32; g.w_shift = 5; g.cpw = (g.rpr + 31) / 32; g.rpw = 1;
    } else {
        g.W = 1; g.w_shift = 0;
        while (g.W < g.rpr) { g.W <<= 1; ++g.w_shift; }
        g.cpw = 1; g.rpw = 32 / g.W;
    }
    return g;
}

inline int tile_warps(int T, const TileGeom& g) {
    return g.rpr >= 32 ? T * g.cpw : (T + g.rpw - 1) / g.rpw;
}

// Where this thread's run is: a warp serves one 32-run piece of a row, or several short rows.
struct RunPlace { int row, q, piece, sub; unsigned int seg_mask; };

__device__ __forceinline__ RunPlace run_place(const TileGeom& g) {
    RunPlace p;
    const int lane = threadIdx.x & 31, warp = threadIdx.x >> 5;
    if (g.W == 32) {
        p.row = warp / g.cpw; p.piece = warp - p.row * g.cpw; p.q = p.piece * 32 + lane;
        p.sub = lane; p.seg_mask = 0xffffffffu;
    } else {
        p.row = warp * g.rpw + (lane >> g.w_shift); p.piece = 0; p.q = lane & (g.W - 1);
        p.sub = p.q; p.seg_mask = ((1u << g.W) - 1u) << (lane & ~(g.W - 1));
    }
    return p;
}

// Sum of v over the lanes of a row piece (v < 2^31 each; the sum may need 37 bits).
__device__ __forceinline__ unsigned long long piece_sum(unsigned int v, unsigned int seg_mask) {
    const unsigned int lo = __reduce_add_sync(seg_mask, v & 0xFFFFu);
    const unsigned int hi = __reduce_add_sync(seg_mask, v >> 16);
    return ((unsigned long long)hi << 16) + lo;
}

// Compact cells.  While a tile is being accumulated its cells can also be kept as ONE 32-bit word
// each, {count : 12 | sum of B : 20}, a quarter of the finished tile's size: the scan then reads
// (and clears) 4 bytes per cell instead of 8, and the finished int64 values go to a buffer of
// their own that the copy unit drains while the next tile is accumulated.  A run of 16 cells is
// 64 bytes; its 16-byte piece p lies at position p ^ ((run >> 1) & 3), so that eight consecutive
// runs read piece p from eight different 16-byte bank groups.  The word only holds what fits:
// the accumulation checks every update (the atomic returns the old word) and a tile that does
// not fit is redone with 64-bit cells.
constexpr unsigned int COMPACT_SUM_BITS = 20;
constexpr unsigned int COMPACT_SUM_MASK = (1u << COMPACT_SUM_BITS) - 1u;
constexpr unsigned int COMPACT_MAX_COUNT = (1u << (32 - COMPACT_SUM_BITS)) - 1u;

__device__ __forceinline__ unsigned int compact_word(unsigned int c) {   // word index of cell c of a tile
    const unsigned int run = c >> 4, k = c & 15u;
    return (run << 4) | (((k >> 2) ^ ((run >> 1) & 3u)) << 2) | (k & 3u);
}

// Loads the 16 cells of one run as {sum, count, sum, count} of two cells each: from the 64-bit
// cell words in place, or from the compact words, which are cleared for the next tile.
template <bool COMPACT>
__device__ __forceinline__ void load_run(uint4 (&v)[RUN / 2], const unsigned char* cells, unsigned int* compact,
                                         unsigned int run, bool valid) {
    if (COMPACT) {
        uint4* h = reinterpret_cast<uint4*>(compact + (run << 4));
        const unsigned int f = (run >> 1) & 3u;
        #pragma unroll
        for (int p = 0; p < 4; ++p) {
            uint4 w = make_uint4(0, 0, 0, 0);
            if (valid) { w = h[p ^ f]; h[p ^ f] = make_uint4(0, 0, 0, 0); }
            v[2 * p] = make_uint4(w.x & COMPACT_SUM_MASK, w.x >> COMPACT_SUM_BITS, w.y & COMPACT_SUM_MASK, w.y >> COMPACT_SUM_BITS);
            v[2 * p + 1] = make_uint4(w.z & COMPACT_SUM_MASK, w.z >> COMPACT_SUM_BITS, w.w & COMPACT_SUM_MASK, w.w >> COMPACT_SUM_BITS);
        }
    } else {
        const unsigned char* mine = cells + ((size_t)run << 7);
        const unsigned int sw = (run & 7u) << 4;          // piece i of the run lies at byte (i*16) ^ sw
        #pragma unroll
        for (int i = 0; i < RUN / 2; ++i)
            v[i] = valid ? *reinterpret_cast<const uint4*>(mine + ((i * 16) ^ sw)) : make_uint4(0, 0, 0, 0);
    }
}

// The 32-bit scan of a tile whose every thread owns a run (rows of a whole number of 32-run
// pieces, a full tile, no spare warps): thread t owns run t.  Straight-line code.  The int64
// results go to the cell buffer `cells` (in place when the cells were accumulated there).
// `drain` (rows of several pieces only): thread 0 waits, in front of the barrier inside, until the
// copy unit has read the cell buffer's previous contents; nothing is written there before it.
template <bool COMPACT>
__device__ __forceinline__ void tile_scan_whole(int cpw, unsigned char* cells, unsigned int* compact,
                                                unsigned long long* cur, uint2* piece_tot, bool drain) {
    const unsigned int tid = threadIdx.x, lane = tid & 31u, warp = tid >> 5;
    const unsigned int row = warp / (unsigned int)cpw, piece = warp - row * (unsigned int)cpw;
    const unsigned int j0 = (piece * 32u + lane) * RUN;
    unsigned char* mine = cells + ((size_t)tid << 7);
    const unsigned int sw = (tid & 7u) << 4;          // piece i of the run lies at byte (i*16) ^ sw

    uint4 v[RUN / 2];     // {sum, count, sum, count} of two cells
    load_run<COMPACT>(v, cells, compact, tid, true);
    unsigned int tn = 0, ts = 0;
    #pragma unroll
    for (int i = 0; i < RUN / 2; ++i) { ts += v[i].x + v[i].z; tn += v[i].y + v[i].w; }
    unsigned int xn = tn, xs = ts;
    #pragma unroll
    for (int off = 1; off < 32; off <<= 1) {
        const unsigned int yn = __shfl_down_sync(0xffffffffu, xn, off);
        const unsigned int ys = __shfl_down_sync(0xffffffffu, xs, off);
        if (lane + off < 32u) { xn += yn; xs += ys; }
    }
    unsigned int N = xn - tn, A = xs - ts;
    if (cpw > 1) {
        if (lane == 0) piece_tot[warp] = make_uint2(xn, xs);
        if (drain && tid == 0) asm volatile("cp.async.bulk.wait_group.read 0;" ::: "memory");
        __syncthreads();
        for (unsigned int kk = piece + 1; kk < (unsigned int)cpw; ++kk) {
            const uint2 t = piece_tot[warp - piece + kk];
            N += t.x; A += t.y;
        }
    }
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
    const unsigned int lo = __reduce_add_sync(0xffffffffu, sn & 0xFFFFu);
    const unsigned int hi = __reduce_add_sync(0xffffffffu, sn >> 16);
    if (lane == 0) atomicAdd(&cur[row], ((unsigned long long)hi << 16) + lo);
}

// The scan of one tile in 32 bits for any geometry; the int64 results go to the cell buffer.
template <bool COMPACT>
__device__ __forceinline__ void tile_scan_narrow(const TileGeom& g, int rows, unsigned char* cells,
                                                 unsigned int* compact, unsigned long long* cur,
                                                 unsigned int* piece_n, unsigned int* piece_s, bool drain) {
    const int lane = threadIdx.x & 31, warp = threadIdx.x >> 5;
    const RunPlace at = run_place(g);
    const bool valid = at.row < rows && at.q < g.rpr;
    const unsigned int j0 = (unsigned int)at.q * RUN;
    const unsigned int run = (unsigned int)(at.row * g.rpr + at.q);
    unsigned char* mine = cells + ((size_t)run << 7);
    const unsigned int sw = (run & 7u) << 4;          // piece i of the run lies at byte (i*16) ^ sw

    uint4 v[RUN / 2];     // {sum, count, sum, count} of two cells
    load_run<COMPACT>(v, cells, compact, run, valid);
    unsigned int tn = 0, ts = 0;
    #pragma unroll
    for (int i = 0; i < RUN / 2; ++i) { ts += v[i].x + v[i].z; tn += v[i].y + v[i].w; }

    // suffix sums over the runs of the piece: what lies above this run
    unsigned int xn = tn, xs = ts;
    for (int off = 1; off < g.W; off <<= 1) {
        const unsigned int yn = __shfl_down_sync(0xffffffffu, xn, off, g.W);
        const unsigned int ys = __shfl_down_sync(0xffffffffu, xs, off, g.W);
        if (at.sub + off < g.W) { xn += yn; xs += ys; }
    }
    unsigned int N = xn - tn, A = xs - ts;
    if (g.cpw > 1) {     // the same for every thread of the block
        if (lane == 0) { piece_n[warp] = xn; piece_s[warp] = xs; }
        if (drain && threadIdx.x == 0) asm volatile("cp.async.bulk.wait_group.read 0;" ::: "memory");
        __syncthreads();
        for (int kk = at.piece + 1; kk < g.cpw; ++kk) {
            N += piece_n[at.row * g.cpw + kk];
            A += piece_s[at.row * g.cpw + kk];
        }
    }
    // from the run's last cell down: N[j], A[j], c[j] = A[j] + j * N[j]
    unsigned int sn = 0;
    #pragma unroll
    for (int i = RUN / 2 - 1; i >= 0; --i) {
        uint4 o;
        N += v[i].w; A += v[i].z; sn += N;
        o.z = A + N * (j0 + 2 * i + 1); o.w = 0;
        N += v[i].y; A += v[i].x; sn += N;
        o.x = A + N * (j0 + 2 * i); o.y = 0;
        if (valid) *reinterpret_cast<uint4*>(mine + ((i * 16) ^ sw)) = o;
    }
    // sum over j of N[j] = sum over the row's requests of R: each is counted on R steps
    const unsigned long long sum_n = piece_sum(sn, at.seg_mask);
    if (at.sub == 0 && at.row < rows && sum_n) atomicAdd(&cur[at.row], sum_n);
}

// The same in 64 bits, with the sums of B in the tile's rows of `curves`; writes the rows itself.
__device__ __forceinline__ void tile_scan_wide(const TileGeom& g, int H, int64_t* curves, int row0, int rows,
                                               const unsigned char* cells, unsigned long long* cur,
                                               unsigned int* piece_n, unsigned long long* piece_s) {
    const int lane = threadIdx.x & 31, warp = threadIdx.x >> 5;
    const RunPlace at = run_place(g);
    const bool valid = at.row < rows && at.q < g.rpr;
    const int j0 = at.q * RUN;
    const unsigned int c0 = (unsigned int)(at.row * g.rpr + at.q) * RUN;     // first cell of the run
    unsigned long long* grow = reinterpret_cast<unsigned long long*>(curves) + (size_t)(row0 + at.row) * H;
    auto count_at = [&](int k) { return *reinterpret_cast<const unsigned int*>(cells + cell_bytes(c0 + k) + 4); };

    unsigned int tn = 0;
    unsigned long long ts = 0;
    if (valid) {
        for (int k = 0; k < RUN; ++k) {
            if (j0 + k < H) { tn += count_at(k); ts += __ldcg(grow + j0 + k); }
        }
    }
    unsigned int xn = tn;
    unsigned long long xs = ts;
    for (int off = 1; off < g.W; off <<= 1) {
        const unsigned int yn = __shfl_down_sync(0xffffffffu, xn, off, g.W);
        const unsigned long long ys = __shfl_down_sync(0xffffffffu, xs, off, g.W);
        if (at.sub + off < g.W) { xn += yn; xs += ys; }
    }
    unsigned int N = xn - tn;
    unsigned long long A = xs - ts;
    if (g.cpw > 1) {
        if (lane == 0) { piece_n[warp] = xn; piece_s[warp] = xs; }
        __syncthreads();
        for (int kk = at.piece + 1; kk < g.cpw; ++kk) {
            N += piece_n[at.row * g.cpw + kk];
            A += piece_s[at.row * g.cpw + kk];
        }
    }
    unsigned long long sum_n = 0;
    if (valid) {
        for (int k = RUN - 1; k >= 0; --k) {
            if (j0 + k < H) {
                N += count_at(k);
                A += __ldcg(grow + j0 + k);
                sum_n += N;
                grow[j0 + k] = A + (unsigned long long)N * (unsigned int)(j0 + k);
            }
        }
    }
    for (int off = g.W >> 1; off > 0; off >>= 1) sum_n += __shfl_down_sync(0xffffffffu, sum_n, off, g.W);
    if (at.sub == 0 && at.row < rows && sum_n) atomicAdd(&cur[at.row], sum_n);
}

// One thread: bulk tensor stores of the runs [run0 + first, run0 + first + n_runs) of the map
// from the cell buffer, as one group.
__device__ __forceinline__ void store_tile_tma(const CUtensorMap* map, const unsigned char* cells, int run0,
                                               int first, int n_runs) {
    for (int r = first; r < first + n_runs; r += TMA_BOX_RUNS) {
        const unsigned int src = (unsigned int)__cvta_generic_to_shared(cells + ((size_t)r << 7));
        asm volatile("cp.async.bulk.tensor.2d.global.shared::cta.bulk_group [%0, {%1, %2}], [%3];"
                     :: "l"(map), "r"(0), "r"(run0 + r), "r"(src) : "memory");
    }
    asm volatile("cp.async.bulk.commit_group;" ::: "memory");
}

}  // namespace

// The map as a matrix of runs for the copy unit: [I * H/16 runs][16 int64], stored from
// shared memory in boxes of `box_runs` runs with the 128-byte swizzle.  Only when a row is a
// whole number of runs and a tile a whole number of boxes; otherwise the kernel stores with
// ordinary instructions.  The encoder is a driver entry point, fetched through the runtime so
// that the library does not link against the driver.
typedef CUresult (*encode_tiled_fn)(CUtensorMap*, CUtensorMapDataType, cuuint32_t, void*, const cuuint64_t*,
                                    const cuuint64_t*, const cuuint32_t*, const cuuint32_t*, CUtensorMapInterleave,
                                    CUtensorMapSwizzle, CUtensorMapL2promotion, CUtensorMapFloatOOBfill);

static encode_tiled_fn tensor_map_encoder() {
    static encode_tiled_fn fn = nullptr;
    static bool tried = false;
    if (!tried) {
        tried = true;
        void* p = nullptr;
        cudaDriverEntryPointQueryResult q;
        if (cudaGetDriverEntryPoint("cuTensorMapEncodeTiled", &p, cudaEnableDefault, &q) == cudaSuccess &&
            q == cudaDriverEntryPointSuccess)
            fn = reinterpret_cast<encode_tiled_fn>(p);
        else
            cudaGetLastError();
    }
    return fn;
}

static bool make_out_map(CUtensorMap* map, int64_t* curves, int I, int H, int T, int box_runs = TMA_BOX_RUNS) {
    memset(map, 0, sizeof(*map));
    if (H % RUN != 0) return false;
    const int runs_per_tile = T * (H / RUN);
    if (runs_per_tile > box_runs && runs_per_tile % box_runs != 0) return false;
    encode_tiled_fn enc = tensor_map_encoder();
    if (!enc) return false;
    const cuuint64_t dims[2] = {(cuuint64_t)RUN, (cuuint64_t)I * (cuuint64_t)(H / RUN)};
    const cuuint64_t strides[1] = {(cuuint64_t)RUN * sizeof(int64_t)};
    const cuuint32_t box[2] = {(cuuint32_t)RUN, (cuuint32_t)(runs_per_tile < box_runs ? runs_per_tile : box_runs)};
    const cuuint32_t elem[2] = {1, 1};
    return enc(map, CU_TENSOR_MAP_DATA_TYPE_INT64, 2, curves, dims, strides, box, elem, CU_TENSOR_MAP_INTERLEAVE_NONE,
               CU_TENSOR_MAP_SWIZZLE_128B, CU_TENSOR_MAP_L2_PROMOTION_NONE,
               CU_TENSOR_MAP_FLOAT_OOB_FILL_NONE) == CUDA_SUCCESS;
}

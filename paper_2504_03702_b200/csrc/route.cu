// Load-aware request router (paper Sec. 4.3.3) as one persistent kernel per batch.
//
// The grid is launched cooperatively (all blocks resident, one per SM).  Block b owns a
// fixed, contiguous set of instance rows for the whole batch, so every read and every fold
// of a row happens inside one block and needs only block-level ordering.  As many of the
// block's rows as fit are copied into shared memory when the kernel starts and are scanned
// from there; folds update both copies, so global memory is current at every moment.
//
// Scoring one arrival (P, D) against a row c[0..H): with Dc = min(D, H),
//     peak = max( max_{j<Dc}(c[j] + P + j),  max_{j>=Dc} c[j] ),
// i.e. the literal scan of the row with the arrival virtually added.
//
// The arrivals form a chain (arrival k+1 must see arrival k folded into its winner), but a
// fold changes ONE row.  So the blocks do not wait for the winner of arrival k before they
// scan for arrival k+1; the exchange runs one arrival behind the scan.  Iteration k:
//   1. warps 1.. scan their share of the block's rows for arrival k against the maps as
//      they are (arrival k-1 not folded yet); meanwhile warp 0 collects the G published
//      minima of arrival k-1 (bounded spin) -> winner w;
//   2. the owner of row w folds arrival k-1 into it and, in the same pass, re-scores that
//      one row for arrival k; block 0 appends the request to the table;
//   3. warp 0 turns the block's peaks into scores, takes the (score, index) minimum and
//      publishes it in a slot tagged with the exchange number, while the other warps go on
//      to the next scan.
// Slots are double buffered by the tag's parity: a block publishes exchange s only after it
// has read every slot of s-1, and nobody reads s-2 after publishing s-1.  Every 64-bit word
// of a slot carries the exchange tag, so the exchange needs no fence on either side; a slot
// has a 128-byte line to itself and is read with a single 16-byte request.
#include "pre_common.cuh"

#include <math_constants.h>

#include <cmath>

namespace {

constexpr int ROUTE_THREADS = 1024;
constexpr int ROUTE_WARPS = ROUTE_THREADS / 32;
constexpr int SCAN_WARPS = ROUTE_WARPS - 1;  // warp 0 coordinates
constexpr long long I64_MIN = (-9223372036854775807LL - 1);
constexpr long long I64_MAX = 9223372036854775807LL;
constexpr unsigned int ABORT_SPIN_LIMIT = 1u << 24;  // polls (with pauses) for the other blocks once a wait has run out
constexpr int GATHER_ILP = 5;                  // exchange slots a lane polls at once
// A block's exchange slot has a 128-byte line to itself: with several slots per line the
// polling of 148 blocks and the stores of the line's owners contend, and one exchange takes
// 3.4 us instead of 1.6 us (measured).
constexpr int SLOT_WORDS = 16;

// 16-byte relaxed forms: one L2 request for the two words of a slot (each 64-bit half is
// atomic by itself and carries its own tag).  Measured: an exchange among 148 blocks takes
// about 1.0 us with one request per polled slot and 0.3 us more for every further request.
__device__ __forceinline__ void st_relaxed_v2(unsigned long long* p, unsigned long long x, unsigned long long y) {
    asm volatile("st.relaxed.gpu.global.v2.u64 [%0], {%1, %2};" ::"l"(p), "l"(x), "l"(y) : "memory");
}
__device__ __forceinline__ void ld_relaxed_v2(const unsigned long long* p, unsigned long long& x, unsigned long long& y) {
    asm volatile("ld.relaxed.gpu.global.v2.u64 {%0, %1}, [%2];" : "=l"(x), "=l"(y) : "l"(p) : "memory");
}
__device__ __forceinline__ unsigned int ld_relaxed_u32(const unsigned int* p) {
    unsigned int v;
    asm volatile("ld.relaxed.gpu.global.u32 %0, [%1];" : "=r"(v) : "l"(p) : "memory");
    return v;
}
__device__ __forceinline__ int ld_relaxed_s32(const int* p) {
    int v;
    asm volatile("ld.relaxed.gpu.global.s32 %0, [%1];" : "=r"(v) : "l"(p) : "memory");
    return v;
}

// Row loads.  Global rows are streamed through L2 without L1 allocation (a row is re-read
// only after the block's whole share has gone by); resident rows come from shared memory.
template <bool SMEM>
__device__ __forceinline__ longlong2 ld_row_v2(const int64_t* p) {
    if (SMEM) {
        longlong2 v;
        const unsigned int addr = (unsigned int)__cvta_generic_to_shared(p);
        asm volatile("ld.shared.v2.s64 {%0, %1}, [%2];" : "=l"(v.x), "=l"(v.y) : "r"(addr) : "memory");
        return v;
    }
    return __ldcg(reinterpret_cast<const longlong2*>(p));
}
template <bool SMEM>
__device__ __forceinline__ long long ld_row(const int64_t* p) {
    if (SMEM) {
        long long v;
        const unsigned int addr = (unsigned int)__cvta_generic_to_shared(p);
        asm volatile("ld.shared.s64 %0, [%1];" : "=l"(v) : "r"(addr) : "memory");
        return v;
    }
    return __ldcg(reinterpret_cast<const long long*>(p));
}

__device__ __forceinline__ long long max64(long long a, long long b) { return a > b ? a : b; }

// Maximum of a signed 64-bit value over the warp with two 32-bit warp reductions.
__device__ __forceinline__ long long warp_max64(long long v) {
    const unsigned int hi = (unsigned int)((unsigned long long)v >> 32) ^ 0x80000000u;  // order preserving
    const unsigned int lo = (unsigned int)v;
    const unsigned int mh = __reduce_max_sync(0xffffffffu, hi);
    const unsigned int ml = __reduce_max_sync(0xffffffffu, hi == mh ? lo : 0u);
    return (long long)(((unsigned long long)(mh ^ 0x80000000u) << 32) | ml);
}

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
    unsigned long long* slots;  // [2][G][SLOT_WORDS]: two tagged words per block and parity, rest of the line unused
    unsigned int* epoch_ptr;  // running exchange counter kept on the device: tags stay dense across launches
    int* status;
    int* abort_flag;
    unsigned int* abort_key;    // 0xffffffff - (smallest exchange number at which a block's wait ran out); 0: none
    unsigned int* abort_count;  // blocks that have given up
    unsigned int spin_limit;    // polls before a wait is declared lost
    const int* done_elsewhere;  // when set and non-zero: the batch has been routed by the summary kernel, nothing to do
    int max_rows;       // ceil(I / G)
    size_t resident_bytes;  // shared memory per block left for resident rows
    // admission queue (ADMIT kernels only): a ring of waiting requests, entry q at (head + q) mod capacity
    int32_t* queue_prompt;
    int32_t* queue_predicted;
    int64_t* queue_state;          // {head, length}, rewritten by block 0 at the end
    const int64_t* queue_entry;    // the same two words as they were when the call was made
    long long queue_capacity;
    int32_t* queue_choice;         // results for the entries that were waiting at entry
    long long hot;                 // floor(overload_level * M): a cell counts when it is above
    double many;                   // overload_share * H: overloaded when more cells than this count
};

constexpr int CHOICE_DROPPED = -1, CHOICE_WAITS = -2, CHOICE_TURNED_AWAY = -3;

// Peak over 64-cell chunks [q0, q1) of one row with the arrival (P, Dc) virtually added
// (chunk q covers steps 64q .. 64q+63, two per lane); the result is per lane.
// FULL: H is a multiple of 64 and 16-byte loads are legal, so no bounds checks are needed.
template <bool FULL, bool SMEM>
__device__ __forceinline__ long long scan_row_chunks(const int64_t* __restrict__ row, int q0, int q1, int P,
                                                     int Dc, int H, int lane) {
    // rx / ry: ramp part, even / odd cell of the pair (ry lacks the odd cell's extra +1); t: after the ramp
    long long rx = I64_MIN, ry = I64_MIN, t = I64_MIN;
    if (FULL) {
        const int qr = Dc >> 6;          // chunks [0, qr) lie entirely on the ramp
        const int qt = (Dc + 63) >> 6;   // chunks [qt, ..) lie entirely after it
        const int64_t* p = row + lane * 2;
        int q = q0;
        const int e1 = q1 < qr ? q1 : qr;
        for (; q + 4 <= e1; q += 4) {
            longlong2 v[4];
            #pragma unroll
            for (int u = 0; u < 4; ++u) v[u] = ld_row_v2<SMEM>(p + (q + u) * 64);
            const long long jp = (long long)(q * 64 + lane * 2) + P;
            #pragma unroll
            for (int u = 0; u < 4; ++u) {
                rx = max64(rx, v[u].x + (jp + u * 64));
                ry = max64(ry, v[u].y + (jp + u * 64));
            }
        }
        for (; q < e1; ++q) {
            const longlong2 v = ld_row_v2<SMEM>(p + q * 64);
            const long long jp = (long long)(q * 64 + lane * 2) + P;
            rx = max64(rx, v.x + jp);
            ry = max64(ry, v.y + jp);
        }
        if (q < q1 && q < qt) {  // the one chunk that holds the end of the ramp
            const longlong2 v = ld_row_v2<SMEM>(p + q * 64);
            const int j = q * 64 + lane * 2;
            const long long jp = (long long)j + P;
            if (j < Dc) rx = max64(rx, v.x + jp); else t = max64(t, v.x);
            if (j + 1 < Dc) ry = max64(ry, v.y + jp); else t = max64(t, v.y);
            ++q;
        }
        long long t2 = I64_MIN;
        for (; q + 4 <= q1; q += 4) {
            longlong2 v[4];
            #pragma unroll
            for (int u = 0; u < 4; ++u) v[u] = ld_row_v2<SMEM>(p + (q + u) * 64);
            #pragma unroll
            for (int u = 0; u < 4; ++u) { t = max64(t, v[u].x); t2 = max64(t2, v[u].y); }
        }
        for (; q < q1; ++q) {
            const longlong2 v = ld_row_v2<SMEM>(p + q * 64);
            t = max64(t, v.x);
            t2 = max64(t2, v.y);
        }
        t = max64(t, t2);
    } else {
        for (int q = q0; q < q1; ++q) {
            const int j = q * 64 + lane * 2;
            const long long jp = (long long)j + P;
            if (j < H) {
                const long long x = ld_row<SMEM>(row + j);
                if (j < Dc) rx = max64(rx, x + jp); else t = max64(t, x);
            }
            if (j + 1 < H) {
                const long long y = ld_row<SMEM>(row + j + 1);
                if (j + 1 < Dc) ry = max64(ry, y + jp); else t = max64(t, y);
            }
        }
    }
    if (ry != I64_MIN) rx = max64(rx, ry + 1);
    return max64(rx, t);
}

// The same scan when every cell of the row segment, with the arrival added, is known to lie
// in [0, 2^32): only the low words take part, one 32-bit max per cell.  H is a multiple of 64.
template <bool SMEM>
__device__ __forceinline__ unsigned int scan_row_chunks_narrow(const int64_t* __restrict__ row, int q0, int q1,
                                                               int P, int Dc, int lane) {
    unsigned int rx = 0, ry = 0, t = 0, t2 = 0;   // all cells are >= 0, so 0 is a neutral start
    bool any_ry = false;
    const int qr = Dc >> 6, qt = (Dc + 63) >> 6;
    const int64_t* p = row + lane * 2;
    int q = q0;
    const int e1 = q1 < qr ? q1 : qr;
    any_ry = q < e1;
    for (; q + 4 <= e1; q += 4) {
        longlong2 v[4];
        #pragma unroll
        for (int u = 0; u < 4; ++u) v[u] = ld_row_v2<SMEM>(p + (q + u) * 64);
        const unsigned int jp = (unsigned int)(q * 64 + lane * 2 + P);
        #pragma unroll
        for (int u = 0; u < 4; ++u) {
            rx = max(rx, (unsigned int)v[u].x + (jp + u * 64));
            ry = max(ry, (unsigned int)v[u].y + (jp + u * 64));
        }
    }
    for (; q < e1; ++q) {
        const longlong2 v = ld_row_v2<SMEM>(p + q * 64);
        const unsigned int jp = (unsigned int)(q * 64 + lane * 2 + P);
        rx = max(rx, (unsigned int)v.x + jp);
        ry = max(ry, (unsigned int)v.y + jp);
    }
    if (q < q1 && q < qt) {  // the one chunk that holds the end of the ramp
        const longlong2 v = ld_row_v2<SMEM>(p + q * 64);
        const int j = q * 64 + lane * 2;
        const unsigned int jp = (unsigned int)(j + P);
        if (j < Dc) rx = max(rx, (unsigned int)v.x + jp); else t = max(t, (unsigned int)v.x);
        if (j + 1 < Dc) { ry = max(ry, (unsigned int)v.y + jp); any_ry = true; } else t = max(t, (unsigned int)v.y);
        ++q;
    }
    for (; q + 4 <= q1; q += 4) {
        longlong2 v[4];
        #pragma unroll
        for (int u = 0; u < 4; ++u) v[u] = ld_row_v2<SMEM>(p + (q + u) * 64);
        #pragma unroll
        for (int u = 0; u < 4; ++u) { t = max(t, (unsigned int)v[u].x); t2 = max(t2, (unsigned int)v[u].y); }
    }
    for (; q < q1; ++q) {
        const longlong2 v = ld_row_v2<SMEM>(p + q * 64);
        t = max(t, (unsigned int)v.x);
        t2 = max(t2, (unsigned int)v.y);
    }
    if (any_ry) rx = max(rx, ry + 1);   // the odd cell of a pair sits one step later
    return max(max(rx, t), t2);
}

// The same again for a resident row kept as 32-bit cells (8-byte load = two cells per lane).
__device__ __forceinline__ unsigned int scan_row_chunks_packed(const uint32_t* __restrict__ row, int q0, int q1,
                                                               int P, int Dc, int lane) {
    unsigned int rx = 0, ry = 0, t = 0, t2 = 0;
    const int qr = Dc >> 6, qt = (Dc + 63) >> 6;
    const unsigned int base = (unsigned int)__cvta_generic_to_shared(row + lane * 2);
    auto ld2 = [&](int q) {
        uint2 v;
        asm volatile("ld.shared.v2.u32 {%0, %1}, [%2];" : "=r"(v.x), "=r"(v.y) : "r"(base + q * 256) : "memory");
        return v;
    };
    int q = q0;
    const int e1 = q1 < qr ? q1 : qr;
    bool any_ry = q < e1;
    for (; q + 4 <= e1; q += 4) {
        uint2 v[4];
        #pragma unroll
        for (int u = 0; u < 4; ++u) v[u] = ld2(q + u);
        const unsigned int jp = (unsigned int)(q * 64 + lane * 2 + P);
        #pragma unroll
        for (int u = 0; u < 4; ++u) { rx = max(rx, v[u].x + (jp + u * 64)); ry = max(ry, v[u].y + (jp + u * 64)); }
    }
    for (; q < e1; ++q) {
        const uint2 v = ld2(q);
        const unsigned int jp = (unsigned int)(q * 64 + lane * 2 + P);
        rx = max(rx, v.x + jp);
        ry = max(ry, v.y + jp);
    }
    if (q < q1 && q < qt) {  // the one chunk that holds the end of the ramp
        const uint2 v = ld2(q);
        const int j = q * 64 + lane * 2;
        const unsigned int jp = (unsigned int)(j + P);
        if (j < Dc) rx = max(rx, v.x + jp); else t = max(t, v.x);
        if (j + 1 < Dc) { ry = max(ry, v.y + jp); any_ry = true; } else t = max(t, v.y);
        ++q;
    }
    for (; q + 4 <= q1; q += 4) {
        uint2 v[4];
        #pragma unroll
        for (int u = 0; u < 4; ++u) v[u] = ld2(q + u);
        #pragma unroll
        for (int u = 0; u < 4; ++u) { t = max(t, v[u].x); t2 = max(t2, v[u].y); }
    }
    for (; q < q1; ++q) {
        const uint2 v = ld2(q);
        t = max(t, v.x);
        t2 = max(t2, v.y);
    }
    if (any_ry) rx = max(rx, ry + 1);
    return max(max(rx, t), t2);
}

// OR of the high words and maximum of the low words of chunks [q0, q1) of one global row.
// A zero OR means every cell lies in [0, 2^32) and the maximum is the true maximum.
__device__ __forceinline__ void inspect_row_chunks(const int64_t* __restrict__ row, int q0, int q1, int lane,
                                                  unsigned int* or_hi, unsigned int* max_lo) {
    unsigned int acc = 0, m = 0;
    const int64_t* p = row + lane * 2;
    for (int q = q0; q < q1; ++q) {
        const longlong2 v = ld_row_v2<false>(p + q * 64);
        acc |= (unsigned int)((unsigned long long)v.x >> 32) | (unsigned int)((unsigned long long)v.y >> 32);
        m = max(m, max((unsigned int)v.x, (unsigned int)v.y));
    }
    *or_hi = acc;
    *max_lo = m;
}

// ADMIT adds the admission queue of Sec. 4.3.3: every block keeps, for its rows, the number of
// steps above the overload level (the scaler's criterion of Sec. 4.3.2) and publishes with its
// best row whether all its rows are overloaded; when all blocks say so the request that was
// being decided is not routed and the batch stops there: what is left waits or is turned away.
template <bool ADMIT>
__global__ void __launch_bounds__(ROUTE_THREADS, 1) pre_route_persistent(const RouteArgs a) {
    extern __shared__ __align__(16) unsigned char smem_raw[];
    long long* pk = reinterpret_cast<long long*>(smem_raw);  // [2][max_rows] peaks, by exchange parity
    long long* sq = pk + 2 * a.max_rows;                     // queued_p of the owned rows
    long long* scd = sq + a.max_rows;                        // current_d of the owned rows
    // bound[r]: an upper bound of row r's largest cell, or I64_MAX when the row has a cell
    // outside [0, 2^32) (or H is not a multiple of 64); a small bound allows the 32-bit scans.
    long long* bound = scd + a.max_rows;
    // order[L]: the L-th row of the scan order; resident and streamed rows alternate, so that
    // every warp's stretch holds both kinds (a streamed chunk waits far longer for its data)
    int* order = reinterpret_cast<int*>(bound + a.max_rows);
    // rstate[r]: RS_RESIDENT while the row's shared-memory copy is in use, RS_WIDE once the row
    // is known to need 64 bits
    int* rstate = order + a.max_rows;
    // over[r] (ADMIT): steps of row r above the overload level; 64 bytes of fixed words per row then, else 48
    int* over = rstate + a.max_rows;
    unsigned char* res = reinterpret_cast<unsigned char*>(rstate + (ADMIT ? 5 : 1) * a.max_rows);  // 16-byte aligned
    // Words that one warp writes for exchange s while others may still read those of s-1 are kept
    // twice, indexed by the parity of the exchange (or of the arrival being scored): the writer of
    // s+1 never touches what the readers of s use, and s+2 is written only after a block barrier.
    __shared__ int sh_winner[2];
    __shared__ double sh_score[2];
    __shared__ int sh_dead;
    __shared__ unsigned int sh_cut;   // after a lost wait: the last exchange that every block had published
    __shared__ int sh_agreed;         // ... and whether all blocks met to agree on it
    __shared__ long long sh_n0;
    __shared__ long long sh_part[ROUTE_WARPS];  // per-warp peaks of the row that was just folded and re-scored
    __shared__ double sh_best_s[2][2];  // [parity][best, second best]: the block's best scores for the arrival being scored
    __shared__ int sh_best_i[2][2];     // ... and their rows
    __shared__ int sh_cnt[ROUTE_WARPS];   // ADMIT: per-warp change of the folded row's overload count
    __shared__ int sh_n_over;             // ADMIT: rows of this block that are overloaded
    __shared__ int sh_all_over[2];        // ADMIT: every block reported all its rows overloaded (by exchange parity)
    constexpr int RS_RESIDENT = 1, RS_WIDE = 2;

    if (a.done_elsewhere && *a.done_elsewhere) return;   // the same word for every block; nobody writes it meanwhile
    const int G = gridDim.x, b = blockIdx.x;
    const int tid = threadIdx.x, lane = tid & 31, warp = tid >> 5;
    const int I = a.I, H = a.H;
    const unsigned int epoch = *a.epoch_ptr;  // block 0 rewrites it at the very end, after the last exchange
    const int row0 = (int)(((long long)b * I) / G);
    const int row1 = (int)(((long long)(b + 1) * I) / G);
    const int nrows = row1 - row0;
    const int cpr = (H + 63) >> 6;  // 64-cell chunks per row (one 16-byte load per lane)
    const bool full = (H & 63) == 0;
    // Chunk range [c0, c1) of this warp (warps 1..) over the block's rows laid end to end.
    // With few rows each row is cut into `parts` equal stretches and a warp takes exactly one
    // (one reduction per warp and arrival); with many rows the chunks are dealt out evenly.
    const int nch = nrows * cpr;
    int c0 = 0, c1 = 0;
    if (warp) {
        int parts = nrows <= SCAN_WARPS ? SCAN_WARPS / nrows : 0;
        if (parts > cpr) parts = cpr;
        if (parts) {
            const int unit = warp - 1;
            if (unit < nrows * parts) {
                const int row = unit / parts, part = unit - row * parts;
                c0 = row * cpr + (int)((long long)cpr * part / parts);
                c1 = row * cpr + (int)((long long)cpr * (part + 1) / parts);
            }
        } else {
            c0 = (int)((long long)nch * (warp - 1) / SCAN_WARPS);
            c1 = (int)((long long)nch * warp / SCAN_WARPS);
        }
    }
    const int first_row = c0 / cpr, first_q = c0 - first_row * cpr;

    for (int r = tid; r < nrows; r += ROUTE_THREADS) {
        sq[r] = a.queued_p[row0 + r];
        scd[r] = a.current_d[row0 + r];
        pk[r] = I64_MIN;                    // buffer 0, used by the first scan
        bound[r] = full ? 0 : I64_MAX;      // the inspection pass raises it
        rstate[r] = full ? 0 : RS_WIDE;
    }
    if (tid == 0) { sh_dead = 0; sh_n0 = *a.n_requests; }
    __syncthreads();
    // Inspection: which rows hold only values in [0, 2^32), and their maxima.  One pass over the
    // block's rows in global memory.
    if (warp && full) {
        int c = c0, row = first_row, q0 = first_q;
        while (c < c1) {
            const int left = c1 - c;
            const int q1 = (cpr - q0) < left ? cpr : q0 + left;
            unsigned int or_hi, max_lo;
            inspect_row_chunks(a.curves + (size_t)(row0 + row) * H, q0, q1, lane, &or_hi, &max_lo);
            or_hi = __reduce_or_sync(0xffffffffu, or_hi);
            max_lo = __reduce_max_sync(0xffffffffu, max_lo);
            if (lane == 0) {
                if (or_hi) atomicOr(&rstate[row], RS_WIDE);
                atomicMax(&bound[row], (long long)max_lo);
            }
            c += q1 - q0;
            ++row;
            q0 = 0;
        }
    }
    __syncthreads();
    // Resident rows: 32-bit cells when every row of the block fits them (twice as many rows
    // stay on chip), else 64-bit cells.
    bool any_wide = false;
    for (int r = tid; r < nrows; r += ROUTE_THREADS) {
        if (rstate[r] & RS_WIDE) { any_wide = true; bound[r] = I64_MAX; }
    }
    const bool packed = __syncthreads_or(any_wide) == 0;
    const size_t row_bytes = (size_t)H * (packed ? 4 : 8);
    const int S = (int)((size_t)nrows < a.resident_bytes / row_bytes ? (size_t)nrows : a.resident_bytes / row_bytes);
    for (int r = tid; r < nrows; r += ROUTE_THREADS) {
        if (r < S) rstate[r] |= RS_RESIDENT;
        const int pairs = S < nrows - S ? S : nrows - S;   // r-th position of the scan order
        int phys;
        if (r < 2 * pairs) phys = (r & 1) ? S + (r >> 1) : (r >> 1);
        else phys = S <= nrows - S ? r : r - pairs;         // the kind that is left over
        order[r] = phys;
    }
    {
        const int64_t* src = a.curves + (size_t)row0 * H;
        const int total = S * H;
        if (packed) {   // H is a multiple of 64 here
            uint32_t* dst = reinterpret_cast<uint32_t*>(res);
            for (int i = tid * 2; i < total; i += ROUTE_THREADS * 2) {
                const longlong2 v = __ldcg(reinterpret_cast<const longlong2*>(src + i));
                *reinterpret_cast<uint2*>(dst + i) = make_uint2((unsigned int)v.x, (unsigned int)v.y);
            }
        } else {
            int64_t* dst = reinterpret_cast<int64_t*>(res);
            if ((H & 1) == 0) {
                for (int i = tid * 2; i < total; i += ROUTE_THREADS * 2)
                    *reinterpret_cast<longlong2*>(dst + i) = __ldcg(reinterpret_cast<const longlong2*>(src + i));
            } else {
                for (int i = tid; i < total; i += ROUTE_THREADS) dst[i] = __ldcg(src + i);
            }
        }
    }
    __syncthreads();
    if (ADMIT) {   // overload counts of the owned rows, one warp per row and trip
        for (int r = warp; r < nrows; r += ROUTE_WARPS) {
            const int64_t* gp = a.curves + (size_t)(row0 + r) * H;
            int cnt = 0;
            for (int j = lane; j < H; j += 32) cnt += __ldcg(gp + j) > a.hot;
            cnt = __reduce_add_sync(0xffffffffu, cnt);
            if (lane == 0) over[r] = cnt;
        }
        __syncthreads();
        if (tid == 0) {
            int n = 0;
            for (int r = 0; r < nrows; ++r) n += (double)over[r] > a.many;
            sh_n_over = n;
            sh_all_over[0] = sh_all_over[1] = 0;
        }
        __syncthreads();
    }
    const long long n0 = sh_n0;
    long long room = a.max_requests - n0;
    if (room < 0) room = 0;
    // ADMIT: the requests that were waiting when the call was made come first, then the arrivals
    long long q_head = 0, q_len = 0;
    if (ADMIT && a.queue_capacity > 0) {   // kept inside the ring whatever the two words hold
        q_head = a.queue_entry[0];
        q_len = a.queue_entry[1];
        if (q_head < 0 || q_head >= a.queue_capacity) q_head = 0;
        if (q_len < 0) q_len = 0;
        if (q_len > a.queue_capacity) q_len = a.queue_capacity;
    }
    const long long n_items = q_len + a.n_arrivals;
    auto item_prompt = [&](long long k) {
        return (ADMIT && k < q_len) ? a.queue_prompt[(q_head + k) % a.queue_capacity] : a.arr_prompt[k - q_len];
    };
    auto item_predicted = [&](long long k) {
        return (ADMIT && k < q_len) ? a.queue_predicted[(q_head + k) % a.queue_capacity] : a.arr_predicted[k - q_len];
    };
    // where the result of item k goes (block 0, one thread)
    auto put_result = [&](long long k, int c, double sc) {
        if (ADMIT && k < q_len) a.queue_choice[k] = c;
        else {
            a.choice[k - q_len] = c;
            if (a.score) a.score[k - q_len] = sc;
        }
    };
    bool blocked = false;         // ADMIT: the pending request found every instance overloaded
    // Identical in every thread of every block: all take the same decisions.
    long long seq = 0;            // exchanges started so far (= requests appended or pending)
    bool saw_bad = false, saw_full = false;
    long long first_bad = I64_MAX, first_full = I64_MAX;   // the first items dropped as malformed / for a full table
    bool pending = false;         // an arrival has been published but not yet folded
    int pP = 0, pD = 0;           // ... its prompt and predicted lengths
    long long pidx = 0;           // ... its index in the batch

    // Collects the published minima of exchange `s` (warp 0 only); result in sh_winner/sh_score.
    // A block's slot is two 64-bit words, [tag:16 | score bits 63..16] and
    // [tag:16 | score bits 15..0 | row:32], read with one 16-byte request.  Every word carries
    // the low 16 bits of the exchange number, so it is known to be current by itself and relaxed
    // loads suffice: tags are dense across launches (the counter lives on the device), so a
    // slot's previous content is always exactly two exchanges old.  All of a lane's slots are
    // polled at once.
    // `once`: every slot is known to be there already; a missing one is an error, not a reason to wait.
    auto gather = [&](long long s, bool once) {
        const unsigned int tag = epoch + (unsigned int)s;
        const unsigned long long tag16 = (unsigned long long)(tag & 0xffffu);
        const unsigned long long* slot = a.slots + (size_t)(tag & 1u) * G * SLOT_WORDS;
        bool lost = false;
        bool all_over = true;
        double bs = CUDART_INF;
        int bi = 0x7fffffff;
        for (int base = 0; base < G && !lost; base += 32 * GATHER_ILP) {
            unsigned long long w[GATHER_ILP][2];
            unsigned int polls = 0;
            for (;;) {
                bool all = true;
                #pragma unroll
                for (int i = 0; i < GATHER_ILP; ++i) {
                    const int cta = base + lane + 32 * i;
                    if (cta < G) ld_relaxed_v2(&slot[(size_t)cta * SLOT_WORDS], w[i][0], w[i][1]);
                    else w[i][0] = w[i][1] = tag16 << 48;
                }
                #pragma unroll
                for (int i = 0; i < GATHER_ILP; ++i) all &= (w[i][0] >> 48) == tag16 && (w[i][1] >> 48) == tag16;
                if (__all_sync(0xffffffffu, all)) break;
                ++polls;
                const bool give_up = once || polls > a.spin_limit || ((polls & 63u) == 0 && ld_relaxed_s32(a.abort_flag));
                if (__any_sync(0xffffffffu, give_up)) { lost = true; break; }
                if (polls > 256) __nanosleep(64);
            }
            if (lost) break;
            #pragma unroll
            for (int i = 0; i < GATHER_ILP; ++i) {
                const int cta = base + lane + 32 * i;
                if (cta < G) {
                    const unsigned long long bits = (w[i][0] << 16) | ((w[i][1] >> 32) & 0xffffull);
                    const double sc = __longlong_as_double((long long)bits);
                    const int idx = (int)(unsigned int)(w[i][1] & (ADMIT ? 0x7fffffffu : 0xffffffffu));
                    if (ADMIT) all_over &= ((w[i][1] >> 31) & 1ull) != 0;   // bit 31 of the row word
                    if (better(sc, idx, bs, bi)) { bs = sc; bi = idx; }
                }
            }
        }
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
                if (once) sh_agreed = 0;
            }
            sh_winner[s & 1] = bi;
            sh_score[s & 1] = bs;
        }
        if (ADMIT) {
            all_over = __all_sync(0xffffffffu, all_over) && !lost;
            if (lane == 0) sh_all_over[s & 1] = all_over;
        }
    };

    // The winner w of the pending arrival is known: the owner really adds it to row w
    // (Sec. 4.3.1 update), block 0 records it.  When `rescore` is set, the same pass takes the
    // folded row's peak for the arrival being scored now (P, ramp length Dc), one partial per warp in sh_part.
    auto settle = [&](int w, bool rescore, int P, int Dc) {
        if (w >= row0 && w < row1) {
            const int r = w - row0;
            int64_t* gp = a.curves + (size_t)w * H;
            const int pDc = pD < H ? pD : H;
            const int st = rstate[r];
            const bool in_smem = (st & RS_RESIDENT) != 0;
            // a packed row leaves shared memory when the fold may take a cell to 2^32
            const bool evict = in_smem && packed && bound[r] + pP + pDc > 0xffffffffLL;
            uint32_t* sp32 = reinterpret_cast<uint32_t*>(res) + (size_t)r * H;
            int64_t* sp64 = reinterpret_cast<int64_t*>(res) + (size_t)r * H;
            long long pkv = I64_MIN;
            int crossed = 0;   // ADMIT: cells the fold takes above the overload level
            // The usual case in few instructions (all 1,024 threads pass here while every other block
            // waits for this one): a resident row of 32-bit cells that stays below 2^32 with both ramps
            // added; two cells per thread, 32-bit arithmetic, one 16-byte store to the map.
            const bool quick = !ADMIT && in_smem && packed && !evict &&
                               bound[r] + pP + pDc + (long long)P + Dc < 0xffffffffLL;
            if (quick) {
                unsigned int pk32 = 0;
                const int upto = rescore ? H : pDc;       // H is even here (packed rows have whole 64-cell chunks)
                for (int j = 2 * tid; j < upto; j += 2 * ROUTE_THREADS) {
                    uint2 v = *reinterpret_cast<const uint2*>(sp32 + j);
                    if (j < pDc) {
                        v.x += (unsigned int)(pP + j);
                        if (j + 1 < pDc) v.y += (unsigned int)(pP + j + 1);
                        *reinterpret_cast<uint2*>(sp32 + j) = v;
                        *reinterpret_cast<ulonglong2*>(gp + j) = make_ulonglong2(v.x, v.y);
                    }
                    const unsigned int x = v.x + (j < Dc ? (unsigned int)(P + j) : 0u);
                    const unsigned int y = v.y + (j + 1 < Dc ? (unsigned int)(P + j + 1) : 0u);
                    pk32 = max(pk32, max(x, y));
                }
                if (rescore) {
                    pk32 = __reduce_max_sync(0xffffffffu, pk32);
                    if (lane == 0) sh_part[warp] = (long long)pk32;
                }
            } else
            for (int j = tid; j < (rescore ? H : pDc); j += ROUTE_THREADS) {
                long long c = !in_smem ? __ldcg(gp + j) : packed ? (long long)sp32[j] : sp64[j];
                if (j < pDc) {
                    if (ADMIT) crossed -= c > a.hot;
                    c += (long long)pP + j;
                    if (ADMIT) crossed += c > a.hot;
                    gp[j] = c;
                    if (in_smem) {
                        if (!packed) sp64[j] = c;
                        else if (!evict) sp32[j] = (uint32_t)c;
                    }
                }
                pkv = max64(pkv, j < Dc ? c + ((long long)P + j) : c);
            }
            if (rescore && !quick) {   // one partial per warp, reduced by warp 0 after the barrier (no contended atomics)
                pkv = warp_max64(pkv);
                if (lane == 0) sh_part[warp] = pkv;
            }
            if (ADMIT) {
                crossed = __reduce_add_sync(0xffffffffu, crossed);
                if (lane == 0) sh_cnt[warp] = crossed;
            }
            __syncthreads();   // block-uniform branch; every thread has read rstate/bound above
            if (tid == 0) {
                if (ADMIT) {
                    int d = 0;
                    for (int x = 0; x < ROUTE_WARPS; ++x) d += sh_cnt[x];
                    const bool was = (double)over[r] > a.many;
                    over[r] += d;
                    if (!was && (double)over[r] > a.many) sh_n_over += 1;
                }
                if (evict) rstate[r] = st & ~RS_RESIDENT;
                if (bound[r] != I64_MAX) bound[r] += (long long)pP + pDc;  // the ramp adds less than this
                sq[r] += pP;
                scd[r] += pD;
                a.queued_p[w] = sq[r];
                a.current_d[w] = scd[r];
            }
        }
        if (b == 0 && tid == 0) {
            const long long slot = n0 + seq - 1;  // the pending arrival is exchange seq-1
            a.prompt[slot] = pP;
            a.generated[slot] = 0;
            a.predicted[slot] = pD;
            a.instance[slot] = w;
            put_result(pidx, w, sh_score[(seq - 1) & 1]);
        }
    };

    for (long long k = 0; k < n_items; ++k) {
        const int P = item_prompt(k), D = item_predicted(k);
        if (P < 0 || D < 1 || P > PRE_FIELD_MAX || D > PRE_FIELD_MAX) {
            saw_bad = true;
            if (ADMIT && k < first_bad) first_bad = k;
            if (b == 0 && tid == 0) put_result(k, CHOICE_DROPPED, 0.0);
            continue;
        }
        if (seq >= room) {
            saw_full = true;
            if (ADMIT && k < first_full) first_full = k;
            if (b == 0 && tid == 0) put_result(k, CHOICE_DROPPED, 0.0);
            continue;
        }
        const int Dc = D < H ? D : H;
        const int buf = (int)(seq & 1);
        long long* bpk = pk + buf * a.max_rows;

        // ---- 1. scan for arrival k (the pending arrival is not folded yet)
        if (warp != 0) {
            int c = c0, row = first_row, q0 = first_q;
            while (c < c1) {
                const int left = c1 - c;
                const int q1 = (cpr - q0) < left ? cpr : q0 + left;
                const int ph = order[row];
                // every cell with the arrival's ramp added stays below 2^32
                const bool narrow = bound[ph] < (long long)0xffffffffu - P - H;
                const bool in_smem = (rstate[ph] & RS_RESIDENT) != 0;
                const int64_t* gp = a.curves + (size_t)(row0 + ph) * H;
                long long v;
                if (in_smem && packed) {
                    if (narrow) {
                        const uint32_t* rp = reinterpret_cast<const uint32_t*>(res) + (size_t)ph * H;
                        v = (long long)__reduce_max_sync(0xffffffffu, scan_row_chunks_packed(rp, q0, q1, P, Dc, lane));
                    } else {   // this arrival's ramp would overflow 32 bits: take the row from global memory
                        v = warp_max64(scan_row_chunks<true, false>(gp, q0, q1, P, Dc, H, lane));
                    }
                } else if (narrow) {
                    const unsigned int u = in_smem
                        ? scan_row_chunks_narrow<true>(reinterpret_cast<const int64_t*>(res) + (size_t)ph * H, q0, q1, P, Dc, lane)
                        : scan_row_chunks_narrow<false>(gp, q0, q1, P, Dc, lane);
                    v = (long long)__reduce_max_sync(0xffffffffu, u);
                } else {
                    if (in_smem) {
                        const int64_t* rp = reinterpret_cast<const int64_t*>(res) + (size_t)ph * H;
                        v = full ? scan_row_chunks<true, true>(rp, q0, q1, P, Dc, H, lane)
                                 : scan_row_chunks<false, true>(rp, q0, q1, P, Dc, H, lane);
                    } else {
                        v = full ? scan_row_chunks<true, false>(gp, q0, q1, P, Dc, H, lane)
                                 : scan_row_chunks<false, false>(gp, q0, q1, P, Dc, H, lane);
                    }
                    v = warp_max64(v);
                }
                if (lane == 0) {
                    if (q1 - q0 == cpr) bpk[ph] = v;   // the whole row is this warp's
                    else atomicMax(&bpk[ph], v);
                }
                c += q1 - q0;
                ++row;
                q0 = 0;
            }
        }
        // ---- 2. Warp 0 collects the winner of the pending arrival while the scan runs.  When the
        //         scan warps are done (named barrier 1 among warps 1..), warp 1 takes the block's two
        //         best rows for arrival k.  Only the row that receives the pending arrival can still
        //         change, so for every other block the best row found here is final.
        if (warp == 0) {
            if (pending) gather(seq - 1, false);
        } else {
            // an aligned barrier wants the whole warp: the loop above ends in a one-lane branch
            __syncwarp();
            asm volatile("bar.sync 1, %0;" ::"n"(ROUTE_THREADS - 32) : "memory");
            if (warp == 1) {
                double b1s = CUDART_INF, b2s = CUDART_INF;
                int b1i = 0x7fffffff, b2i = 0x7fffffff;
                for (int r = lane; r < nrows; r += 32) {
                    // the peak with the arrival added is an upper bound of the row as it stands
                    if (!(rstate[r] & RS_WIDE)) bound[r] = bpk[r];
                    const double s = score_of(sq[r], scd[r], bpk[r], P, D, a.theta, a.beta);
                    const int i = row0 + r;
                    if (better(s, i, b1s, b1i)) { b2s = b1s; b2i = b1i; b1s = s; b1i = i; }
                    else if (better(s, i, b2s, b2i)) { b2s = s; b2i = i; }
                }
                #pragma unroll
                for (int off = 16; off > 0; off >>= 1) {
                    const double o1s = __shfl_xor_sync(0xffffffffu, b1s, off), o2s = __shfl_xor_sync(0xffffffffu, b2s, off);
                    const int o1i = __shfl_xor_sync(0xffffffffu, b1i, off), o2i = __shfl_xor_sync(0xffffffffu, b2i, off);
                    if (better(o1s, o1i, b1s, b1i)) {
                        // the other side's best wins: second = better(my best, its second)
                        if (better(b1s, b1i, o2s, o2i)) { b2s = b1s; b2i = b1i; } else { b2s = o2s; b2i = o2i; }
                        b1s = o1s; b1i = o1i;
                    } else if (better(o1s, o1i, b2s, b2i)) { b2s = o1s; b2i = o1i; }
                }
                if (lane == 0) { sh_best_s[buf][0] = b1s; sh_best_s[buf][1] = b2s; sh_best_i[buf][0] = b1i; sh_best_i[buf][1] = b2i; }
            } else {
                for (int r = tid - 64; r < nrows; r += ROUTE_THREADS - 64) pk[(buf ^ 1) * a.max_rows + r] = I64_MIN;
            }
        }
        __syncthreads();  // B: winner of the pending arrival known to the block
        if (sh_dead) break;
        if (ADMIT && pending && sh_all_over[(seq - 1) & 1]) { blocked = true; break; }   // the pending request is not routed

        // ---- 3. fold the pending arrival (owner only), publish the block's best row for arrival k
        const int w = sh_winner[(seq - 1) & 1];   // exchange seq-1 decided the pending arrival
        const bool owner = pending && w >= row0 && w < row1;
        if (pending) settle(w, true, P, Dc);   // for the owner: ends with the folded row's peak in sh_part
        if (warp == 0) {
            double b1s = sh_best_s[buf][0];
            int b1i = sh_best_i[buf][0];
            if (owner) {
                // the folded row's score changed: best = better(best of the other rows, folded row)
                __syncwarp();   // lane 0 updated sq/scd of that row inside settle
                const int r = w - row0;
                const long long fixed_peak = warp_max64(sh_part[lane]);
                const double s = score_of(sq[r], scd[r], fixed_peak, P, D, a.theta, a.beta);
                if (b1i == w) { b1s = sh_best_s[buf][1]; b1i = sh_best_i[buf][1]; }
                if (better(s, w, b1s, b1i)) { b1s = s; b1i = w; }
            }
            if (lane == 0) {
                const unsigned int tag = epoch + (unsigned int)seq;  // dense: one tag per exchange
                const unsigned long long tag16 = (unsigned long long)(tag & 0xffffu) << 48;
                unsigned long long* slot = a.slots + ((size_t)(tag & 1u) * G + b) * SLOT_WORDS;
                const unsigned long long bits = (unsigned long long)__double_as_longlong(b1s);
                // ADMIT: bit 31 of the row word says that every row of this block is overloaded (lane 0 is the
                // thread that keeps sh_n_over, so it sees its own latest update)
                const unsigned int flag = (ADMIT && sh_n_over == nrows) ? 0x80000000u : 0u;
                st_relaxed_v2(slot, tag16 | (bits >> 16), tag16 | ((bits & 0xffffull) << 32) | flag | (unsigned int)b1i);
            }
        }
        if (owner) __syncthreads();  // C: nobody scans the folded row before the fold is complete
        pending = true; pP = P; pD = D; pidx = k;
        ++seq;
        // No barrier here for the other blocks: their warps go on to the next scan (which fills
        // the other peak buffer) while warp 0 publishes.
    }

    // ---- the last arrival is still pending
    if (pending && !sh_dead && !blocked) {
        __syncthreads();
        if (warp == 0) gather(seq - 1, false);
        __syncthreads();
        if (ADMIT && !sh_dead && sh_all_over[(seq - 1) & 1]) blocked = true;
        if (!sh_dead && !blocked) settle(sh_winner[(seq - 1) & 1], false, 0, 0);
    }

    // ---- A wait ran out, here or in another block (every block ends up here then: the block that
    // gave up publishes nothing more, so nobody gets past the next exchange).  The blocks meet and
    // agree on m, the smallest exchange at which any of them gave up.  Every block had published m
    // before it could wait for it, so a block that gave up at m reads the slots of m once more, now
    // complete, and settles m like the blocks that got one exchange further.  Requests up to the one
    // of exchange m are routed and folded everywhere, nothing after it is.
    const bool dead = sh_dead != 0;
    long long settled = (dead || blocked) && pending ? seq - 1 : seq;    // requests really added, as this block sees it
    long long undone_from = dead ? pidx : n_items;                       // first item that gets no decision
    unsigned int next_epoch = epoch + (unsigned int)seq;
    if (dead) {
        const unsigned int lost_s = (unsigned int)(seq - 1);     // the exchange whose slots did not all arrive here
        if (tid == 0) {
            atomicMax(a.abort_key, 0xffffffffu - lost_s);
            __threadfence();
            atomicAdd(a.abort_count, 1u);
            bool met = true;
            unsigned int polls = 0;
            while (ld_relaxed_u32(a.abort_count) < (unsigned int)G) {
                if (++polls > ABORT_SPIN_LIMIT) { met = false; break; }
                __nanosleep(200);
            }
            __threadfence();
            sh_cut = 0xffffffffu - ld_relaxed_u32(a.abort_key);
            sh_agreed = met ? 1 : 0;
        }
        __syncthreads();
        const unsigned int m = sh_cut;
        if (sh_agreed) {
            next_epoch = epoch + m + 2u;      // past every tag this launch may have left in a slot
            if (lost_s == m) {
                if (warp == 0) gather((long long)m, true);
                __syncthreads();
                if (sh_agreed) {
                    if (ADMIT && sh_all_over[m & 1]) {
                        blocked = true;
                    } else {
                        settle(sh_winner[m & 1], false, 0, 0);
                        settled = seq;
                        undone_from = pidx + 1;
                    }
                }
            }
        }
        // (without agreement - a block that never came - the maps may hold one request more than the
        // table: PRE_ETIMEOUT then means that the state has to be rebuilt)
    }

    if (b == 0 && tid == 0) {
        *a.n_requests = n0 + settled;
        *a.epoch_ptr = next_epoch;
        // what the loop noted beyond a blocked request is decided again below and does not count here
        const long long decided = (ADMIT && blocked) ? pidx : n_items;
        if (saw_bad && (!ADMIT || first_bad < decided)) atomicOr(a.status, PRE_ST_BADREQ);
        if (saw_full && (!ADMIT || first_full < decided)) atomicOr(a.status, PRE_ST_CAPACITY);
    }

    if (!ADMIT && b == 0 && dead) {
        for (long long k = undone_from + tid; k < n_items; k += ROUTE_THREADS) put_result(k, CHOICE_DROPPED, 0.0);
    }

    if (ADMIT && b == 0) {
        // Everything from the blocked request on: a request that was waiting keeps its place; an
        // arrival joins the tail of the queue while there is room and is turned away otherwise
        // (a malformed arrival is dropped).  Nothing else reads or writes these arrays any more:
        // the other blocks only look at items up to the one they are scanning, whose fields they
        // read before the exchange that stopped the batch.
        __syncthreads();
        const bool lost = dead;
        // after a lost wait nothing more is decided: waiting requests keep their place, arrivals are dropped
        const long long stop = blocked ? pidx : (lost ? undone_from : n_items);
        const long long left = stop < q_len ? q_len - stop : 0;          // waiting entries that stay
        for (long long k = stop + tid; k < q_len; k += ROUTE_THREADS) a.queue_choice[k] = CHOICE_WAITS;
        __shared__ long long sh_joined;
        __shared__ int sh_warp_ok[ROUTE_WARPS];
        __shared__ int sh_any_bad;
        if (tid == 0) { sh_joined = 0; sh_any_bad = 0; }
        __syncthreads();
        const long long a0 = (stop > q_len ? stop : q_len) - q_len;      // first arrival that was not decided
        for (long long base = a0; base < a.n_arrivals && !lost; base += ROUTE_THREADS) {
            const long long i = base + tid;
            int P = -1, D = 0;
            if (i < a.n_arrivals) { P = a.arr_prompt[i]; D = a.arr_predicted[i]; }
            const bool ok = i < a.n_arrivals && !(P < 0 || D < 1 || P > PRE_FIELD_MAX || D > PRE_FIELD_MAX);
            const unsigned int vote = __ballot_sync(0xffffffffu, ok);
            if (lane == 0) sh_warp_ok[warp] = __popc(vote);
            __syncthreads();
            long long rank = sh_joined + __popc(vote & ((1u << lane) - 1u));
            int total = 0;
            for (int x = 0; x < ROUTE_WARPS; ++x) { if (x < warp) rank += sh_warp_ok[x]; total += sh_warp_ok[x]; }
            if (i < a.n_arrivals) {
                int c = CHOICE_DROPPED;
                if (ok) {
                    if (left + rank < a.queue_capacity) {
                        const long long pos = (q_head + q_len + rank) % a.queue_capacity;   // behind the last one waiting
                        a.queue_prompt[pos] = P;
                        a.queue_predicted[pos] = D;
                        c = CHOICE_WAITS;
                    } else {
                        c = CHOICE_TURNED_AWAY;
                    }
                } else {
                    sh_any_bad = 1;
                }
                a.choice[i] = c;
                if (a.score) a.score[i] = 0.0;
            }
            __syncthreads();
            if (tid == 0) sh_joined += total;
            __syncthreads();
        }
        for (long long i = a0 + tid; i < a.n_arrivals && lost; i += ROUTE_THREADS) {
            a.choice[i] = CHOICE_DROPPED;
            if (a.score) a.score[i] = 0.0;
        }
        if (tid == 0) {
            long long joined = lost ? 0 : sh_joined;
            if (left + joined > a.queue_capacity) joined = a.queue_capacity - left;
            a.queue_state[0] = a.queue_capacity > 0 ? (q_head + (q_len - left)) % a.queue_capacity : 0;
            a.queue_state[1] = left + joined;
            if (blocked && sh_any_bad) atomicOr(a.status, PRE_ST_BADREQ);
        }
    }
}

}  // namespace

// Shared-memory split of one instantiation: `fixed_per_row` bytes of per-row words, the rest for resident rows.
template <bool ADMIT>
static cudaError_t configure_one(pre_ctx* ctx, int G, int max_rows, size_t limit, size_t* smem_out,
                                 size_t* resident_out) {
    const int H = ctx->cfg.horizon;
    const size_t fixed = (size_t)max_rows * (ADMIT ? 64 : 48);  // five 8-byte and two 4-byte words per row (+ the overload count)
    cudaFuncAttributes attr;
    cudaError_t e = cudaFuncGetAttributes(&attr, pre_route_persistent<ADMIT>);
    if (e != cudaSuccess) return e;
    const size_t spare = 256;   // left unused; the occupancy query below confirms that the block still fits
    if (fixed + attr.sharedSizeBytes + spare > limit) return cudaErrorInvalidConfiguration;
    // what is left beside the fixed part holds resident rows (the kernel decides how many)
    size_t resident_bytes = limit - attr.sharedSizeBytes - spare - fixed;
    if (resident_bytes > (size_t)max_rows * H * sizeof(int64_t)) resident_bytes = (size_t)max_rows * H * sizeof(int64_t);
    resident_bytes &= ~(size_t)15;
    const size_t smem = fixed + resident_bytes;
    // (the limit is shared by every context of the process: always the device maximum)
    e = cudaFuncSetAttribute(pre_route_persistent<ADMIT>, cudaFuncAttributeMaxDynamicSharedMemorySize,
                             (int)(limit - attr.sharedSizeBytes));
    if (e != cudaSuccess) return e;
    int per_sm = 0;
    e = cudaOccupancyMaxActiveBlocksPerMultiprocessor(&per_sm, pre_route_persistent<ADMIT>, ROUTE_THREADS, smem);
    if (e != cudaSuccess) return e;
    if (per_sm < 1) return cudaErrorInvalidConfiguration;
    (void)G;
    *smem_out = smem;
    *resident_out = resident_bytes;
    return cudaSuccess;
}

cudaError_t pre_route_configure(pre_ctx* ctx) {
    const int I = ctx->cfg.n_instances;
    const int G = ctx->n_sm < I ? ctx->n_sm : I;  // one block per SM, never more blocks than rows
    const int max_rows = (I + G - 1) / G;
    cudaDeviceProp prop;
    cudaError_t e = cudaGetDeviceProperties(&prop, ctx->device);
    if (e != cudaSuccess) return e;
    const size_t limit = (size_t)prop.sharedMemPerBlockOptin;
    e = configure_one<false>(ctx, G, max_rows, limit, &ctx->route_smem, &ctx->route_resident_bytes);
    if (e != cudaSuccess) return e;
    e = configure_one<true>(ctx, G, max_rows, limit, &ctx->route_smem_admit, &ctx->route_resident_bytes_admit);
    if (e != cudaSuccess) return e;
    ctx->route_blocks = G;
    ctx->route_threads = ROUTE_THREADS;
    return cudaSuccess;
}

static void fill_route_args(RouteArgs& a, pre_ctx* ctx, const int32_t* arr_prompt, const int32_t* arr_predicted,
                            int64_t n_arrivals, int64_t* curves, int64_t* queued_p, int64_t* current_d,
                            int32_t* prompt, int32_t* generated, int32_t* predicted, int32_t* instance,
                            int64_t* n_requests, int32_t* choice, double* score) {
    a.arr_prompt = arr_prompt; a.arr_predicted = arr_predicted; a.n_arrivals = n_arrivals;
    a.curves = curves; a.queued_p = queued_p; a.current_d = current_d;
    a.prompt = prompt; a.generated = generated; a.predicted = predicted; a.instance = instance;
    a.n_requests = n_requests; a.max_requests = ctx->cfg.max_requests;
    a.choice = choice; a.score = score;
    a.I = ctx->cfg.n_instances; a.H = ctx->cfg.horizon;
    a.theta = ctx->theta; a.beta = ctx->cfg.beta;
    a.slots = ctx->d_slots; a.epoch_ptr = ctx->d_epoch;
    a.status = ctx->d_status; a.abort_flag = ctx->d_abort;
    a.abort_key = reinterpret_cast<unsigned int*>(ctx->d_abort + 1);
    a.abort_count = reinterpret_cast<unsigned int*>(ctx->d_abort + 2);
    a.spin_limit = ctx->spin_limit;
    a.done_elsewhere = nullptr;
    a.max_rows = (a.I + ctx->route_blocks - 1) / ctx->route_blocks;
    a.resident_bytes = ctx->route_resident_bytes;
    a.queue_prompt = nullptr; a.queue_predicted = nullptr; a.queue_state = nullptr; a.queue_entry = nullptr;
    a.queue_capacity = 0; a.queue_choice = nullptr; a.hot = 0; a.many = 0.0;
}

// PRE_ROUTE_AUTO takes the summary kernel when its scores are whole numbers (beta and t_mem * M whole: one
// integer pass per arrival); with binary64 scores its chains of binary64 operations leave it level with the
// scanning kernel (measured: 2.83 against 3.12 us per arrival on 4,096 x 2,048 instances x steps, 2.57 against
// 2.43 on 1,024 x 1,024), so it runs them only when it is selected outright.
static bool pre_route_summary_wanted(const pre_ctx* ctx) {
    if (ctx->route_path == PRE_ROUTE_SCAN) return false;
    if (ctx->route_path == PRE_ROUTE_SUMMARY) return true;
    const double beta = ctx->cfg.beta, theta = ctx->theta;
    return beta == floor(beta) && theta == floor(theta) && beta <= 1048576.0 && theta < 1073741824.0;
}

cudaError_t pre_launch_route(pre_ctx* ctx, const int32_t* arr_prompt, const int32_t* arr_predicted,
                             int64_t n_arrivals, int64_t* curves, int64_t* queued_p, int64_t* current_d,
                             int32_t* prompt, int32_t* generated, int32_t* predicted, int32_t* instance,
                             int64_t* n_requests, int32_t* choice, double* score, cudaStream_t s) {
    if (n_arrivals == 0) return cudaSuccess;
    // The summary kernel takes the batch when the shape fits it; it declines (on the device) when 32-bit
    // arithmetic could overflow during the batch, and the scanning kernel launched behind it then does
    // the work.  When the summary kernel has routed the batch the scanning kernel returns at once.
    const bool summaries = pre_route_summary_wanted(ctx) && pre_route_summary_fits(ctx);
    cudaError_t e = cudaSuccess;
    if (summaries) {
        e = pre_launch_route_summary(ctx, arr_prompt, arr_predicted, n_arrivals, curves, queued_p, current_d, prompt,
                                     generated, predicted, instance, n_requests, choice, score, s);
        if (e != cudaSuccess) return e;
    }
    e = cudaMemsetAsync(ctx->d_abort, 0, 3 * sizeof(int), s);   // flag, agreed exchange, blocks met
    if (e != cudaSuccess) return e;
    RouteArgs a;
    fill_route_args(a, ctx, arr_prompt, arr_predicted, n_arrivals, curves, queued_p, current_d, prompt, generated,
                    predicted, instance, n_requests, choice, score);
    if (summaries) a.done_elsewhere = ctx->d_rs_handled;
    void* params[] = {(void*)&a};
    return cudaLaunchCooperativeKernel((const void*)pre_route_persistent<false>, dim3(ctx->route_blocks),
                                       dim3(ROUTE_THREADS), params, ctx->route_smem, s);
}

cudaError_t pre_launch_route_admit(pre_ctx* ctx, const int32_t* arr_prompt, const int32_t* arr_predicted,
                                   int64_t n_arrivals, double overload_level, double overload_share,
                                   int32_t* queue_prompt, int32_t* queue_predicted, int64_t* queue_state,
                                   int64_t queue_capacity, int32_t* queue_choice, int64_t* curves,
                                   int64_t* queued_p, int64_t* current_d, int32_t* prompt, int32_t* generated,
                                   int32_t* predicted, int32_t* instance, int64_t* n_requests, int32_t* choice,
                                   double* score, cudaStream_t s) {
    // The kernel's blocks read the queue's head and length while block 0 may already be writing the
    // new ones: they read a copy taken here, in stream order.
    cudaError_t e = cudaMemcpyAsync(ctx->d_queue_entry, queue_state, 2 * sizeof(int64_t), cudaMemcpyDeviceToDevice, s);
    if (e != cudaSuccess) return e;
    // For a whole number c, c > x holds exactly when c > floor(x): the per-cell test is done on integers.
    double hot = floor(overload_level * (double)ctx->cfg.capacity_tokens);
    if (hot > 9.2e18) hot = 9.2e18;
    if (hot < -9.2e18) hot = -9.2e18;
    const double many = overload_share * (double)ctx->cfg.horizon;
    // as for pre_route_batch: the summary kernel first where the shape fits it, the scanning kernel behind it
    const bool summaries = pre_route_summary_wanted(ctx) && pre_route_summary_admit_fits(ctx);
    if (summaries) {
        e = pre_launch_route_summary_admit(ctx, arr_prompt, arr_predicted, n_arrivals, (long long)hot, many, queue_prompt,
                                           queue_predicted, queue_state, queue_capacity, queue_choice, curves, queued_p,
                                           current_d, prompt, generated, predicted, instance, n_requests, choice, score,
                                           s);
        if (e != cudaSuccess) return e;
    }
    e = cudaMemsetAsync(ctx->d_abort, 0, 3 * sizeof(int), s);
    if (e != cudaSuccess) return e;
    RouteArgs a;
    fill_route_args(a, ctx, arr_prompt, arr_predicted, n_arrivals, curves, queued_p, current_d, prompt, generated,
                    predicted, instance, n_requests, choice, score);
    if (summaries) a.done_elsewhere = ctx->d_rs_handled;
    a.resident_bytes = ctx->route_resident_bytes_admit;
    a.queue_prompt = queue_prompt; a.queue_predicted = queue_predicted; a.queue_state = queue_state;
    a.queue_entry = ctx->d_queue_entry; a.queue_capacity = queue_capacity; a.queue_choice = queue_choice;
    a.hot = (long long)hot;
    a.many = many;
    void* params[] = {(void*)&a};
    return cudaLaunchCooperativeKernel((const void*)pre_route_persistent<true>, dim3(ctx->route_blocks),
                                       dim3(ROUTE_THREADS), params, ctx->route_smem_admit, s);
}

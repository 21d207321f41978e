// Load-aware request router (paper Sec. 4.3.3) on per-row summaries of the maps.
//
// The score of an arrival (P, D) against a row c[0..H) needs one number of the row, the peak
// of the map with the arrival's ramp added (Sec. 4.3.1 update), Dc = min(D, H):
//     peak = max( max_{j<Dc}(c[j] + P + j),  max_{j>=Dc} c[j] ).
// Four numbers per row decide it without reading the row in almost every case:
//     top  = max_j (c[j] + j)          jtop = the first step where that maximum is taken
//     rmax = max_j c[j]                c0   = c[0]
//   * Dc > jtop:  the ramp covers the step of the maximum, so max_{j<Dc}(c[j]+j) = top; and
//                 P + top >= c[j] for every j, so   peak = P + top   exactly;
//   * otherwise:  max(rmax, P + c0) <= peak <= P + top   (the ramp covers step 0; top bounds every step).
// In maps of requests that are being decoded the occupancy falls as requests finish, the maximum
// of c[j] + j sits at the first steps, and the first case is the rule.  The kernel never relies on
// that: a row that is only bounded and could hold the smallest score is scanned cell by cell.
//
// Two kernels per batch:
//   pre_summarise_rows   one pass over the maps: the four numbers of every row, the rows' token
//                        counts (queued_p + current_d) and the guards that tell whether 32-bit
//                        arithmetic stays exact for the whole batch;
//   pre_route_summaries  routes the batch with ONE block: summaries in shared memory, no exchange
//                        between blocks, hence no device-side wait on another block anywhere.
//
// pre_route_summaries works in rounds, one arrival and two block barriers per round, three groups of warps:
//   score warps:  every row's score for the arrival from its summary; the warp's smallest score by a
//                 warp reduction, the block's smallest (score, row) by a shared-memory atomic minimum
//                 (whole-number scores) or one (score, row) per warp (binary64 scores);
//   control warp: before the first barrier it writes the last decision's outputs, takes the pending
//                 rows' lower bounds and walks to the next well-formed arrival; between the barriers
//                 it decides: the pass's best row unless a pending row could do better;
//   fold warps:   add an arrival to its row in the map (Sec. 4.3.1 update) and take the row's new
//                 summary in the same pass - RS_LAG rounds after the decision, so that the row's
//                 cells can be fetched a round ahead and no decision waits for a fold.
// The instances' token counts (Sec. 4.3.3: queued prompt tokens, tokens being decoded) are brought up
// to date once, after the last round, from the new table rows.
// Between its decision and its fold a row is "pending": it is left out of the scoring pass and
// represented by a lower bound of its score (its token count is exact at once; the cell that
// held `top` only grows).  A pending row whose lower bound could win makes the round a stall:
// nothing is decided, the folds go on, and the arrival is decided once the row is exact again.
// The decisions are therefore the same as with every fold done at once.
#include "pre_common.cuh"

#include <math_constants.h>

#include <cmath>

namespace {

constexpr int RS_FOLD_WARPS = 8;
constexpr int RS_FOLD_THREADS = 32 * RS_FOLD_WARPS;
constexpr int RS_CONTROL_WARP = RS_FOLD_WARPS;     // the warp after the fold warps decides; the score warps follow it
constexpr int RS_MAX_SCORE_WARPS = 10;      // 640 threads with the fold and control warps: 96 registers per thread, no spills
constexpr int RS_MAX_THREADS = RS_FOLD_THREADS + 32 + 32 * RS_MAX_SCORE_WARPS;
#ifndef PRE_RS_LAG
#define PRE_RS_LAG 3
#endif
constexpr int RS_LAG = PRE_RS_LAG;         // rounds between a decision and the fold of its row
constexpr int RS_PENDING = RS_LAG + 1;     // rows that can be pending at once (and row slots in shared memory)
// Distance between the binary32 estimate of a score and the binary64 score, relative to
// estimate + 2 * beta * theta: eight roundings of 2^-24 each on terms that add up to at most that
// (2^-21), taken four times as large.
constexpr float RS_EPS = 1.9073486328125e-06f;   // 2^-19
constexpr int RS_ROWS_PER_LANE = 16;       // rows of one score lane at most (the host picks the score warps accordingly)
constexpr int SUM_THREADS = 256;
// whole-number scores: token count of a row that is left out of the pass (pending, or padding)
constexpr unsigned int RS_OUT = 0xc0000000u;

// named barriers (0 is __syncthreads)

// guard words written by the summarising kernel
constexpr int GUARD_MAX_CELL = 0, GUARD_MAX_BASE = 1, GUARD_BAD = 2, GUARD_SUM_RAMP = 3, GUARD_SUM_TOKENS = 4,
              GUARD_MAX_PD = 5, GUARD_MAX_JTOP = 6;

struct __align__(16) Item {
    int P, D, Dc;
    int k;   // index in the batch; -1: the batch has ended
};

// {token count, rmax, top, c0} of a row; jtop is kept beside it
typedef uint4 RowSummary;

// A row between its decision and its fold.
struct __align__(16) Pending {
    int row;                 // -1: free
    int P, D, Dc;            // the arrival that goes into it
    unsigned int tokens;     // token count with the arrival (exact)
    unsigned int top_lb;     // cell jw + jw with the arrival added: a lower bound of the new top
    unsigned int jw;         // the step of that cell (the old jtop)
    unsigned int rmax;       // old largest cell: a lower bound of the new one
    unsigned int c0;         // cell 0 with the arrival added (exact)
    unsigned int unused[3];  // (three 16-byte stores write an entry)
};

__device__ __forceinline__ void cp_async4(void* smem_dst, const void* gsrc) {
    const unsigned int d = (unsigned int)__cvta_generic_to_shared(smem_dst);
    asm volatile("cp.async.ca.shared.global [%0], [%1], 4;" ::"r"(d), "l"(gsrc) : "memory");
}
__device__ __forceinline__ void cp_async_commit() { asm volatile("cp.async.commit_group;" ::: "memory"); }
__device__ __forceinline__ unsigned int warp_max_u32(unsigned int v) {
    #pragma unroll
    for (int off = 16; off > 0; off >>= 1) v = max(v, __shfl_xor_sync(0xffffffffu, v, off));
    return v;
}


// Score of one instance, binary64, every operation rounded on its own (the sums of whole
// numbers below 2^53 are exact, so adding the two token counts first changes nothing).
__device__ __forceinline__ double summary_score(unsigned int tokens, unsigned int peak, int P, int D, double theta,
                                                double beta) {
    double over = __dsub_rn((double)peak, theta);
    if (over < 0.0) over = 0.0;
    const double l = (double)((unsigned long long)tokens + (unsigned long long)P + (unsigned long long)D);
    return __dadd_rn(l, __dmul_rn(beta, over));
}

__device__ __forceinline__ bool better_row(double s, int i, double bs, int bi) {
    return s < bs || (s == bs && i < bi);
}

struct SumArgs {
    const int64_t* curves;
    const int64_t* queued_p;
    const int64_t* current_d;
    const int32_t* arr_prompt;
    const int32_t* arr_predicted;
    long long n_arrivals;
    int I, H;
    RowSummary* summary;
    uint32_t* jtop;
    unsigned long long* guard;
    // admission queue (pre_route_admit): steps above the overload level per row, the waiting requests' totals
    int32_t* over;                 // NULL: not wanted
    long long hot;
    const int32_t* queue_prompt;
    const int32_t* queue_predicted;
    const int64_t* queue_entry;    // {head, length} as they were when the call was made
    long long queue_capacity;
};

// One warp per row.
__global__ void __launch_bounds__(SUM_THREADS) pre_summarise_rows(const SumArgs a) {
    const int tid = threadIdx.x, lane = tid & 31;
    const int row = blockIdx.x * (SUM_THREADS / 32) + (tid >> 5);
    const int H = a.H;
    bool bad = false;
    if (row < a.I) {
        const int64_t* src = a.curves + (size_t)row * H;
        unsigned int rmax = 0, top = 0, jtop = 0;
        int above = 0;
        auto take = [&](long long v, int j) {
            above += v > a.hot;
            bad |= (v < 0) || (v > 0xffffffffLL);
            const unsigned int c = (unsigned int)v;
            rmax = max(rmax, c);
            const unsigned long long t = (unsigned long long)c + (unsigned long long)j;
            if (t > 0xffffffffull) bad = true;
            if ((unsigned int)t > top) { top = (unsigned int)t; jtop = (unsigned int)j; }   // a lane's steps ascend
        };
        if ((H & 1) == 0) {
            for (int j = 2 * lane; j < H; j += 64) {
                const longlong2 v = __ldcs(reinterpret_cast<const longlong2*>(src + j));
                take(v.x, j);
                take(v.y, j + 1);
            }
        } else {
            for (int j = lane; j < H; j += 32) take(__ldcs(src + j), j);
        }
        rmax = __reduce_max_sync(0xffffffffu, rmax);
        const unsigned int t = __reduce_max_sync(0xffffffffu, top);
        const unsigned int jt = __reduce_min_sync(0xffffffffu, top == t ? jtop : 0xffffffffu);
        above = __reduce_add_sync(0xffffffffu, above);
        if (lane == 0 && a.over) a.over[row] = above;
        if (lane == 0) {
            const long long q = a.queued_p[row], d = a.current_d[row];
            const long long tok = q + d;
            const bool ok = q >= 0 && d >= 0 && q <= 0xffffffffLL && d <= 0xffffffffLL && tok <= 0xffffffffLL;
            if (!ok) bad = true;
            a.summary[row] = make_uint4(ok ? (unsigned int)tok : 0u, rmax, t, (unsigned int)src[0]);
            a.jtop[row] = jt;
            if (ok) atomicMax(a.guard + GUARD_MAX_BASE, (unsigned long long)tok);
            if (rmax) atomicMax(a.guard + GUARD_MAX_CELL, (unsigned long long)rmax);
            if (jt) atomicMax(a.guard + GUARD_MAX_JTOP, (unsigned long long)jt);
        }
    }
    if (__any_sync(0xffffffffu, bad) && lane == 0) atomicOr(a.guard + GUARD_BAD, 1ull);
    // the arrivals' own totals: what the batch can add to a cell (ramps) and to a row's token count
    unsigned long long ramp = 0, tokens = 0;
    unsigned int max_pd = 0;
    auto count = [&](int P, int D) {
        if (P < 0 || D < 1 || P > PRE_FIELD_MAX || D > PRE_FIELD_MAX) return;
        ramp += (unsigned long long)P + (unsigned long long)(D < H ? D : H);
        tokens += (unsigned long long)P + (unsigned long long)D;
        max_pd = max(max_pd, (unsigned int)P + (unsigned int)D);
    };
    for (long long k = (long long)blockIdx.x * SUM_THREADS + tid; k < a.n_arrivals; k += (long long)gridDim.x * SUM_THREADS)
        count(a.arr_prompt[k], a.arr_predicted[k]);
    if (a.queue_capacity > 0) {   // the waiting requests are routed before the arrivals
        long long q_head = a.queue_entry[0], q_len = a.queue_entry[1];
        if (q_head < 0 || q_head >= a.queue_capacity) q_head = 0;
        if (q_len < 0) q_len = 0;
        if (q_len > a.queue_capacity) q_len = a.queue_capacity;
        for (long long k = (long long)blockIdx.x * SUM_THREADS + tid; k < q_len; k += (long long)gridDim.x * SUM_THREADS) {
            const long long at = (q_head + k) % a.queue_capacity;
            count(a.queue_prompt[at], a.queue_predicted[at]);
        }
    }
    #pragma unroll
    for (int off = 16; off > 0; off >>= 1) {
        ramp += __shfl_xor_sync(0xffffffffu, ramp, off);
        tokens += __shfl_xor_sync(0xffffffffu, tokens, off);
    }
    max_pd = __reduce_max_sync(0xffffffffu, max_pd);
    if (lane == 0 && (ramp | tokens)) {
        atomicAdd(a.guard + GUARD_SUM_RAMP, ramp);
        atomicAdd(a.guard + GUARD_SUM_TOKENS, tokens);
        atomicMax(a.guard + GUARD_MAX_PD, (unsigned long long)max_pd);
    }
}

struct RouteSumArgs {
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
    const RowSummary* summary0;
    const uint32_t* jtop0;
    const unsigned long long* guard;
    int* status;
    int* handled;   // 1: this kernel routed the batch; 0: the scanning kernel has to
    int score_warps;
    // admission queue (ADMIT kernels only): a ring of waiting requests, entry q at (head + q) mod capacity
    int32_t* queue_prompt;
    int32_t* queue_predicted;
    int64_t* queue_state;          // {head, length}, rewritten at the end
    const int64_t* queue_entry;    // the same two words as they were when the call was made
    long long queue_capacity;
    int32_t* queue_choice;         // results for the entries that were waiting at entry
    long long hot;                 // floor(overload_level * M): a cell counts when it is above
    double many;                   // overload_share * H: overloaded when more cells than this count
    const int32_t* over0;          // [I] steps above the level per row, from the summarising kernel
};


// CPT: cells of the folded row per fold thread (H <= CPT * RS_FOLD_THREADS).
// VEC: H is even, so 16-byte accesses to the rows are legal.
// The block has RS_FOLD_WARPS fold warps, the control warp and a.score_warps score warps.
// ADMIT adds the admission queue of Sec. 4.3.3: the requests that were waiting come first; a request that
// finds every instance overloaded (the scaler's criterion of Sec. 4.3.2: more than `many` steps of the
// row above `hot`) is not routed and the batch stops there: what is left waits or is turned away.
// KIND: which scores the instantiation takes, chosen by the host from beta and theta (measured: with both kinds in
// one kernel and the choice made at run time the whole-number rounds take 6 % longer, 8 % with the queue):
//   RS_WHOLE      whole-number scores (beta and theta whole numbers); the kernel declines the batch when the
//                 device-side bounds do not keep every score below 2^30;
//   RS_WHOLE_BIG  the same for more than RS_ROWS_PER_LANE rows per score lane (contexts of more than 5,120
//                 instances): the pass goes on beyond its unrolled part;
//   RS_BINARY64   binary64 scores, RS_ROWS_PER_LANE rows per score lane at most.
constexpr int RS_WHOLE = 0, RS_WHOLE_BIG = 1, RS_BINARY64 = 2;
template <int CPT, bool VEC, bool ADMIT, int KIND>
__global__ void __launch_bounds__(RS_MAX_THREADS, 1) pre_route_summaries(const RouteSumArgs a) {
    constexpr bool BIG = KIND == RS_WHOLE_BIG;
    constexpr bool whole = KIND != RS_BINARY64;
    extern __shared__ __align__(16) unsigned char rs_smem[];
    const int I = a.I, H = a.H;
    const int Ip = (I + 31) & ~31;
    uint2* tt = reinterpret_cast<uint2*>(rs_smem);          // [Ip] {token count (RS_OUT: left out of the pass), top}
    uint2* aux = tt + Ip;                                   // [Ip] {rmax, c0}
    uint32_t* jst = reinterpret_cast<uint32_t*>(aux + Ip);  // [Ip] jtop
    int* over = reinterpret_cast<int*>(jst + Ip);           // [Ip] ADMIT: steps of the row above the overload level
    __shared__ Item sh_item[2];             // the arrival to decide, by round parity
    __shared__ int sh_decided[2];           // whether the round decided its arrival
    __shared__ Pending pend[RS_PENDING];
    __shared__ unsigned long long sh_wkey[2][RS_MAX_SCORE_WARPS];   // binary64 scores: the warps' best rows, score bits
    __shared__ unsigned long long sh_best[2];   // whole-number scores: the smallest score << 32 | row of all warps (atomic minimum)
    __shared__ int sh_wrow[2][RS_MAX_SCORE_WARPS];
    __shared__ uint4 sh_fold[RS_FOLD_WARPS];   // per fold warp {rmax, top, jtop, -}
    __shared__ unsigned int sh_jmax;        // no row's jtop is larger
    __shared__ int sh_mode;                 // 0: decline the batch
    __shared__ long long sh_n0;
    __shared__ int sh_arr_p[64], sh_arr_d[64];   // the arrivals around the walker's position
    __shared__ int sh_n_over;               // ADMIT: rows known to be overloaded
    __shared__ int sh_blocked;              // ADMIT: a request found every instance overloaded ...
    __shared__ long long sh_blocked_k;      // ... this one
    __shared__ int sh_warp_ok[RS_MAX_THREADS / 32];   // (the tail of ADMIT)
    __shared__ long long sh_joined;
    __shared__ int sh_any_bad;

    const int tid = threadIdx.x, lane = tid & 31, warp = tid >> 5;
    const int nsw = a.score_warps, nst = 32 * nsw, nthreads = RS_FOLD_THREADS + 32 + nst;
    const double theta = a.theta, beta = a.beta;
    if (tid == 0) {
        const unsigned long long mc = a.guard[GUARD_MAX_CELL], mb = a.guard[GUARD_MAX_BASE];
        // every cell, every cell + step with a prompt added, and every token count stay below 2^32 all batch long
        const unsigned long long peak_bound = mc + a.guard[GUARD_SUM_RAMP] + (unsigned long long)H + (unsigned long long)PRE_FIELD_MAX;
        const unsigned long long token_bound = mb + a.guard[GUARD_SUM_TOKENS];
        // (and the batch is short enough for the round counters below to be 32-bit numbers)
        const bool ok = a.guard[GUARD_BAD] == 0 && peak_bound <= 0xffffffffull && token_bound < (unsigned long long)RS_OUT &&
                        a.n_arrivals + (ADMIT ? a.queue_capacity : 0) < (1ll << 26);
        // Whole-number scores: with beta and theta whole numbers every term of the score is a whole number
        // below 2^53, each binary64 operation is exact, and the score is the same number in integer
        // arithmetic; it is taken in 32 bits when even the largest possible score stays below 2^30.
        bool exact = ok && beta == floor(beta) && theta == floor(theta) && beta <= 1048576.0 && theta < 1073741824.0;
        if (exact) exact = token_bound + a.guard[GUARD_MAX_PD] + (unsigned long long)beta * peak_bound < (1ull << 30);
        sh_mode = ok && (exact || !whole) ? 1 : 0;
        sh_n0 = *a.n_requests;
        sh_jmax = (unsigned int)a.guard[GUARD_MAX_JTOP];
        for (int x = 0; x < RS_PENDING; ++x) pend[x].row = -1;
        sh_best[0] = sh_best[1] = 0xffffffffffffffffull;
        sh_n_over = 0;
        sh_blocked = 0;
        sh_blocked_k = 0;
        sh_joined = 0;
        sh_any_bad = 0;
    }
    __syncthreads();
    if (sh_mode == 0) {
        if (tid == 0) *a.handled = 0;
        return;
    }
    const unsigned int beta_i = whole ? (unsigned int)beta : 0u;
    const int theta_i = whole ? (int)theta : 0;
    for (int i = tid; i < Ip; i += nthreads) {
        const RowSummary q = i < I ? a.summary0[i] : make_uint4(RS_OUT, 0, 0, 0);
        tt[i] = make_uint2(q.x, q.z);
        aux[i] = make_uint2(q.y, q.w);
        jst[i] = i < I ? a.jtop0[i] : 0u;
        if (ADMIT) {
            over[i] = i < I ? a.over0[i] : 0;
            if (i < I && (double)over[i] > a.many) atomicAdd(&sh_n_over, 1);
        }
    }
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
    // where the result of item k goes
    auto put_result = [&](long long k, int c, double sc) {
        if (ADMIT && k < q_len) a.queue_choice[k] = c;
        else {
            a.choice[k - q_len] = c;
            if (a.score) a.score[k - q_len] = sc;
        }
    };
    const long long n0 = sh_n0;
    long long room = a.max_requests - n0;
    if (room < 0) room = 0;
    const float thetaf = (float)theta, betaf = (float)beta;
    const float c0f = 2.0f * betaf * thetaf;

    // ---- the walker turns the batch into the sequence of requests that are really routed;
    // malformed arrivals and those beyond the table's room are answered on the spot.  The deciding
    // warp runs it, all lanes alike; the arrivals come through a ring of two 32-entry chunks in shared
    // memory, each chunk copied while the one before it is being used.
    auto copy_chunk = [&](long long first) {
        const long long k = first + lane;
        if (k < a.n_arrivals) {
            cp_async4(&sh_arr_p[k & 63], a.arr_prompt + k);
            cp_async4(&sh_arr_d[k & 63], a.arr_predicted + k);
        }
        cp_async_commit();
    };
    // (32-bit numbers: the batch has fewer than 2^26 items, or the kernel has declined it above)
    const int items = (int)n_items, waiting = (int)q_len;
    const int room_i = room > 0x7fffffffLL ? 0x7fffffff : (int)room;
    int cursor = 0, entered = 0;   // (control warp, all lanes alike) items looked at, requests found
    int first_bad = 0x7fffffff, first_full = 0x7fffffff;   // the first items dropped as malformed / for a full table
    auto walk_next = [&]() {
        Item it;
        it.P = it.D = it.Dc = 0;
        it.k = -1;
        while (cursor < items) {
            int P, D;
            if (ADMIT && cursor < waiting) {
                const long long at = (q_head + cursor) % a.queue_capacity;
                P = a.queue_prompt[at];
                D = a.queue_predicted[at];
            } else {
                const int ac = cursor - waiting;
                if ((ac & 31) == 0) {   // a new chunk: its copy was started a chunk ago; start the next one
                    asm volatile("cp.async.wait_group 0;" ::: "memory");
                    __syncwarp();
                    copy_chunk(ac + 32);
                }
                P = sh_arr_p[ac & 63];
                D = sh_arr_d[ac & 63];
            }
            const bool bad = P < 0 || D < 1 || P > PRE_FIELD_MAX || D > PRE_FIELD_MAX;
            if (bad || entered >= room_i) {
                if (bad && cursor < first_bad) first_bad = cursor;
                if (!bad && cursor < first_full) first_full = cursor;
                if (lane == 0) put_result(cursor, -1, 0.0);
                ++cursor;
                continue;
            }
            it.P = P; it.D = D; it.Dc = D < H ? D : H; it.k = cursor;
            ++cursor; ++entered;
            break;
        }
        return it;
    };
    // (control warp) the last decision, not yet written out
    int out_w = -1, out_k = 0, out_P = 0, out_D = 0;
    long long out_slot = 0;
    double out_score = 0.0;
    // (the instance's two token counts are brought up to date after the last round, from the new table rows)
    auto flush_outputs = [&]() {
        if (out_w < 0) return;
        if (lane == 0) { a.prompt[out_slot] = out_P; a.generated[out_slot] = 0; }
        if (lane == 1) { a.predicted[out_slot] = out_D; a.instance[out_slot] = out_w; }
        if (lane == 2) put_result(out_k, out_w, out_score);
        out_w = -1;
    };
    Item nxt;               // (control warp) the arrival after the one being decided, walked to ahead of time
    bool have_nxt = false;
    nxt.P = nxt.D = nxt.Dc = 0; nxt.k = -1;
    if (warp == RS_CONTROL_WARP) {
        copy_chunk(0);
        const Item first = walk_next();
        if (lane == 0) sh_item[0] = first;
    }
    __syncthreads();

    const int sw_id = warp - RS_FOLD_WARPS - 1;   // score warps
    // ADMIT: the overload level against 32-bit cells (a negative level: every cell is above it)
    const int hot_all = (ADMIT && a.hot < 0) ? 1 : 0;
    const unsigned int hot_u = a.hot < 0 ? 0u : (a.hot > 0xffffffffLL ? 0xffffffffu : (unsigned int)a.hot);
    // fold warps: thread t holds cells 2t, 2t+1, then the same 2 * RS_FOLD_THREADS further on (16-byte accesses, a warp
    // reads 512 contiguous bytes); without 16-byte accesses cells t, t + RS_FOLD_THREADS, ...
    auto cell = [&](int u) { return VEC ? 2 * tid + (u >> 1) * (2 * RS_FOLD_THREADS) + (u & 1) : tid + u * RS_FOLD_THREADS; };
    unsigned int c[CPT], cn[CPT];              // fold warps: the row being folded, the row fetched for the next fold
    int fetched = -1;                          // the row in cn[]
    // literal scan of one row by a warp: the peak with the arrival (P, Dc) added
    auto scan_row = [&](int i, int P, int Dc) {
        const int64_t* src = a.curves + (size_t)i * H;
        unsigned int pk = 0;
        if (VEC) {
            for (int j = 2 * lane; j < H; j += 64) {
                const longlong2 v = __ldcg(reinterpret_cast<const longlong2*>(src + j));
                pk = max(pk, (unsigned int)v.x + (j < Dc ? (unsigned int)(P + j) : 0u));
                pk = max(pk, (unsigned int)v.y + (j + 1 < Dc ? (unsigned int)(P + j + 1) : 0u));
            }
        } else {
            for (int j = lane; j < H; j += 32)
                pk = max(pk, (unsigned int)__ldcg(src + j) + (j < Dc ? (unsigned int)(P + j) : 0u));
        }
        return __reduce_max_sync(0xffffffffu, pk);
    };
    auto fetch = [&](int row, unsigned int* dst) {
        const int64_t* src = a.curves + (size_t)row * H;
        if (VEC) {
            #pragma unroll
            for (int u = 0; u < CPT; u += 2) {
                longlong2 v = make_longlong2(0, 0);
                if (cell(u) < H) v = __ldcg(reinterpret_cast<const longlong2*>(src + cell(u)));
                dst[u] = (unsigned int)v.x; dst[u + 1] = (unsigned int)v.y;
            }
        } else {
            #pragma unroll
            for (int u = 0; u < CPT; ++u) dst[u] = cell(u) < H ? (unsigned int)__ldcg(src + cell(u)) : 0u;
        }
    };
    auto whole_over = [&](unsigned int peak) { return (int)peak > theta_i ? peak - (unsigned int)theta_i : 0u; };

    int ndec = 0, nfold = 0;   // decisions made, folds done: every thread keeps them
    bool stalled = false;
    bool blocked = false;            // ADMIT: a request found every instance overloaded: no more decisions, the folds go on
    // Every arrival is decided after at most RS_PENDING stalled rounds and folded RS_LAG rounds later:
    // the loop below ends by itself.  The limit only keeps a mistake in that reasoning from spinning.
    const int round_limit = (int)((n_items + 2) * (RS_PENDING + 2) + 64);
    bool overrun = false;
    for (int round = 0;; ++round) {
        if (round > round_limit) { overrun = true; break; }
        const int par = round & 1;
        const Item it = sh_item[par];
        const bool have = it.k >= 0 && !blocked;
        if (!have && nfold == ndec) break;
        const bool do_fold = nfold < ndec && (ndec - nfold >= RS_LAG || !have || stalled);
        unsigned int pend_lb_i = 0xffffffffu;   // (control warp) lower bound of pending entry nfold + lane for this arrival
        double pend_lb_d = CUDART_INF;
        int pend_row = -1;
        bool pend_uncertain = false;   // ADMIT: that row was not overloaded when it was decided; its fold may change that
        if (warp == RS_CONTROL_WARP) {
            // =============================== control warp, while the pass runs ===============================
            // what does not depend on the pass: the last decision's outputs, the pending rows' lower
            // bounds, the arrival after this one
            flush_outputs();
            if (lane == 0) sh_best[par ^ 1] = 0xffffffffffffffffull;   // the next round's minimum starts afresh
            if (have) {
                const int d = nfold + lane;
                if (lane < RS_PENDING && d < ndec) {
                    const Pending p = pend[d % RS_PENDING];
                    const unsigned int peak_lb = (unsigned int)it.Dc > p.jw ? (unsigned int)it.P + p.top_lb
                                                                             : max(p.rmax, (unsigned int)it.P + p.c0);
                    pend_row = p.row;
                    pend_uncertain = ADMIT && p.unused[0] == 0u;
                    if (whole) pend_lb_i = p.tokens + beta_i * whole_over(peak_lb);   // (without the arrival's own P + D, like the pass)
                    else pend_lb_d = summary_score(p.tokens, peak_lb, it.P, it.D, theta, beta);
                }
                if (!have_nxt) { nxt = walk_next(); have_nxt = true; }
            }
        } else if (warp > RS_CONTROL_WARP) {
            // =============================== score warps: every row's score for arrival `it` ===============================
            if (have) {
                const int P = it.P, D = it.D, Dc = it.Dc;
                const unsigned int PD = (unsigned int)P + (unsigned int)D;
                if (whole) {
                    unsigned int best = 0xffffffffu;   // scores without the arrival's own P + D
                    int brow = 0x7fffffff;
                    const int K = P - theta_i;
                    if ((unsigned int)Dc > sh_jmax) {
                        // every row's summary gives its peak: two words per row
                        // (a trip count known to the compiler, unrolled by eight: measured against a run-time trip
                        // count and against 4 and 16)
                        #pragma unroll 8
                        for (int u = 0; u < RS_ROWS_PER_LANE; ++u) {
                            const int i = sw_id * 32 + lane + u * nst;
                            if (i < Ip) {
                                const uint2 q = tt[i];
                                const unsigned int t = q.x + beta_i * (unsigned int)max((int)q.y + K, 0);
                                if (t < best) { best = t; brow = i; }
                            }
                        }
                        if (BIG) {   // the lane's rows beyond those
                            for (int i = sw_id * 32 + lane + RS_ROWS_PER_LANE * nst; i < Ip; i += nst) {
                                const uint2 q = tt[i];
                                const unsigned int t = q.x + beta_i * (unsigned int)max((int)q.y + K, 0);
                                if (t < best) { best = t; brow = i; }
                            }
                        }
                    } else {
                        // Some rows are only bounded.  First the smallest upper bound among the warp's rows
                        // (every row's score is at most the score with peak P + top): no row whose lower
                        // bound exceeds it can hold the smallest score.  Then the rows: exact ones compete,
                        // bounded ones that pass that test are scanned by the warp.
                        unsigned int reach = 0xffffffffu;
                        for (int i = sw_id * 32 + lane; i < Ip; i += nst) {
                            const uint2 q = tt[i];
                            reach = min(reach, q.x + beta_i * (unsigned int)max((int)q.y + K, 0));
                        }
                        reach = __reduce_min_sync(0xffffffffu, reach);
                        for (int base = sw_id * 32; base < Ip; base += nst) {
                            const int i = base + lane;
                            const uint2 q = tt[i];
                            bool undecided = false;
                            if (q.x != RS_OUT) {
                                if ((unsigned int)Dc > jst[i]) {
                                    const unsigned int t = q.x + beta_i * (unsigned int)max((int)q.y + K, 0);
                                    if (t < best) { best = t; brow = i; }
                                } else {
                                    const uint2 x = aux[i];
                                    undecided = q.x + beta_i * whole_over(max(x.x, (unsigned int)P + x.y)) <= min(best, reach);
                                }
                            }
                            unsigned int todo = __ballot_sync(0xffffffffu, undecided);
                            while (todo) {
                                const int src = __ffs(todo) - 1;
                                todo &= todo - 1;
                                const int row = base + src;
                                const unsigned int t = tt[row].x + beta_i * whole_over(scan_row(row, P, Dc));
                                if (lane == src && t < best) { best = t; brow = row; }   // a lane's rows ascend
                            }
                        }
                    }
                    // The smallest (score, row) of all score warps: the warp's smallest score by a warp reduction, then
                    // the lanes that hold it (one, but for ties) take the block's minimum of score << 32 | row.
                    const unsigned int wbest = __reduce_min_sync(0xffffffffu, best);
                    if (best == wbest && wbest < RS_OUT) atomicMin(&sh_best[par], ((unsigned long long)best << 32) | (unsigned int)brow);
                } else {
                    // Binary64 scores, per warp.  First every row's score in binary32: a lower and an upper
                    // estimate (the same number when the summary gives the peak exactly), kept in registers.
                    // The warp's smallest upper estimate bounds which of its rows can hold its smallest score;
                    // only those get the binary64 score (each operation rounded on its own), and a row that is
                    // only bounded and passes the test is scanned.  The warps' exact best rows are compared by
                    // the deciding warp, so the block's best row is found without a barrier among the warps.
                    auto estimate = [&](unsigned int tokens, unsigned int peak) {
                        return fmaf(betaf, fmaxf((float)peak - thetaf, 0.0f), (float)(tokens + PD));
                    };
                    float est[RS_ROWS_PER_LANE];
                    float umin = 3.402823466e38f;
                    const bool all_exact = (unsigned int)Dc > sh_jmax;   // every row's summary gives its peak: two words per row
                    if (all_exact) {
                        #pragma unroll
                        for (int u = 0; u < RS_ROWS_PER_LANE; ++u) {
                            const int i = sw_id * 32 + lane + u * nst;
                            est[u] = CUDART_INF_F;
                            if (i < Ip) {
                                const uint2 q = tt[i];
                                if (q.x != RS_OUT) est[u] = estimate(q.x, (unsigned int)P + q.y);
                            }
                            umin = fminf(umin, est[u]);
                        }
                    } else {
                        #pragma unroll
                        for (int u = 0; u < RS_ROWS_PER_LANE; ++u) {
                            const int i = sw_id * 32 + lane + u * nst;
                            est[u] = CUDART_INF_F;
                            if (i < Ip) {
                                const uint2 q = tt[i];
                                if (q.x != RS_OUT) {
                                    const unsigned int up = (unsigned int)P + q.y;
                                    const uint2 x = aux[i];
                                    const unsigned int lo = (unsigned int)Dc > jst[i] ? up : max(x.x, (unsigned int)P + x.y);
                                    umin = fminf(umin, estimate(q.x, up));
                                    est[u] = estimate(q.x, lo);
                                }
                            }
                        }
                    }
                    // estimates are >= 0 and never NaN here (fminf drops a NaN): their bit patterns order like the values
                    const float E = __uint_as_float(0xffffffffu - warp_max_u32(0xffffffffu - __float_as_uint(umin)));
                    // lower_m * (1 - eps) <= E * (1 + eps) + 2 * eps * c0 for the row m of the warp's smallest score
                    const float T = fmaf(E, 1.0f + RS_EPS, 2.0f * RS_EPS * c0f) * (1.0f + 3.0f * RS_EPS);
                    double dbs = CUDART_INF;
                    int dbi = 0x7fffffff;
                    bool bounded = false;   // a row of this lane passes the test but its summary only bounds its peak
                    #pragma unroll
                    for (int u = 0; u < RS_ROWS_PER_LANE; ++u) {
                        if (!(est[u] > T)) {   // (never for a row that is left out: its estimate is infinite ... unless T is)
                            const int i = sw_id * 32 + lane + u * nst;
                            const uint2 q = i < Ip ? tt[i] : make_uint2(RS_OUT, 0u);
                            if (q.x != RS_OUT) {
                                if (all_exact || (unsigned int)Dc > jst[i]) {
                                    const double sc = summary_score(q.x, (unsigned int)P + q.y, P, D, theta, beta);
                                    if (better_row(sc, i, dbs, dbi)) { dbs = sc; dbi = i; }
                                } else {
                                    bounded = true;
                                }
                            }
                        }
                    }
                    if (__any_sync(0xffffffffu, bounded)) {   // rare: the rows again, the bounded ones that pass are scanned
                        for (int base = sw_id * 32; base < Ip; base += nst) {
                            const int i = base + lane;
                            const uint2 q = tt[i];
                            bool undecided = false;
                            if (q.x != RS_OUT && !((unsigned int)Dc > jst[i])) {
                                const uint2 x = aux[i];
                                undecided = !(estimate(q.x, max(x.x, (unsigned int)P + x.y)) > T);
                            }
                            unsigned int todo = __ballot_sync(0xffffffffu, undecided);
                            while (todo) {
                                const int src = __ffs(todo) - 1;
                                todo &= todo - 1;
                                const int row = base + src;
                                const double sc = summary_score(tt[row].x, scan_row(row, P, Dc), P, D, theta, beta);
                                if (lane == src && better_row(sc, row, dbs, dbi)) { dbs = sc; dbi = row; }
                            }
                        }
                    }
                    // the warp's smallest (score, row): scores are >= 0, their bit patterns order like the values
                    unsigned long long key = (unsigned long long)__double_as_longlong(dbs);
                    int wrow = dbi;
                    #pragma unroll
                    for (int off = 16; off > 0; off >>= 1) {
                        const unsigned long long k2 = __shfl_xor_sync(0xffffffffu, key, off);
                        const int r2 = __shfl_xor_sync(0xffffffffu, wrow, off);
                        if (k2 < key || (k2 == key && r2 < wrow)) { key = k2; wrow = r2; }
                    }
                    if (lane == 0) {
                        sh_wkey[par][sw_id] = key;
                        sh_wrow[par][sw_id] = wrow;
                    }
                }
            }
        } else if (do_fold) {
            // =============================== fold warps: entry nfold goes into its row ===============================
            const Pending p = pend[nfold % RS_PENDING];
            const int w = p.row, P = p.P, Dc = p.Dc;
            int64_t* grow = a.curves + (size_t)w * H;
            if (fetched == w) {
                #pragma unroll
                for (int u = 0; u < CPT; ++u) c[u] = cn[u];
            } else {
                fetch(w, c);
            }
            // the row of the next entry, when it is known already, is fetched while this fold runs
            fetched = -1;
            if (CPT <= 8 && nfold + 1 < ndec) {   // (registers allowing)
                fetched = pend[(nfold + 1) % RS_PENDING].row;
                fetch(fetched, cn);
            }
            #pragma unroll
            for (int u = 0; u < CPT; ++u)
                if (cell(u) < Dc) c[u] += (unsigned int)(P + cell(u));
            if (VEC) {
                #pragma unroll
                for (int u = 0; u < CPT; u += 2)   // (a pair whose second cell lies past the ramp writes that cell back unchanged)
                    if (cell(u) < Dc) *reinterpret_cast<longlong2*>(grow + cell(u)) = make_longlong2((long long)c[u], (long long)c[u + 1]);
            } else {
                #pragma unroll
                for (int u = 0; u < CPT; ++u)
                    if (cell(u) < Dc) grow[cell(u)] = (long long)c[u];
            }
            unsigned int rmax = 0, top = 0, jtop = 0xffffffffu;
            int above = 0;
            #pragma unroll
            for (int u = 0; u < CPT; ++u) {   // a thread's steps ascend with u
                const int j = cell(u);
                if (j < H) {
                    if (ADMIT) above += hot_all | (c[u] > hot_u);
                    rmax = max(rmax, c[u]);
                    const unsigned int t = c[u] + (unsigned int)j;
                    if (t > top) { top = t; jtop = (unsigned int)j; }   // (a lane whose cells + steps are all 0 names no step)
                }
            }
            // the warp's largest cell, largest cell + step and the first step that has it (warp reductions: the fold
            // warps are the longest chain of a round, and a butterfly of shuffles is three times as many instructions)
            rmax = __reduce_max_sync(0xffffffffu, rmax);
            const unsigned int wt = __reduce_max_sync(0xffffffffu, top);   // (a lane without cells has top 0 and no step)
            const unsigned int wj = __reduce_min_sync(0xffffffffu, top == wt ? jtop : 0xffffffffu);
            if (ADMIT) above = __reduce_add_sync(0xffffffffu, above);
            if (lane == 0) sh_fold[warp] = make_uint4(rmax, wt, wj, (unsigned int)above);
        }
        __syncthreads();   // the pass and the fold's per-warp maxima are complete
        if (warp == RS_CONTROL_WARP) {
            if (have) {
                // ---- the decision.  The pass's best row wins unless a pending row could do better.
                const int P = it.P, D = it.D, Dc = it.Dc;
                const unsigned int PD = (unsigned int)P + (unsigned int)D;
                double b1s = CUDART_INF;   // binary64 path: the pass's best score
                unsigned int b1i = 0xffffffffu;   // whole-number path: the same without the arrival's own P + D
                int b1r = -1;
                if (whole) {
                    // the score warps took the minimum over all of them already
                    const unsigned long long key = sh_best[par];
                    if (key != 0xffffffffffffffffull) { b1i = (unsigned int)(key >> 32); b1r = (int)(unsigned int)key; }
                } else {   // binary64 scores: (score bits, row) pairs, smallest first, by shuffles
                    unsigned long long key = lane < nsw ? sh_wkey[par][lane] : 0xffffffffffffffffull;
                    int row = lane < nsw ? sh_wrow[par][lane] : 0x7fffffff;
                    for (int off = 1; off < nsw; off <<= 1) {
                        const unsigned long long k2 = __shfl_xor_sync(0xffffffffu, key, off);
                        const int r2 = __shfl_xor_sync(0xffffffffu, row, off);
                        if (k2 < key || (k2 == key && r2 < row)) { key = k2; row = r2; }
                    }
                    key = __shfl_sync(0xffffffffu, key, 0);   // lanes beyond the warps' count hold no result of their own
                    row = __shfl_sync(0xffffffffu, row, 0);
                    if (row != 0x7fffffff) {
                        b1s = __longlong_as_double((long long)key);
                        b1r = row;
                    }
                }
                bool stall = b1r < 0;
                if (pend_row >= 0) {
                    const bool could_win = whole ? (pend_lb_i < b1i || (pend_lb_i == b1i && pend_row < b1r))
                                                 : better_row(pend_lb_d, pend_row, b1s, b1r);
                    if (pend_row == b1r || could_win) stall = true;
                }
                stall = __any_sync(0xffffffffu, stall);
                if (ADMIT) {
                    // every instance overloaded?  Rows are counted once their state is known; a pending row that was
                    // not overloaded when it was decided may have become so.
                    const int uncertain = __popc(__ballot_sync(0xffffffffu, pend_uncertain));
                    const int n_over = sh_n_over;
                    if (n_over >= I) {   // the request is not routed: the batch stops here
                        stall = true;
                        if (lane == 0) { sh_blocked = 1; sh_blocked_k = it.k; }
                    } else if (n_over + uncertain >= I) {
                        stall = true;
                    }
                }
                if (!stall) {
                    // the row is pending from now on: exact token count, bounds for the rest
                    const int w = b1r;
                    if (lane == 0) {
                        const uint2 q = tt[w], x = aux[w];
                        const unsigned int jw = jst[w];
                        uint4* dst = reinterpret_cast<uint4*>(&pend[ndec % RS_PENDING]);
                        dst[0] = make_uint4((unsigned int)w, (unsigned int)P, (unsigned int)D, (unsigned int)Dc);
                        dst[1] = make_uint4(q.x + PD, q.y + ((int)jw < Dc ? (unsigned int)P + jw : 0u), jw, x.x);
                        dst[2] = make_uint4(x.y + (unsigned int)P, (ADMIT && (double)over[w] > a.many) ? 1u : 0u, 0u, 0u);
                        tt[w] = make_uint2(RS_OUT, 0u);
                        *reinterpret_cast<uint4*>(&sh_item[par ^ 1]) = make_uint4((unsigned int)nxt.P, (unsigned int)nxt.D, (unsigned int)nxt.Dc, (unsigned int)nxt.k);
                    }
                    // what the outside sees of the decision is written while the next pass runs
                    out_w = w; out_k = it.k; out_P = P; out_D = D; out_slot = n0 + ndec;
                    out_score = whole ? (double)(b1i + PD) : b1s;
                    have_nxt = false;
                } else if (lane == 0) {
                    sh_item[par ^ 1] = it;
                }
                if (lane == 0) {
                    sh_decided[par] = stall ? 0 : 1;
                }
            } else if (lane == 0) {
                sh_item[par ^ 1] = it;   // the batch has ended; the remaining folds go on
            }
        } else if (tid == 0 && do_fold) {
            // ---- the folded row's new summary; the row takes part in the next pass again
            const Pending p = pend[nfold % RS_PENDING];
            unsigned int rmax = 0, top = 0, jtop = 0xffffffffu;
            int above = 0;
            #pragma unroll
            for (int x = 0; x < RS_FOLD_WARPS; ++x) {   // the first step at which the largest cell + step is taken
                const uint4 q = sh_fold[x];
                above += (int)q.w;
                rmax = max(rmax, q.x);
                if (q.z != 0xffffffffu && (jtop == 0xffffffffu || q.y > top || (q.y == top && q.z < jtop))) { top = q.y; jtop = q.z; }
            }
            if (jtop == 0xffffffffu) jtop = 0u;
            aux[p.row] = make_uint2(rmax, c[0]);
            jst[p.row] = jtop;
            if (jtop > sh_jmax) sh_jmax = jtop;
            if (ADMIT) {
                const bool was = (double)over[p.row] > a.many;
                over[p.row] = above;
                if (!was && (double)above > a.many) sh_n_over += 1;
            }
            tt[p.row] = make_uint2(p.tokens, top);
        }
        __syncthreads();
        if (have) {
            stalled = sh_decided[par] == 0;
            if (!stalled) ++ndec;
        } else {
            stalled = false;
        }
        if (do_fold) ++nfold;
        if (ADMIT && sh_blocked) blocked = true;
    }
    if (warp == RS_CONTROL_WARP) flush_outputs();
    if (overrun && tid == 0) atomicOr(a.status, PRE_ST_TIMEOUT);
    // Every routed request adds its prompt to its instance's queued tokens and its predicted length to the tokens
    // being decoded (Sec. 4.3.3): one reduction each per new table row, by the whole block, instead of two
    // reductions in every round's chain.
    __syncthreads();
    for (int i = tid; i < ndec; i += nthreads) {
        const int w = a.instance[n0 + i];
        atomicAdd(reinterpret_cast<unsigned long long*>(a.queued_p + w), (unsigned long long)a.prompt[n0 + i]);
        atomicAdd(reinterpret_cast<unsigned long long*>(a.current_d + w), (unsigned long long)a.predicted[n0 + i]);
    }
    asm volatile("cp.async.wait_group 0;" ::: "memory");
    // what the walker noted beyond a blocked request is decided again below and does not count here
    const long long decided = (ADMIT && blocked) ? sh_blocked_k : n_items;
    if (tid == RS_FOLD_THREADS) {   // the control warp kept the walker's notes
        *a.n_requests = n0 + ndec;
        int flags = 0;
        if (first_bad < decided) flags |= PRE_ST_BADREQ;
        if (first_full < decided) flags |= PRE_ST_CAPACITY;
        if (flags) atomicOr(a.status, flags);
        *a.handled = 1;
    }
    if (ADMIT) {
        // Everything from the blocked request on: a request that was waiting keeps its place; an arrival joins
        // the tail of the queue while there is room and is turned away otherwise (a malformed arrival is
        // dropped).  Nothing else reads or writes these arrays any more.
        __syncthreads();
        const long long stop = decided;
        const long long left = stop < q_len ? q_len - stop : 0;          // waiting entries that stay
        for (long long k = stop + tid; k < q_len; k += nthreads) a.queue_choice[k] = -2;
        const long long a0 = (stop > q_len ? stop : q_len) - q_len;      // first arrival that was not decided
        const int nw = nthreads >> 5;
        for (long long base = a0; base < a.n_arrivals; base += nthreads) {
            const long long i = base + tid;
            int P = -1, D = 0;
            if (i < a.n_arrivals) { P = a.arr_prompt[i]; D = a.arr_predicted[i]; }
            const bool ok = i < a.n_arrivals && !(P < 0 || D < 1 || P > PRE_FIELD_MAX || D > PRE_FIELD_MAX);
            const unsigned int vote = __ballot_sync(0xffffffffu, ok);
            if (lane == 0) sh_warp_ok[warp] = __popc(vote);
            __syncthreads();
            long long rank = sh_joined + __popc(vote & ((1u << lane) - 1u));
            int total = 0;
            for (int x = 0; x < nw; ++x) { if (x < warp) rank += sh_warp_ok[x]; total += sh_warp_ok[x]; }
            if (i < a.n_arrivals) {
                int c = -1;
                if (ok) {
                    if (left + rank < a.queue_capacity) {
                        const long long pos = (q_head + q_len + rank) % a.queue_capacity;   // behind the last one waiting
                        a.queue_prompt[pos] = P;
                        a.queue_predicted[pos] = D;
                        c = -2;
                    } else {
                        c = -3;
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
        if (tid == 0) {
            long long joined = sh_joined;
            if (left + joined > a.queue_capacity) joined = a.queue_capacity - left;
            a.queue_state[0] = a.queue_capacity > 0 ? (q_head + (q_len - left)) % a.queue_capacity : 0;
            a.queue_state[1] = left + joined;
            if (blocked && sh_any_bad) atomicOr(a.status, PRE_ST_BADREQ);
        }
    }
}

}  // namespace

// ---- host side

static size_t summaries_smem_bytes(int I, bool admit) {
    const size_t Ip = (size_t)((I + 31) & ~31);
    return Ip * (2 * sizeof(uint2) + sizeof(uint32_t) + (admit ? sizeof(int) : 0));
}

// Score warps: sixteen rows per score thread up to RS_MAX_SCORE_WARPS warps, more rows per thread beyond (measured:
// 4,096 instances are fastest with 8 score warps, 1,024 with 2 to 4; more warps lengthen the block barriers more
// than they shorten the pass, and a block of more than 640 threads leaves 64 registers per thread: 70 % slower).
static int summaries_score_warps(int I) {
    int w = (I + RS_ROWS_PER_LANE * 32 - 1) / (RS_ROWS_PER_LANE * 32);
    return w < 1 ? 1 : (w > RS_MAX_SCORE_WARPS ? RS_MAX_SCORE_WARPS : w);
}

// beta and theta = t_mem * M whole numbers of moderate size: the scores can be taken in whole-number arithmetic
static bool summaries_whole_numbers(const pre_ctx* ctx) {
    const double beta = ctx->cfg.beta, theta = ctx->theta;
    return beta == floor(beta) && theta == floor(theta) && beta <= 1048576.0 && theta < 1073741824.0;
}

template <int CPT, bool ADMIT, int KIND>
static const void* summaries_kernel(bool vec) {
    return vec ? (const void*)pre_route_summaries<CPT, true, ADMIT, KIND> : (const void*)pre_route_summaries<CPT, false, ADMIT, KIND>;
}
template <bool ADMIT, int KIND>
static const void* summaries_kernel_of_kind(int H) {
    const bool vec = (H & 1) == 0;
    if (H <= 4 * RS_FOLD_THREADS) return summaries_kernel<4, ADMIT, KIND>(vec);
    if (H <= 8 * RS_FOLD_THREADS) return summaries_kernel<8, ADMIT, KIND>(vec);
    if (H <= 16 * RS_FOLD_THREADS) return summaries_kernel<16, ADMIT, KIND>(vec);
    return summaries_kernel<32, ADMIT, KIND>(vec);
}
// nullptr: no instantiation takes this context (binary64 scores with more than RS_ROWS_PER_LANE rows per score lane)
template <bool ADMIT>
static const void* summaries_kernel_for(const pre_ctx* ctx) {
    const int H = ctx->cfg.horizon, I = ctx->cfg.n_instances;
    const bool big = I > RS_ROWS_PER_LANE * 32 * RS_MAX_SCORE_WARPS;
    if (summaries_whole_numbers(ctx))
        return big ? summaries_kernel_of_kind<ADMIT, RS_WHOLE_BIG>(H) : summaries_kernel_of_kind<ADMIT, RS_WHOLE>(H);
    return big ? nullptr : summaries_kernel_of_kind<ADMIT, RS_BINARY64>(H);
}

template <bool ADMIT>
static cudaError_t summaries_configure_one(pre_ctx* ctx, size_t limit, size_t* smem_out) {
    const int I = ctx->cfg.n_instances;
    *smem_out = 0;
    const void* fn = summaries_kernel_for<ADMIT>(ctx);
    if (fn == nullptr) return cudaSuccess;
    cudaFuncAttributes attr;
    cudaError_t e = cudaFuncGetAttributes(&attr, fn);
    if (e != cudaSuccess) return e;
    const size_t smem = summaries_smem_bytes(I, ADMIT);
    if (smem + attr.sharedSizeBytes + 256 > limit) return cudaSuccess;   // too many instances
    e = cudaFuncSetAttribute(fn, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)smem);
    if (e != cudaSuccess) return e;
    *smem_out = smem;
    return cudaSuccess;
}

cudaError_t pre_route_summary_configure(pre_ctx* ctx) {
    ctx->route_summary_smem = 0;
    ctx->route_summary_smem_admit = 0;
    if (ctx->cfg.horizon > 32 * RS_FOLD_THREADS) return cudaSuccess;
    cudaDeviceProp prop;
    cudaError_t e = cudaGetDeviceProperties(&prop, ctx->device);
    if (e != cudaSuccess) return e;
    e = summaries_configure_one<false>(ctx, (size_t)prop.sharedMemPerBlockOptin, &ctx->route_summary_smem);
    if (e != cudaSuccess) return e;
    return summaries_configure_one<true>(ctx, (size_t)prop.sharedMemPerBlockOptin, &ctx->route_summary_smem_admit);
}

bool pre_route_summary_fits(const pre_ctx* ctx) { return ctx->route_summary_smem != 0 && ctx->d_rs_summary != nullptr; }
bool pre_route_summary_admit_fits(const pre_ctx* ctx) {
    return ctx->route_summary_smem_admit != 0 && ctx->d_rs_summary != nullptr && ctx->d_rs_over != nullptr;
}

static void fill_summary_args(pre_ctx* ctx, SumArgs& p, RouteSumArgs& a, const int32_t* arr_prompt,
                              const int32_t* arr_predicted, int64_t n_arrivals, int64_t* curves, int64_t* queued_p,
                              int64_t* current_d, int32_t* prompt, int32_t* generated, int32_t* predicted,
                              int32_t* instance, int64_t* n_requests, int32_t* choice, double* score) {
    const int I = ctx->cfg.n_instances, H = ctx->cfg.horizon;
    p.curves = curves; p.queued_p = queued_p; p.current_d = current_d;
    p.arr_prompt = arr_prompt; p.arr_predicted = arr_predicted; p.n_arrivals = n_arrivals;
    p.I = I; p.H = H;
    p.summary = reinterpret_cast<RowSummary*>(ctx->d_rs_summary);
    p.jtop = ctx->d_rs_jtop; p.guard = ctx->d_rs_guard;
    p.over = nullptr; p.hot = 0; p.queue_prompt = nullptr; p.queue_predicted = nullptr; p.queue_entry = nullptr;
    p.queue_capacity = 0;
    a.arr_prompt = arr_prompt; a.arr_predicted = arr_predicted; a.n_arrivals = n_arrivals;
    a.curves = curves; a.queued_p = queued_p; a.current_d = current_d;
    a.prompt = prompt; a.generated = generated; a.predicted = predicted; a.instance = instance;
    a.n_requests = n_requests; a.max_requests = ctx->cfg.max_requests;
    a.choice = choice; a.score = score;
    a.I = I; a.H = H;
    a.theta = ctx->theta; a.beta = ctx->cfg.beta;
    a.summary0 = p.summary; a.jtop0 = p.jtop; a.guard = p.guard;
    a.status = ctx->d_status; a.handled = ctx->d_rs_handled;
    a.score_warps = summaries_score_warps(I);
    a.queue_prompt = nullptr; a.queue_predicted = nullptr; a.queue_state = nullptr; a.queue_entry = nullptr;
    a.queue_capacity = 0; a.queue_choice = nullptr; a.hot = 0; a.many = 0.0; a.over0 = nullptr;
}

template <bool ADMIT>
static cudaError_t launch_summary_kernels(pre_ctx* ctx, const SumArgs& p, const RouteSumArgs& a, cudaStream_t s) {
    const int I = ctx->cfg.n_instances;
    cudaError_t e = cudaMemsetAsync(ctx->d_rs_guard, 0, 8 * sizeof(unsigned long long), s);
    if (e != cudaSuccess) return e;
    const int rows_per_block = SUM_THREADS / 32;
    pre_summarise_rows<<<(I + rows_per_block - 1) / rows_per_block, SUM_THREADS, 0, s>>>(p);
    e = cudaGetLastError();
    if (e != cudaSuccess) return e;
    void* params[] = {(void*)&a};
    return cudaLaunchKernel(summaries_kernel_for<ADMIT>(ctx), dim3(1), dim3(RS_FOLD_THREADS + 32 + 32 * a.score_warps), params,
                            ADMIT ? ctx->route_summary_smem_admit : ctx->route_summary_smem, s);
}

cudaError_t pre_launch_route_summary(pre_ctx* ctx, const int32_t* arr_prompt, const int32_t* arr_predicted,
                                     int64_t n_arrivals, int64_t* curves, int64_t* queued_p, int64_t* current_d,
                                     int32_t* prompt, int32_t* generated, int32_t* predicted, int32_t* instance,
                                     int64_t* n_requests, int32_t* choice, double* score, cudaStream_t s) {
    SumArgs p;
    RouteSumArgs a;
    fill_summary_args(ctx, p, a, arr_prompt, arr_predicted, n_arrivals, curves, queued_p, current_d, prompt, generated,
                      predicted, instance, n_requests, choice, score);
    return launch_summary_kernels<false>(ctx, p, a, s);
}

// The queue's head and length must have been copied to ctx->d_queue_entry on the stream before this call.
cudaError_t pre_launch_route_summary_admit(pre_ctx* ctx, const int32_t* arr_prompt, const int32_t* arr_predicted,
                                           int64_t n_arrivals, long long hot, double many, int32_t* queue_prompt,
                                           int32_t* queue_predicted, int64_t* queue_state, int64_t queue_capacity,
                                           int32_t* queue_choice, int64_t* curves, int64_t* queued_p,
                                           int64_t* current_d, int32_t* prompt, int32_t* generated, int32_t* predicted,
                                           int32_t* instance, int64_t* n_requests, int32_t* choice, double* score,
                                           cudaStream_t s) {
    SumArgs p;
    RouteSumArgs a;
    fill_summary_args(ctx, p, a, arr_prompt, arr_predicted, n_arrivals, curves, queued_p, current_d, prompt, generated,
                      predicted, instance, n_requests, choice, score);
    p.over = ctx->d_rs_over; p.hot = hot;
    p.queue_prompt = queue_prompt; p.queue_predicted = queue_predicted; p.queue_entry = ctx->d_queue_entry;
    p.queue_capacity = queue_capacity;
    a.queue_prompt = queue_prompt; a.queue_predicted = queue_predicted; a.queue_state = queue_state;
    a.queue_entry = ctx->d_queue_entry; a.queue_capacity = queue_capacity; a.queue_choice = queue_choice;
    a.hot = hot; a.many = many; a.over0 = ctx->d_rs_over;
    return launch_summary_kernels<true>(ctx, p, a, s);
}

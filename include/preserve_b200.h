/* preserve_b200 — load anticipator and load-aware request router on one B200 (sm_100a).
 *
 * C ABI of the library.  The operations are those of PreServe's prediction-based
 * management, Sec. 4.3.1 "Instance Load Anticipator" and Sec. 4.3.3 "Load-aware
 * Request Router" of the paper (arXiv 2504.03702).
 *
 * Conventions for every entry point
 *   - Pointers named d_* are DEVICE pointers owned by the caller.  The library never
 *     frees, reallocates or keeps them after the call's work has run on the stream.
 *   - `stream` is a cudaStream_t passed as void* (NULL = the legacy default stream).
 *     Calls enqueue work on that stream and return without synchronising, unless
 *     stated otherwise.  One context serves one stream at a time; calls on one
 *     context are not thread-safe.
 *   - Return value: PRE_OK (0) or a negative pre_error.  Argument errors are found on
 *     the host before anything is launched.  Errors that only the device can see
 *     (malformed request fields, a full request table, a wait that ran out) are
 *     recorded in a device status word that pre_status() reads; the kernels skip the
 *     offending item and never write out of bounds or trap.
 *
 * Data layout
 *   - Request table, structure of arrays, int32 each, capacity max_requests:
 *       prompt[r]    P  prompt tokens            (0 <= P,  P + g < 2^28)
 *       generated[r] g  tokens generated so far  (g >= 0)
 *       predicted[r] D  predicted response tokens (D >= 1, D - g < 2^28)
 *       instance[r]     instance the request runs on, in [0, n_instances)
 *     A request with g >= D has finished; it stays in the table as a tombstone and
 *     contributes nothing.  Any other violation is a malformed request: it is skipped
 *     and PRE_EBADREQ is recorded.
 *   - curves: int64[n_instances * horizon], row-major, 16-byte aligned.  curves[i*H + j]
 *     is the anticipated number of KV tokens held by instance i at j decode iterations
 *     from now: the paper's load-look-ahead map entry U_j times the capacity M,
 *     restricted to the next H = l iterations.
 *   - queued_p, current_d: int64[n_instances]; the router's "queued tokens to be
 *     prefilled" and "tokens still to be generated" per instance (Sec. 4.3.3).
 */
#ifndef PRESERVE_B200_H
#define PRESERVE_B200_H

#include <stdint.h>

#ifdef __cplusplus
extern "C" {
#endif

typedef enum pre_error {
    PRE_OK = 0,
    PRE_EINVAL = -1,    /* null or misaligned pointer, size out of range, bad config        */
    PRE_ECAPACITY = -2, /* request table full: the arrivals that did not fit were not routed */
    PRE_EBADREQ = -3,   /* a malformed request or arrival was skipped                        */
    PRE_ETIMEOUT = -4,  /* a bounded device-side wait ran out; the call stopped early (see   */
                        /* pre_route_batch and pre_anticipate for what is left behind)       */
    PRE_ECUDA = -5,     /* a CUDA runtime call failed (see pre_last_cuda_error)              */
    PRE_ENOMEM = -6,    /* scratch allocation failed in pre_create                           */
    PRE_ESIZE = -7      /* problem larger than the built-in scratch of pre_anticipate_static */
} pre_error;

typedef struct pre_ctx pre_ctx; /* opaque; owns only internal device scratch */

typedef struct pre_config {
    int32_t n_instances;     /* I >= 1 */
    int32_t horizon;         /* H >= 1: look-ahead window in decode iterations (the paper's l);
                                at most 8192 */
    int64_t capacity_tokens; /* M >= 1: KV token capacity of one instance (Sec. 4.3.1) */
    double t_mem;            /* T_mem, ideal memory usage; 0.8 in the paper (Sec. 4.3.3) */
    double beta;             /* penalty coefficient; 1.0 in the paper (Sec. 4.3.3) */
    int64_t max_requests;    /* capacity of the request table arrays, >= 1, < 2^31 */
} pre_config;

/* Creates a context on the current CUDA device and allocates its scratch (8 bytes per
 * table slot, 8 bytes per instance, and one index word per build tile and 4,096 table
 * slots: a few MB).  *out is set only on success. */
int pre_create(const pre_config* cfg, pre_ctx** out);

/* Frees the scratch.  The caller must have synchronised the stream first. */
int pre_destroy(pre_ctx* ctx);

/* Load-look-ahead maps from the request table (Sec. 4.3.1: for a request with P prompt
 * and D predicted response tokens, U'_i = (U_i*M + (P + i))/M for i in [0, D)).
 * A request that has generated g tokens is that ramp seen g iterations later, so
 *     curves[i][j] = sum over live requests r of instance i with j < D_r - g_r
 *                    of (P_r + g_r + j),          0 <= j < H,
 *     current_d[i] = sum over live requests r of instance i of (D_r - g_r).
 * Overwrites d_curves (I*H) and d_current_d (I).  n_requests is a host value,
 * 0 <= n_requests <= max_requests.  The request arrays are only read. */
int pre_anticipate(pre_ctx* ctx, const int32_t* d_prompt, const int32_t* d_generated,
                   const int32_t* d_predicted, const int32_t* d_instance, int64_t n_requests,
                   int64_t* d_curves, int64_t* d_current_d, void* stream);

/* pre_anticipate without a context and without any allocation.  (The paper has no counterpart:
 * this entry point exists for the sake of its callers, it computes exactly what pre_anticipate
 * computes.)
 *
 * Who needs it: code that runs where device memory may not be requested or returned - for
 * example a plug-in inside a serving engine that has handed the whole GPU to its own pool
 * allocator, a callback that runs while the CUDA allocator's lock is held, or a latency-critical
 * control loop where a cudaMalloc (which can synchronise the device) is not acceptable.
 * pre_create allocates scratch; this call uses scratch that is part of the library image
 * instead, about 3.1 MB that every GPU which loads the library holds until the process exits.
 *
 * Limits (PRE_ESIZE beyond them): n_requests <= 262,144; n_instances <= 65,536; at most 2,048
 * build tiles, which covers n_instances * horizon up to roughly 16 million cells (4,096 x 2,048
 * needs 1,024 tiles); device ordinal below 64.  horizon <= 8192 as everywhere.
 *
 * Arguments as for pre_anticipate, with the shape passed directly.  d_flags (DEVICE int32,
 * may be NULL, zeroed by the caller) receives a non-zero value if a malformed request was
 * skipped.  The call launches on `stream` and returns without synchronising; it calls no
 * cudaMalloc, cudaFree or other allocating routine.
 *
 * The first call on each device, made with that device current, looks up the device address
 * of the built-in scratch and raises the kernels' shared-memory limits; make that first call
 * before any stream capture begins.  All calls on a device share the one scratch area, which
 * keeps whatever the last call left in it: two calls whose work overlaps on the GPU (different
 * streams, or different host threads) race and give wrong maps - order them on one stream or
 * with events.  Nothing in the scratch needs clearing between calls (the one part that must
 * start at zero, a word per instance, is cleared again by the call that used it).  As with the other
 * entry points, do not call it from two host threads at the same time. */
int pre_anticipate_static(int32_t n_instances, int32_t horizon, const int32_t* d_prompt,
                          const int32_t* d_generated, const int32_t* d_predicted, const int32_t* d_instance,
                          int64_t n_requests, int64_t* d_curves, int64_t* d_current_d, int32_t* d_flags,
                          void* stream);

/* Routes n_arrivals requests in array order (Sec. 4.3.3).  For arrival (P, D) and every
 * instance i the anticipator "virtually" adds the request to the map and takes the peak
 * over the window,
 *     peak_i = max over j in [0,H) of curves[i][j] + (j < min(D,H) ? P + j : 0),
 *     L_i = (queued_p[i] + P) + (current_d[i] + D) + beta * max(0, peak_i - t_mem*M),
 * evaluated in binary64 with each operation rounded separately (no fused multiply-add);
 * the arrival goes to argmin_i L_i, the lowest index among equal scores.  The chosen
 * instance then really receives it, before the next arrival is scored:
 *     curves[i*][j] += P + j for j < min(D,H); queued_p[i*] += P; current_d[i*] += D;
 *     (P, 0, D, i*) is appended to the request table at index *d_n_requests, which advances.
 * d_choice[k] (int32) receives i*, or -1 if arrival k was malformed (P < 0, D < 1, either
 * >= 2^28) or did not fit in the table; d_score[k] (binary64, may be NULL) the winning L.
 * *d_n_requests is a DEVICE int64, read at the start and written at the end of the batch.
 *
 * Two kernels implement the call with identical results (pre_route_select picks one).  The summary
 * kernel keeps four numbers per row (largest cell, largest cell + step and where it sits, cell 0)
 * that give the peak of almost every row for any arrival without reading the row, scans the few
 * rows they leave undecided, routes with a single block and waits for nobody; it takes the batch
 * when the context's instances fit its shared memory, every value stays below 2^32 during the
 * batch and the batch (with the waiting requests of pre_route_admit) has fewer than 2^26 entries,
 * which it checks on the device.  Otherwise the scanning kernel routes: it reads every cell
 * for every arrival, its blocks exchange their best instances through device memory and wait
 * for one another a bounded number of polls.  If such a wait runs out (PRE_ETIMEOUT from
 * pre_status; it should never happen on a GPU that runs the kernel alone), the blocks agree on
 * the last arrival that every one of them had scored: arrivals up to that one are routed exactly
 * as above (maps, queued_p, current_d, table and *d_n_requests all include them and nothing
 * else), every later arrival gets PRE_CHOICE_DROPPED and score 0, and the context stays usable.
 * Only if the blocks cannot even meet to agree (a second, much longer bounded wait) may the maps
 * hold one request more than the table; rebuild them with pre_anticipate then. */
int pre_route_batch(pre_ctx* ctx, const int32_t* d_arr_prompt, const int32_t* d_arr_predicted,
                    int64_t n_arrivals, int64_t* d_curves, int64_t* d_queued_p, int64_t* d_current_d,
                    int32_t* d_prompt, int32_t* d_generated, int32_t* d_predicted, int32_t* d_instance,
                    int64_t* d_n_requests, int32_t* d_choice, double* d_score, void* stream);

/* One decode iteration (iteration-level batching, Sec. 2; the map covers "the next
 * iterations", Sec. 4.3.1).  Every live request generates one token (g += 1; it becomes a
 * tombstone when g reaches D); every map moves one iteration closer,
 *     curves'[i][j] = curves[i][j+1] for j < H-1,
 *     curves'[i][H-1] = sum over requests of i with D - g' >= H of (P + g' + H - 1), g' = g + 1;
 * current_d[i] drops by the number of requests of i that were live; queued_p[i] becomes 0
 * (every queued prefill is taken to finish within the iteration).  *d_n_requests (DEVICE
 * int64) is only read.  Afterwards pre_anticipate on the table reproduces d_curves. */
int pre_step(pre_ctx* ctx, int32_t* d_prompt, int32_t* d_generated, int32_t* d_predicted,
             int32_t* d_instance, const int64_t* d_n_requests, int64_t* d_curves,
             int64_t* d_queued_p, int64_t* d_current_d, void* stream);

/* Values of d_choice / d_queue_choice below zero. */
#define PRE_CHOICE_DROPPED     (-1)  /* malformed request, or the request table is full */
#define PRE_CHOICE_WAITS       (-2)  /* every instance overloaded: the request is in the queue */
#define PRE_CHOICE_TURNED_AWAY (-3)  /* every instance overloaded and the queue is full */

/* Router with its admission queue (Sec. 4.3.3: an incoming request is held back while all
 * instances are overloaded and is turned away once the queue is full).  The paper does not
 * define "overloaded" for the router; the scaler's criterion of Sec. 4.3.2 is used, on the maps
 * as they stand, without the request:
 *     instance i is overloaded  <=>  #{ j in [0,H) : curves[i][j] > overload_level * M } > overload_share * H
 * (binary64 products; the paper's values are 0.95 and 0.10).
 * One call decides, in this order, the requests that were waiting at entry (oldest first) and
 * then the n_arrivals new ones.  While some instance is not overloaded a request is routed
 * exactly as by pre_route_batch (score, argmin, update of the winner, append to the table).
 * The first request that finds every instance overloaded is not routed, and neither is any
 * request after it (maps only grow during a call): a waiting request keeps its place, an
 * arrival joins the tail of the queue while it has room and is turned away otherwise.
 * The queue is a ring owned by the caller, all DEVICE memory: d_queue_prompt/d_queue_predicted
 * (int32[queue_capacity]), d_queue_state (int64[2] = {head, length}; entry q, 0 = oldest, is at
 * (head + q) mod queue_capacity; start with {0, 0}).  queue_capacity may be 0 (nobody waits).
 * Results: d_queue_choice[q] (int32[queue_capacity], written for the entries waiting at entry) and
 * d_choice[k] for the arrivals receive the instance index or one of the PRE_CHOICE_* values;
 * d_score[k] (may be NULL) the winning L of a routed arrival, 0 otherwise.  Entries that leave
 * the queue are a prefix of it.  Other arguments, errors and the status word as for
 * pre_route_batch; n_arrivals and queue_capacity below 2^30.  After a wait that ran out
 * (PRE_ETIMEOUT) the requests decided so far are as described for pre_route_batch, waiting
 * requests that were not reached keep their place and arrivals that were not reached are dropped. */
int pre_route_admit(pre_ctx* ctx, const int32_t* d_arr_prompt, const int32_t* d_arr_predicted, int64_t n_arrivals,
                    double overload_level, double overload_share, int32_t* d_queue_prompt,
                    int32_t* d_queue_predicted, int64_t* d_queue_state, int64_t queue_capacity,
                    int32_t* d_queue_choice, int64_t* d_curves, int64_t* d_queued_p, int64_t* d_current_d,
                    int32_t* d_prompt, int32_t* d_generated, int32_t* d_predicted, int32_t* d_instance,
                    int64_t* d_n_requests, int32_t* d_choice, double* d_score, void* stream);

/* Refinement of the maps against real response lengths (Sec. 4.3.1, the paragraph after the
 * map update).  d_actual[r] (DEVICE int32, >= 1) is the real response length of table row r as
 * the serving engine learns it; call once per tick, after pre_step.  For every row r below
 * *d_n_requests (DEVICE int64, only read):
 *   finished early:  g < D and d_actual[r] <= g.  The tokens anticipated for the rest of the
 *       prediction are taken out, curves[inst][j] -= P + g + j for j in [0, min(D-g, H)),
 *       current_d[inst] -= D - g, and the row is closed at its real length, d_predicted[r] = g.
 *   still running at the predicted end:  g == D and d_actual[r] > g.  The response is extended
 *       by E = ceil(D / 5) tokens (0.2 times the length reached, at least one),
 *       curves[inst][j] += P + g + j for j in [0, min(E, H)), current_d[inst] += E,
 *       d_predicted[r] = D + E.  Repeats on later ticks until the request ends; an extension
 *       that overshoots is taken out by the first rule.
 *   otherwise nothing changes.  Afterwards pre_anticipate on the table reproduces d_curves.
 * d_counts (DEVICE int64[3], may be NULL) receives {early finishes, extensions, malformed rows}.
 * A malformed row (as for pre_anticipate, or d_actual[r] < 1, or D > 2^30) is skipped and
 * PRE_EBADREQ reported by pre_status.  Asynchronous on `stream`; map cells are updated with
 * integer reductions, so the result does not depend on the order of the rows. */
int pre_refine(pre_ctx* ctx, const int32_t* d_prompt, const int32_t* d_generated, int32_t* d_predicted,
               const int32_t* d_instance, const int32_t* d_actual, const int64_t* d_n_requests,
               int64_t* d_curves, int64_t* d_current_d, int64_t* d_counts, void* stream);

/* Signals for the proactive instance scaler (Sec. 4.3.2), read off the maps as they stand.
 * The scaler treats an instance as potentially overloaded when its anticipated KV usage is
 * above 95 % of the capacity on more than 10 % of the window's steps, and it may scale down only
 * when every instance stays below T_f = 30 % over the whole window, the number of instances to
 * isolate being N_c - sum(max U')/T_f.
 *     d_over_count[i] (int32) = #{ j in [0,H) : curves[i][j] > overload_level * M }
 *     d_row_max[i]    (int64) = max_j curves[i][j]                      (= max(U') * M)
 *     d_summary[0] = #{ i : over_count[i] > overload_share * H }        (potentially overloaded)
 *     d_summary[1] = #{ i : not (row_max[i] < idle_level * M) }         (0: scale-down may fire)
 *     d_summary[2] = sum_i row_max[i]          (isolate N_c - d_summary[2] / (M * idle_level))
 * The three products are binary64; comparisons are made in binary64 (token counts below 2^53
 * convert exactly).  The paper's values are 0.95, 0.10 and 0.30.  d_summary is int64[3], all
 * pointers DEVICE, the maps are only read. */
int pre_scaler_signals(pre_ctx* ctx, const int64_t* d_curves, double overload_level, double overload_share,
                       double idle_level, int32_t* d_over_count, int64_t* d_row_max, int64_t* d_summary,
                       void* stream);

/* One scheduler tick in one call: pre_step, then (when d_actual is given) pre_refine against the
 * real response lengths, then (when the three signal outputs are given) pre_scaler_signals on the
 * maps as the first two leave them (Sec. 2, Sec. 4.3.1, Sec. 4.3.2).  Results are those of the three
 * calls made one after the other, bit for bit; the table is read once and the maps are read and
 * written once instead of twice and three times.  d_actual may be NULL (no refinement; d_counts is
 * then zeroed if given).  d_over_count, d_row_max and d_summary are given together or all NULL.
 * Every other argument as for the three calls. */
int pre_tick(pre_ctx* ctx, int32_t* d_prompt, int32_t* d_generated, int32_t* d_predicted, int32_t* d_instance,
             const int32_t* d_actual, const int64_t* d_n_requests, int64_t* d_curves, int64_t* d_queued_p,
             int64_t* d_current_d, double overload_level, double overload_share, double idle_level,
             int32_t* d_over_count, int64_t* d_row_max, int64_t* d_summary, int64_t* d_counts, void* stream);

/* Full-width maps (Sec. 4.3.1: the load-look-ahead map covers the next L iterations, L the
 * largest response the model can produce, e.g. 4,096; the load is projected over the next l
 * iterations, e.g. l = 100, for the router of Sec. 4.3.3).  A row is kept as a ring over
 * absolute iterations,
 *     d_ring[i*width + (head + j) mod width] = tokens of instance i at j iterations from now,
 * 0 <= j < width = L, int64, row-major; *d_head (DEVICE int64, in [0, width)) is where "now"
 * is.  A decode iteration then moves no map data.  The three calls below take a context whose
 * horizon is the WINDOW l (the same context routes on the window); width >= horizon, else
 * PRE_EINVAL.  A full-width map is built by pre_anticipate on a second context whose horizon
 * is L, into d_ring with *d_head = 0.  One scheduler tick on full-width maps is
 *     pre_ring_step, pre_ring_window, pre_route_batch (or pre_route_admit) on the window,
 *     pre_ring_fold with the choices the router returned,
 * and gives the decisions of a router that takes its peaks over the first l steps of the
 * full-width maps and really adds each routed request's whole ramp: no score of a batch
 * depends on a step beyond the window, and the additions beyond it commute.
 * With pre_route_admit the routed requests are not only arrivals (waiting requests come first,
 * and the queue's slots may be rewritten during the call): fold from the rows the call appended to
 * the request table instead - pre_ring_fold(d_prompt + n0, d_predicted + n0, d_instance + n0,
 * n1 - n0, ...) with n0, n1 the request count before and after the call; those rows are exactly
 * the routed requests, each with its instance. */

/* d_window[i*l + j] = d_ring[i*width + (head + j) mod width], j < l: the dense maps of width
 * l (16-byte aligned) that pre_route_batch, pre_route_admit and pre_scaler_signals take. */
int pre_ring_window(pre_ctx* ctx, const int64_t* d_ring, int32_t width, const int64_t* d_head, int64_t* d_window,
                    void* stream);

/* The real map update of Sec. 4.3.1 for a routed batch: for every arrival k with
 * d_choice[k] in [0, n_instances), d_ring[choice][(head + j) mod width] += P_k + j for
 * j < min(D_k, width).  Entries below zero (dropped, waiting, turned away) are skipped.
 * The router has already updated the window copy, queued_p, current_d and the request
 * table; this call only brings the ring up to date.  Integer reductions: the result does
 * not depend on the order in which the arrivals are applied. */
int pre_ring_fold(pre_ctx* ctx, const int32_t* d_arr_prompt, const int32_t* d_arr_predicted, const int32_t* d_choice,
                  int64_t n_arrivals, int64_t* d_ring, int32_t width, const int64_t* d_head, void* stream);

/* One decode iteration on ring maps: the request table, queued_p and current_d change as in
 * pre_step; every row's slot at the head (step 0, now past) receives what enters at step
 * width-1 (the requests with at least `width` tokens still to come; none when width is the
 * model's largest response), and *d_head becomes (head + 1) mod width.  Afterwards the
 * logical map equals what pre_anticipate builds from the advanced table. */
int pre_ring_step(pre_ctx* ctx, int32_t* d_prompt, int32_t* d_generated, int32_t* d_predicted, int32_t* d_instance,
                  const int64_t* d_n_requests, int64_t* d_ring, int32_t width, int64_t* d_head, int64_t* d_queued_p,
                  int64_t* d_current_d, void* stream);

/* pre_refine (Sec. 4.3.1, the correction of the maps against real response lengths) on ring
 * maps: the same rule, with step j of a row at d_ring[i*width + (head + j) mod width] and the
 * ramps cut at `width` instead of the window.  Call it once per tick after pre_ring_step and
 * before pre_ring_window, so that the router sees the corrected window. */
int pre_ring_refine(pre_ctx* ctx, const int32_t* d_prompt, const int32_t* d_generated, int32_t* d_predicted,
                    const int32_t* d_instance, const int32_t* d_actual, const int64_t* d_n_requests, int64_t* d_ring,
                    int32_t width, const int64_t* d_head, int64_t* d_current_d, int64_t* d_counts, void* stream);

/* Synchronises `stream`, then returns and clears the device status: the most severe of
 * PRE_ETIMEOUT, PRE_ECAPACITY, PRE_EBADREQ recorded since the last call, PRE_ECUDA if the
 * stream reports a CUDA error, else PRE_OK. */
int pre_status(pre_ctx* ctx, void* stream);

/* The cudaError_t value of the last failed runtime call on this context (0 if none). */
int pre_last_cuda_error(const pre_ctx* ctx);

/* Which kernel routes the batches of pre_route_batch and pre_route_admit on this context: PRE_ROUTE_AUTO (default:
 * the summary kernel when the shape fits it and beta and t_mem * M are whole numbers - its fast case -, the
 * scanning kernel otherwise or when the summary kernel declines a batch), PRE_ROUTE_SCAN (always the scanning kernel), PRE_ROUTE_SUMMARY (as
 * AUTO, but PRE_ESIZE here when the shape does not fit the summary kernel).  Results do not
 * depend on it. */
#define PRE_ROUTE_AUTO    0
#define PRE_ROUTE_SCAN    1
#define PRE_ROUTE_SUMMARY 2
int pre_route_select(pre_ctx* ctx, int32_t path);

/* Test hook, not part of the method: sets how many polls a device-side wait of this context's
 * kernels makes before it gives up (default 2^22; 0 gives up at the first unsuccessful poll).
 * It exists so that a test can make a wait run out without disturbing the GPU: nothing faults or
 * spins for long, the kernels leave through their ordinary give-up path and pre_status returns
 * PRE_ETIMEOUT. */
int pre_test_set_spin_limit(pre_ctx* ctx, uint32_t polls);

/* Static, human-readable text for a pre_error value. */
const char* pre_strerror(int code);

/* Launch geometry chosen for this context, for reports: number of thread blocks of the
 * persistent routing kernel and instance rows per build tile.  Either pointer may be NULL. */
int pre_query(const pre_ctx* ctx, int32_t* route_blocks, int32_t* tile_rows);

/* More of the same, for reports: out[0] = bytes of shared memory each block of the routing kernel
 * has for resident map rows, out[1] = threads of a routing block, out[2] = blocks of the
 * single-launch anticipator build (0 when this shape uses the two-kernel build), out[3] = the
 * largest table (rows) that build takes. */
int pre_query_layout(const pre_ctx* ctx, int64_t out[4]);

#ifdef __cplusplus
}
#endif
#endif /* PRESERVE_B200_H */

// CPU oracle for the load anticipator and the load-aware request router.
//
// TEST INFRASTRUCTURE ONLY.  This file is the slow, sequential, plainly written
// statement of what the CUDA library must compute.  Nothing in the product path
// may call it; it shares no code with the CUDA sources and includes none of
// their headers.  All pointers are host pointers.
//
// Notation (paper, Sec. 4.3.1 "Instance Load Anticipator" and Sec. 4.3.3
// "Load-aware Request Router"):
//   I  instances, H look-ahead steps (the paper's l), M token capacity.
//   request r = (P prompt tokens, g tokens generated so far, D predicted
//   response tokens, inst).  c_i[j] = anticipated KV tokens of instance i at
//   j decode steps from now = the paper's U_j * M.
//
// Readings taken where the paper is silent (each is repeated where used):
//   * the ramp "U_i*M += P + i, i in [0, D)" is half-open: D steps holding
//     P, P+1, ..., P+D-1 tokens and nothing from step D on;
//   * a request that already generated g tokens is the same ramp seen g steps
//     later: P+g+j tokens at step j for j in [0, D-g);
//   * only the first H steps of a map are stored; the ramp is cut at H;
//   * a request with g >= D is finished and contributes nothing; a request
//     with D < 1, g < 0, P < 0 or inst outside [0, I) is malformed and skipped.
//
// Pins (tests/test_oracle_*.py): brute-force enumeration written separately in
// the tests, the closed forms of a single ramp, the step/rebuild identity, the
// fold/rebuild identity, greedy least-loaded routing as the beta = 0 special
// case, exact rational evaluation of the score; for the refinement a second
// hand-computed example, the closed form of the removed tokens, the chain of
// extensions and the equality with the definition on the refined table; for
// the admission queue a hand-computed example, the plain router as the special
// case that never blocks, and an exact-arithmetic restatement over several calls; for the
// router on full-width maps the plain router as the case l = L, an exact-arithmetic
// restatement with a window, and the equality of the maps with a rebuild.  The capacity rule M and the
// queued_p model are this build's readings, not the paper's: parity unpinned
// for those two (they are inputs, the arithmetic on them is pinned).
#include <cstdint>
#include <cstdlib>
#include <cstring>
#include <vector>

namespace {

inline bool well_formed(int32_t P, int32_t g, int32_t D, int32_t inst, int32_t I) {
    return P >= 0 && g >= 0 && D >= 1 && inst >= 0 && inst < I;
}

// Router score of one instance (Sec. 4.3.3):
//   L = L_p + L_d + beta * L_m,  L_p = queued_p + P,  L_d = current_d + D,
//   L_m = max(0, U_k - T_mem) * M  with  U_k*M = peak.
// Evaluated in binary64 as max(0, peak - T_mem*M) so that the token counts,
// which are whole numbers below 2^53, enter without a division.
inline double score_of(int64_t queued_p, int64_t current_d, int64_t peak, int32_t P, int32_t D,
                       double theta, double beta) {
    double over = (double)peak - theta;
    if (over < 0.0) over = 0.0;
    double lp = (double)(queued_p + (int64_t)P);
    double ld = (double)(current_d + (int64_t)D);
    double lm = beta * over;
    double l = lp + ld;
    l = l + lm;
    return l;
}

// Peak of instance row c[0..H) after virtually adding a new request (P, D):
// the request holds P+j tokens at step j for j < min(D, H) (Sec. 4.3.3,
// "virtually adds r ... returns the peak memory usage over the next l iterations").
inline int64_t peak_with(const int64_t* c, int32_t H, int32_t P, int32_t D) {
    int64_t peak = INT64_MIN;
    for (int32_t j = 0; j < H; ++j) {
        int64_t v = c[j];
        if (j < D) v += (int64_t)P + j;
        if (v > peak) peak = v;
    }
    return peak;
}

}  // namespace

extern "C" {

// Sec. 4.3.1, map update, written as the definition: every live request adds
// its occupancy to each step it is still running.  Also the decode backlog
// current_d_i = sum of (D - g) over the live requests of instance i.
void orc_anticipate(const int32_t* P, const int32_t* g, const int32_t* D, const int32_t* inst,
                    int64_t n, int32_t I, int32_t H, int64_t* curves, int64_t* current_d) {
    std::memset(curves, 0, sizeof(int64_t) * (size_t)I * (size_t)H);
    std::memset(current_d, 0, sizeof(int64_t) * (size_t)I);
    for (int64_t r = 0; r < n; ++r) {
        if (!well_formed(P[r], g[r], D[r], inst[r], I)) continue;
        if (g[r] >= D[r]) continue;  // finished
        int64_t remaining = (int64_t)D[r] - g[r];
        int64_t* c = curves + (size_t)inst[r] * (size_t)H;
        for (int64_t j = 0; j < remaining && j < H; ++j) c[j] += (int64_t)P[r] + g[r] + j;
        current_d[inst[r]] += remaining;
    }
}

// Sec. 4.3.3 taken literally, one arrival after the other.  For each arrival:
// score every instance, pick the least (lowest index on equal scores), then
// really add the request to the chosen instance (map, queued_p, current_d,
// request table) before the next arrival is looked at.
// Returns the number of arrivals routed (stops early when the table is full).
int64_t orc_route_batch(const int32_t* aP, const int32_t* aD, int64_t A, int32_t I, int32_t H,
                        int64_t M, double t_mem, double beta, int64_t* curves, int64_t* queued_p,
                        int64_t* current_d, int32_t* P, int32_t* g, int32_t* D, int32_t* inst,
                        int64_t* n_requests, int64_t max_requests, int32_t* choice, double* score) {
    const double theta = t_mem * (double)M;
    int64_t k = 0;
    for (; k < A; ++k) {
        if (*n_requests >= max_requests) break;
        if (aP[k] < 0 || aD[k] < 1) { choice[k] = -1; if (score) score[k] = 0.0; continue; }  // malformed
        int32_t best = -1;
        double best_l = 0.0;
        for (int32_t i = 0; i < I; ++i) {
            int64_t peak = peak_with(curves + (size_t)i * H, H, aP[k], aD[k]);
            double l = score_of(queued_p[i], current_d[i], peak, aP[k], aD[k], theta, beta);
            if (best < 0 || l < best_l) { best = i; best_l = l; }
        }
        int64_t* c = curves + (size_t)best * H;
        for (int32_t j = 0; j < H && j < aD[k]; ++j) c[j] += (int64_t)aP[k] + j;
        queued_p[best] += aP[k];
        current_d[best] += aD[k];
        int64_t slot = (*n_requests)++;
        P[slot] = aP[k]; g[slot] = 0; D[slot] = aD[k]; inst[slot] = best;
        choice[k] = best;
        if (score) score[k] = best_l;
    }
    for (int64_t r = k; r < A; ++r) { choice[r] = -1; if (score) score[r] = 0.0; }
    return k;
}

// The router on full-width maps (Sec. 4.3.1: the map covers the next L iterations, L the
// largest response the model can produce, while the anticipator projects the load "over the
// next l iterations" for the router, Sec. 4.3.3).  The peak is taken over the first l steps of
// a row of width L; the real update adds the whole ramp, min(D, L) steps.  Everything else is
// orc_route_batch.  With l = L the two are the same function.
int64_t orc_route_window(const int32_t* aP, const int32_t* aD, int64_t A, int32_t I, int32_t L, int32_t l,
                         int64_t M, double t_mem, double beta, int64_t* maps, int64_t* queued_p,
                         int64_t* current_d, int32_t* P, int32_t* g, int32_t* D, int32_t* inst,
                         int64_t* n_requests, int64_t max_requests, int32_t* choice, double* score) {
    const double theta = t_mem * (double)M;
    int64_t k = 0;
    for (; k < A; ++k) {
        if (*n_requests >= max_requests) break;
        if (aP[k] < 0 || aD[k] < 1) { choice[k] = -1; if (score) score[k] = 0.0; continue; }  // malformed
        int32_t best = -1;
        double best_l = 0.0;
        for (int32_t i = 0; i < I; ++i) {
            int64_t peak = peak_with(maps + (size_t)i * L, l, aP[k], aD[k]);      // the next l iterations
            double sc = score_of(queued_p[i], current_d[i], peak, aP[k], aD[k], theta, beta);
            if (best < 0 || sc < best_l) { best = i; best_l = sc; }
        }
        int64_t* c = maps + (size_t)best * L;
        for (int32_t j = 0; j < L && j < aD[k]; ++j) c[j] += (int64_t)aP[k] + j;  // the whole ramp
        queued_p[best] += aP[k];
        current_d[best] += aD[k];
        int64_t slot = (*n_requests)++;
        P[slot] = aP[k]; g[slot] = 0; D[slot] = aD[k]; inst[slot] = best;
        choice[k] = best;
        if (score) score[k] = best_l;
    }
    for (int64_t r = k; r < A; ++r) { choice[r] = -1; if (score) score[r] = 0.0; }
    return k;
}

// Same decisions as orc_route_batch through an identity instead of a rescan.
// For a row c, with  PM[j] = max_{t<=j}(c[t]+t)  and  SM[j] = max_{t>=j} c[t],
//   peak(P, D) = max(P + PM[Dc-1], SM[Dc]),  Dc = min(D, H)   (SM[H] = none),
// because the virtual ramp adds P+t on t < Dc and nothing after.  Only the
// chosen row changes per arrival, so only its PM/SM are rebuilt.  This is an
// accelerator for the large configurations; tests admit it only after it
// reproduces orc_route_batch exactly on the configurations the literal form
// can finish.
int64_t orc_route_batch_fast(const int32_t* aP, const int32_t* aD, int64_t A, int32_t I, int32_t H,
                             int64_t M, double t_mem, double beta, int64_t* curves,
                             int64_t* queued_p, int64_t* current_d, int32_t* P, int32_t* g,
                             int32_t* D, int32_t* inst, int64_t* n_requests, int64_t max_requests,
                             int32_t* choice, double* score) {
    const double theta = t_mem * (double)M;
    std::vector<int64_t> PM((size_t)I * H), SM((size_t)I * H);
    auto rebuild = [&](int32_t i) {
        const int64_t* c = curves + (size_t)i * H;
        int64_t* pm = PM.data() + (size_t)i * H;
        int64_t* sm = SM.data() + (size_t)i * H;
        int64_t m = INT64_MIN;
        for (int32_t j = 0; j < H; ++j) { int64_t v = c[j] + j; if (v > m) m = v; pm[j] = m; }
        m = INT64_MIN;
        for (int32_t j = H - 1; j >= 0; --j) { if (c[j] > m) m = c[j]; sm[j] = m; }
    };
    for (int32_t i = 0; i < I; ++i) rebuild(i);
    int64_t k = 0;
    for (; k < A; ++k) {
        if (*n_requests >= max_requests) break;
        if (aP[k] < 0 || aD[k] < 1) { choice[k] = -1; if (score) score[k] = 0.0; continue; }  // malformed
        const int32_t Dc = aD[k] < H ? aD[k] : H;
        int32_t best = -1;
        double best_l = 0.0;
        for (int32_t i = 0; i < I; ++i) {
            int64_t peak = (int64_t)aP[k] + PM[(size_t)i * H + (Dc - 1)];
            if (Dc < H && SM[(size_t)i * H + Dc] > peak) peak = SM[(size_t)i * H + Dc];
            double l = score_of(queued_p[i], current_d[i], peak, aP[k], aD[k], theta, beta);
            if (best < 0 || l < best_l) { best = i; best_l = l; }
        }
        int64_t* c = curves + (size_t)best * H;
        for (int32_t j = 0; j < Dc; ++j) c[j] += (int64_t)aP[k] + j;
        rebuild(best);
        queued_p[best] += aP[k];
        current_d[best] += aD[k];
        int64_t slot = (*n_requests)++;
        P[slot] = aP[k]; g[slot] = 0; D[slot] = aD[k]; inst[slot] = best;
        choice[k] = best;
        if (score) score[k] = best_l;
    }
    for (int64_t r = k; r < A; ++r) { choice[r] = -1; if (score) score[r] = 0.0; }
    return k;
}

// All instance scores of ONE arrival against the present state, nothing is
// changed.  Used to check single sampled decisions of a long batch.
void orc_score_all(int32_t aP, int32_t aD, int32_t I, int32_t H, int64_t M, double t_mem, double beta,
                   const int64_t* curves, const int64_t* queued_p, const int64_t* current_d,
                   double* score, int64_t* peak) {
    const double theta = t_mem * (double)M;
    for (int32_t i = 0; i < I; ++i) {
        int64_t pk = peak_with(curves + (size_t)i * H, H, aP, aD);
        if (peak) peak[i] = pk;
        score[i] = score_of(queued_p[i], current_d[i], pk, aP, aD, theta, beta);
    }
}

// One decode iteration (iteration-level batching, Sec. 2; the map covers "the
// next iterations", Sec. 4.3.1): every live request has produced one more
// token.  The maps move one step closer: c'[j] = c[j+1]; the step that enters
// the window, H-1, is filled from the requests still running then.  Readings:
// the decode backlog drops by one token per live request, and every queued
// prefill is assumed done within the iteration (queued_p <- 0).
void orc_step(int32_t* P, int32_t* g, int32_t* D, int32_t* inst, int64_t n, int32_t I, int32_t H,
              int64_t* curves, int64_t* queued_p, int64_t* current_d) {
    std::vector<int64_t> enter((size_t)I, 0);
    for (int64_t r = 0; r < n; ++r) {
        if (!well_formed(P[r], g[r], D[r], inst[r], I)) continue;
        if (g[r] >= D[r]) continue;
        current_d[inst[r]] -= 1;
        g[r] += 1;
        // still running H-1 steps after the tick?
        if ((int64_t)D[r] - g[r] > (int64_t)H - 1)
            enter[inst[r]] += (int64_t)P[r] + g[r] + (H - 1);
    }
    for (int32_t i = 0; i < I; ++i) {
        int64_t* c = curves + (size_t)i * H;
        for (int32_t j = 0; j + 1 < H; ++j) c[j] = c[j + 1];
        c[H - 1] = enter[i];
        queued_p[i] = 0;
    }
}

// Signals for the proactive instance scaler (Sec. 4.3.2), read off the maps as they stand.
//   over_count[i] = number of steps j in [0, H) whose anticipated KV usage exceeds
//                   overload_level (95 %) of the capacity:  c_i[j] > overload_level * M;
//   instance i is "potentially overloaded" when that happens in more than overload_share
//   (10 %) of the steps:  over_count[i] > overload_share * H;
//   row_max[i]    = max_j c_i[j]  (the paper's max(U') times M);
//   an instance keeps the scale-down action from firing unless its usage stays below
//   idle_level (T_f = 30 %) throughout the window:  row_max[i] < idle_level * M.
// summary = { number of potentially overloaded instances,
//             number of instances that are NOT below idle_level throughout,
//             sum over instances of row_max }   (the number of instances to isolate is then
//             N_c - summary[2] / (M * T_f), left to the caller).
// Thresholds are binary64 products; token counts (< 2^53) convert exactly.
void orc_scaler_signals(const int64_t* curves, int32_t I, int32_t H, int64_t M, double overload_level,
                        double overload_share, double idle_level, int32_t* over_count, int64_t* row_max,
                        int64_t* summary) {
    const double hot = overload_level * (double)M;
    const double many = overload_share * (double)H;
    const double idle = idle_level * (double)M;
    summary[0] = summary[1] = summary[2] = 0;
    for (int32_t i = 0; i < I; ++i) {
        const int64_t* c = curves + (size_t)i * H;
        int32_t cnt = 0;
        int64_t mx = INT64_MIN;
        for (int32_t j = 0; j < H; ++j) {
            if ((double)c[j] > hot) ++cnt;
            if (c[j] > mx) mx = c[j];
        }
        over_count[i] = cnt;
        row_max[i] = mx;
        if ((double)cnt > many) summary[0] += 1;
        if (!((double)mx < idle)) summary[1] += 1;
        summary[2] += mx;
    }
}

// Refinement of the maps when a request's real response length differs from the predicted
// one (Sec. 4.3.1, the paragraph after the map update).  actual[r] is the real length as the
// serving engine learns it; the call is made after the decode iteration of a tick.
//   * finished early (g < D and the engine reports the request done, actual <= g): the tokens
//     anticipated for the rest of the prediction are taken out again,
//         U_i*M -= P + i   for i in [g, D)     (request steps; window step j = i - g),
//     and the request is closed at its real length (D <- g).
//   * still running at the predicted end (g == D and actual > g): the response is virtually
//     extended by 0.2 times its length so far and the map updated for the extension,
//         U_i*M += P + i   for i in [D, D + E),  E = ceil(D / 5)  (at least one token),
//     D <- D + E.  Repeated on later ticks until the request completes; an extension that
//     overshoots is taken out by the first rule.
// Readings: the paper writes the extension as 0.2 times the ground-truth length, which is not
// known while the request runs; the length reached so far (g = D at that moment) is used, as
// the exact fraction D/5 rounded up.  The decode backlog follows the prediction: -(D - g) on
// an early finish, +E on an extension.  Steps beyond the stored window are cut as in the build.
// counts = { early finishes, extensions, malformed entries skipped }.
void orc_refine(const int32_t* P, const int32_t* g, int32_t* D, const int32_t* inst, const int32_t* actual,
                int64_t n, int32_t I, int32_t H, int64_t* curves, int64_t* current_d, int64_t* counts) {
    counts[0] = counts[1] = counts[2] = 0;
    for (int64_t r = 0; r < n; ++r) {
        if (!well_formed(P[r], g[r], D[r], inst[r], I) || actual[r] < 1) { counts[2] += 1; continue; }
        int64_t* c = curves + (size_t)inst[r] * H;
        if (g[r] < D[r] && actual[r] <= g[r]) {
            for (int64_t i = g[r]; i < D[r]; ++i) {
                const int64_t j = i - g[r];
                if (j < H) c[j] -= (int64_t)P[r] + i;
            }
            current_d[inst[r]] -= (int64_t)D[r] - g[r];
            D[r] = g[r];
            counts[0] += 1;
        } else if (g[r] == D[r] && actual[r] > g[r]) {
            const int64_t E = ((int64_t)D[r] + 4) / 5;
            for (int64_t i = D[r]; i < (int64_t)D[r] + E; ++i) {
                const int64_t j = i - g[r];
                if (j < H) c[j] += (int64_t)P[r] + i;
            }
            current_d[inst[r]] += E;
            D[r] = (int32_t)((int64_t)D[r] + E);
            counts[1] += 1;
        }
    }
}

// Router with its admission queue (Sec. 4.3.3, the sentences before the score: an incoming
// request waits when all instances are overloaded and is turned away when the queue is full).
// The paper does not say when an instance counts as overloaded for the router; the scaler's
// criterion of Sec. 4.3.2 is taken, evaluated on the maps as they stand, without the request:
//   instance i is overloaded  <=>  #{ j in [0,H) : c_i[j] > overload_level * M } > overload_share * H.
// One call handles, in this order, the requests already waiting (oldest first) and then the
// new arrivals.  For each: if every instance is overloaded the request waits (a waiting one
// keeps its place, a new one joins the tail while the queue has room, otherwise it is turned
// away); if not, it is routed exactly as by orc_route_batch.  Maps only grow during a call, so
// once every instance is overloaded it stays so until the call ends.
// The queue is a ring: entry q (0 = oldest) is at (head + q) mod capacity, qstate = {head, length}.
// Results: instance index, -1 malformed or request table full (dropped), -2 waits, -3 turned away;
// for the entries that were waiting at entry in qchoice[q], for the arrivals in choice[k].
// fast != 0 keeps running maxima and overload counts instead of rescanning (same decisions,
// admitted by tests only after it equals the literal mode).
void orc_route_admit(const int32_t* aP, const int32_t* aD, int64_t A, int32_t I, int32_t H, int64_t M,
                     double t_mem, double beta, double overload_level, double overload_share,
                     int32_t* qP, int32_t* qD, int64_t* qstate, int64_t qcap, int32_t* qchoice,
                     int64_t* curves, int64_t* queued_p, int64_t* current_d, int32_t* P, int32_t* g,
                     int32_t* D, int32_t* inst, int64_t* n_requests, int64_t max_requests,
                     int32_t* choice, double* score, int32_t fast) {
    const double theta = t_mem * (double)M;
    const double hot = overload_level * (double)M;
    const double many = overload_share * (double)H;
    const int64_t head = qstate[0], len0 = qstate[1];
    std::vector<int64_t> PM, SM;
    std::vector<int32_t> over;
    auto rebuild = [&](int32_t i) {
        const int64_t* c = curves + (size_t)i * H;
        int64_t* pm = PM.data() + (size_t)i * H;
        int64_t* sm = SM.data() + (size_t)i * H;
        int64_t m = INT64_MIN;
        int32_t cnt = 0;
        for (int32_t j = 0; j < H; ++j) {
            int64_t v = c[j] + j; if (v > m) m = v; pm[j] = m;
            if ((double)c[j] > hot) ++cnt;
        }
        m = INT64_MIN;
        for (int32_t j = H - 1; j >= 0; --j) { if (c[j] > m) m = c[j]; sm[j] = m; }
        over[i] = cnt;
    };
    if (fast) {
        PM.resize((size_t)I * H); SM.resize((size_t)I * H); over.resize((size_t)I);
        for (int32_t i = 0; i < I; ++i) rebuild(i);
    }
    auto all_overloaded = [&]() {
        for (int32_t i = 0; i < I; ++i) {
            int32_t cnt = 0;
            if (fast) cnt = over[i];
            else {
                const int64_t* c = curves + (size_t)i * H;
                for (int32_t j = 0; j < H; ++j) if ((double)c[j] > hot) ++cnt;
            }
            if (!((double)cnt > many)) return false;
        }
        return true;
    };
    bool blocked = false;
    int64_t left = 0;       // waiting entries that stay
    int64_t joined = 0;     // arrivals that joined the queue
    for (int64_t k = 0; k < len0 + A; ++k) {
        const bool waiting = k < len0;
        const int32_t rP = waiting ? qP[(head + k) % qcap] : aP[k - len0];
        const int32_t rD = waiting ? qD[(head + k) % qcap] : aD[k - len0];
        int32_t* out = waiting ? &qchoice[k] : &choice[k - len0];
        double* sc = (!waiting && score) ? &score[k - len0] : nullptr;
        if (sc) *sc = 0.0;
        if (blocked && waiting) { *out = -2; ++left; continue; }      // keeps its place, not looked at
        if (rP < 0 || rD < 1) { *out = -1; continue; }                // malformed: dropped
        if (!blocked) {
            if (*n_requests >= max_requests) { *out = -1; continue; } // request table full: dropped
            if (all_overloaded()) blocked = true;
        }
        if (blocked) {
            if (waiting) { *out = -2; ++left; }
            else if (left + joined < qcap) {
                const int64_t pos = (head + len0 + joined) % qcap;    // behind the last waiting entry
                qP[pos] = rP; qD[pos] = rD;
                ++joined;
                *out = -2;
            } else {
                *out = -3;
            }
            continue;
        }
        const int32_t Dc = rD < H ? rD : H;
        int32_t best = -1;
        double best_l = 0.0;
        for (int32_t i = 0; i < I; ++i) {
            int64_t peak;
            if (fast) {
                peak = (int64_t)rP + PM[(size_t)i * H + (Dc - 1)];
                if (Dc < H && SM[(size_t)i * H + Dc] > peak) peak = SM[(size_t)i * H + Dc];
            } else {
                peak = peak_with(curves + (size_t)i * H, H, rP, rD);
            }
            double l = score_of(queued_p[i], current_d[i], peak, rP, rD, theta, beta);
            if (best < 0 || l < best_l) { best = i; best_l = l; }
        }
        int64_t* c = curves + (size_t)best * H;
        for (int32_t j = 0; j < Dc; ++j) c[j] += (int64_t)rP + j;
        if (fast) rebuild(best);
        queued_p[best] += rP;
        current_d[best] += rD;
        int64_t slot = (*n_requests)++;
        P[slot] = rP; g[slot] = 0; D[slot] = rD; inst[slot] = best;
        *out = best;
        if (sc) *sc = best_l;
    }
    // entries that left are a prefix of the old queue
    qstate[0] = qcap > 0 ? (head + (len0 - left)) % qcap : 0;
    qstate[1] = left + joined;
}

}  // extern "C"

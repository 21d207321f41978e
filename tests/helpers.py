"""Independent, deliberately naive Python restatements used to pin the oracle."""
from fractions import Fraction

import numpy as np


def brute_curves(prompt, generated, predicted, instance, n_inst, horizon):
    """c_i[j] = sum over requests r of instance i still running at step j of (P_r + g_r + j)."""
    c = [[0] * horizon for _ in range(n_inst)]
    for i in range(n_inst):
        for j in range(horizon):
            tot = 0
            for p, g, d, s in zip(prompt, generated, predicted, instance):
                if int(s) == i and j < int(d) - int(g):
                    tot += int(p) + int(g) + j
            c[i][j] = tot
    return np.array(c, dtype=np.int64).reshape(n_inst, horizon)


def exact_route(curves, queued_p, current_d, arr_prompt, arr_predicted, capacity, t_mem=Fraction(4, 5),
                beta=Fraction(1), window=None):
    """Greedy router in exact rational arithmetic on Python ints. Returns choices, scores, final state.
    `window`: peaks are taken over the first `window` steps only (default: the whole row)."""
    c = [[int(v) for v in row] for row in curves]
    q = [int(v) for v in queued_p]
    cd = [int(v) for v in current_d]
    n_inst, horizon = len(c), len(c[0])
    theta = Fraction(t_mem) * capacity
    choices, scores = [], []
    for p, d in zip(arr_prompt, arr_predicted):
        p, d = int(p), int(d)
        best, best_l = None, None
        for i in range(n_inst):
            peak = max(c[i][j] + ((p + j) if j < d else 0) for j in range(horizon if window is None else window))
            l = (q[i] + p) + (cd[i] + d) + Fraction(beta) * max(Fraction(0), peak - theta)
            if best is None or l < best_l:
                best, best_l = i, l
        for j in range(min(d, horizon)):
            c[best][j] += p + j
        q[best] += p
        cd[best] += d
        choices.append(best)
        scores.append(best_l)
    return choices, scores, np.array(c, dtype=np.int64), np.array(q, dtype=np.int64), np.array(cd, dtype=np.int64)


def load_worked_example(path):
    out = {"request": [], "curve": {}, "curve_after": {}, "curve_step": {}}
    for line in open(path):
        line = line.strip()
        if not line or line.startswith("#"):
            continue
        key, *vals = line.split()
        vals = [int(v) for v in vals]
        if key == "request":
            out["request"].append(vals)
        elif key in ("curve", "curve_after", "curve_step"):
            out[key][vals[0]] = vals[1:]
        else:
            out[key] = vals
    return out


def exact_admit(curves, queued_p, current_d, waiting, arrivals, capacity, queue_capacity, level, share,
                t_mem=Fraction(4, 5), beta=Fraction(1)):
    """Router with the admission queue in exact arithmetic: waiting requests (oldest first) then
    arrivals; a request waits when every instance is overloaded (more than share*H steps above
    level*capacity), joins the queue while there is room, is turned away otherwise.
    Returns (results for the waiting ones, results for the arrivals, new queue, curves, queued_p, current_d)."""
    c = np.array(curves, dtype=np.int64)
    q = np.array(queued_p, dtype=np.int64)
    cd = np.array(current_d, dtype=np.int64)
    horizon = c.shape[1]

    def everyone_overloaded():
        for row in c:
            steps = sum(1 for v in row if Fraction(int(v)) > Fraction(level) * capacity)
            if not Fraction(steps) > Fraction(share) * horizon:
                return False
        return True

    stay, joined, res_wait, res_arr = [], [], [], []
    blocked = False
    for k, (p, d) in enumerate(list(waiting) + list(arrivals)):
        is_waiting = k < len(waiting)
        out = res_wait if is_waiting else res_arr
        if not blocked and everyone_overloaded():
            blocked = True
        if blocked:
            if is_waiting:
                stay.append((p, d)); out.append(-2)
            elif len(stay) + len(joined) < queue_capacity:
                joined.append((p, d)); out.append(-2)
            else:
                out.append(-3)
            continue
        ch, _, c, q, cd = exact_route(c, q, cd, [p], [d], capacity, t_mem, beta)
        out.append(ch[0])
    return res_wait, res_arr, stay + joined, c, q, cd

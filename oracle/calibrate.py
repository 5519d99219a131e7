"""Test infrastructure: Algorithm 2 (slope-based per-class uncertainty thresholds, Sec. 3.2)
written out step by step in plain Python integers.  Not part of the product path.

Reading of the algorithm (the paper gives it in outline only):
  * D = validation flows with the fast model's predicted label, whether that prediction was
    correct, and the uncertainty score u.
  * Per class L (flows PREDICTED as L): sort its scores; the candidate thresholds are the
    quantiles q_k = (Q - k)/Q, k = 1..Q, picked by Algorithm 1's rule (1-based index
    ceil(q_k * m), clamped to 1); k = 0 is "nothing assigned", threshold = the class maximum.
  * For each threshold, C_k / I_k = correct / incorrect flows of the class with u > T_k.
  * R = per class, in order of falling threshold, the steps with their increments
    dI = I_k - I_(k-1), dA = (C_k + I_k) - (C_(k-1) + I_(k-1)); steps that assign nothing new
    (dA = 0) are no operating points of their own and are left out; slope = dI / dA.
  * Thresholds start at each class's maximum; while fewer than floor(a * |D|) validation
    flows are assigned, the queue holds the next step of every class, the step with the
    largest slope (compared exactly as fractions; ties: larger dA, then lower class) is
    taken: that class's threshold drops to the step's threshold.
  * A class nobody was predicted as keeps the global maximum of U.
"""
import numpy as np


def per_class_slopes(U, pred, correct, C, Q):
    """R of GetPerClassSlope: list per class of (T, dI, dA) in order of falling threshold."""
    U = np.asarray(U, np.float32)
    pred = np.asarray(pred)
    correct = np.asarray(correct).astype(bool)
    R, tmax = [], []
    for L in range(C):
        sel = pred == L
        u = np.sort(U[sel])
        ok = correct[sel]
        uu = U[sel]
        m = len(u)
        items = []
        if m == 0:
            R.append(items)
            tmax.append(None)
            continue
        tmax.append(np.float32(u[-1]))
        prev_c = prev_i = 0
        for k in range(1, Q + 1):
            idx = -((-(Q - k) * m) // Q)            # ceil((Q-k)*m / Q) in integers
            idx = min(max(idx, 1), m)
            T = np.float32(u[idx - 1])
            c = int(np.count_nonzero(ok & (uu > T)))
            i = int(np.count_nonzero(~ok & (uu > T)))
            dI, dA = i - prev_i, (c + i) - (prev_c + prev_i)
            if dA > 0:
                items.append((T, dI, dA))
            prev_c, prev_i = c, i
        R.append(items)
    return R, tmax


def per_class_thresholds(U, pred, correct, C, Q, a_num, a_den):
    """GetPerClassThresholds for the assigned portion a = a_num / a_den.
    Returns (tau fp32[C], number of validation flows assigned, order of the steps taken)."""
    U = np.asarray(U, np.float32)
    R, tmax = per_class_slopes(U, pred, correct, C, Q)
    gmax = np.float32(U.max()) if len(U) else np.float32(0)
    TD = [gmax if t is None else t for t in tmax]
    nxt = [0] * C
    target = (a_num * len(U)) // a_den
    assigned, taken = 0, []
    while assigned < target:
        best = None
        for L in range(C):
            if nxt[L] < len(R[L]):
                _, dI, dA = R[L][nxt[L]]
                if best is None:
                    best = L
                else:
                    _, bI, bA = R[best][nxt[best]]
                    lhs, rhs = dI * bA, bI * dA      # dI/dA > bI/bA ?
                    if lhs > rhs or (lhs == rhs and dA > bA):
                        best = L
        if best is None:
            break
        T, dI, dA = R[best][nxt[best]]
        TD[best] = T
        assigned += dA
        nxt[best] += 1
        taken.append(best)
    return np.array(TD, np.float32), assigned, taken

"""ctypes front end of the CPU oracle (test infrastructure; see serveflow_oracle.c).

Only tests, the smoke check and the benchmark's CPU-baseline leg import this
package.  It shares nothing with the CUDA library.  `build()` compiles the C file
with gcc; the functions below marshal numpy arrays and call it.
"""
import ctypes as C
import os
import subprocess
from concurrent.futures import ThreadPoolExecutor

import numpy as np

_HERE = os.path.dirname(os.path.abspath(__file__))
_SRC = os.path.join(_HERE, "serveflow_oracle.c")
_SO = os.path.join(_HERE, "libserveflow_oracle.so")
_lib = None

TAU_MARGIN = float(np.float32(np.log(0.7 / 0.3)))   # ln(0.7/0.3) rounded to fp32


def build(force=False):
    """Compile the oracle (no FMA contraction, no fast-math)."""
    if force or not os.path.exists(_SO) or os.path.getmtime(_SO) < os.path.getmtime(_SRC):
        cmd = ["gcc", "-O2", "-ffp-contract=off", "-fno-fast-math", "-std=c11", "-shared", "-fPIC",
               "-o", _SO, _SRC, "-lm"]
        subprocess.run(cmd, check=True)
    return _SO


def lib():
    global _lib
    if _lib is None:
        build()
        _lib = C.CDLL(_SO)
        _lib.sfo_u128_to_f32.restype = C.c_float
        _lib.sfo_u128_to_f32.argtypes = [C.c_uint64, C.c_uint64]
        _lib.sfo_bf16_round.restype = C.c_float
        _lib.sfo_bf16_round.argtypes = [C.c_float]
        _lib.sfo_least_confidence.restype = C.c_float
        _lib.sfo_entropy.restype = C.c_double
        _lib.sfo_sigmoid.restype = C.c_double
        _lib.sfo_sigmoid.argtypes = [C.c_double]
        _lib.sfo_route_lc.restype = C.c_uint64
        _lib.sfo_route_absmargin.restype = C.c_uint64
        _lib.sfo_route_entropy.restype = C.c_uint64
        _lib.sfo_route_softmax_lc.restype = C.c_uint64
        _lib.sfo_softmax_lc.restype = C.c_double
        _lib.sfo_ilog.restype = C.c_uint32
        _lib.sfo_ilog.argtypes = [C.c_uint32]
    return _lib


def _p(a):
    return None if a is None else a.ctypes.data_as(C.c_void_p)


def _c(a, dt):
    return np.ascontiguousarray(a, dtype=dt)


def u128_to_f32(v):
    v = int(v)
    return float(lib().sfo_u128_to_f32(C.c_uint64(v >> 64), C.c_uint64(v & ((1 << 64) - 1))))


def bf16_round(x):
    return float(lib().sfo_bf16_round(C.c_float(float(x))))


def ilog(a):
    return int(lib().sfo_ilog(C.c_uint32(int(a))))


def sigmoid(m):
    return float(lib().sfo_sigmoid(C.c_double(float(m))))


def least_confidence(p):
    p = _c(p, np.float32)
    return float(lib().sfo_least_confidence(_p(p), C.c_uint32(p.shape[-1])))


def entropy(p):
    p = _c(p, np.float32)
    return float(lib().sfo_entropy(_p(p), C.c_uint32(p.shape[-1])))


def _ranges(n, threads):
    threads = max(1, min(int(threads), int(n) if n else 1))
    step = (n + threads - 1) // threads
    return [(lo, min(n, lo + step)) for lo in range(0, n, step)] if n else []


def _run(fn, n, threads):
    """Run fn(lo, hi) over contiguous ranges; ctypes calls release the GIL."""
    rs = _ranges(n, threads)
    if len(rs) <= 1:
        for lo, hi in rs:
            fn(lo, hi)
        return
    with ThreadPoolExecutor(max_workers=len(rs)) as ex:
        list(ex.map(lambda r: fn(*r), rs))


def extract_features(pk, N, F, n_valid=None, threads=1):
    size = _c(pk["size"], np.uint16)
    iat = _c(pk["iat_us"], np.uint32)
    db = _c(pk["dir_bits"], np.uint32)
    n, pitch = size.shape
    words = db.shape[1]
    assert words == (pitch + 31) // 32
    nv = None if n_valid is None else _c(n_valid, np.uint8)
    feat = np.empty((n, F), dtype=np.float32)
    L = lib()

    def work(lo, hi):
        L.sfo_extract_features(_p(size[lo:hi]), _p(iat[lo:hi]), _p(db[lo:hi]),
                               None if nv is None else _p(nv[lo:hi]), C.c_uint64(hi - lo),
                               C.c_uint32(pitch), C.c_uint32(N), C.c_uint32(F), _p(feat[lo:hi]))
    _run(work, n, threads)
    return feat


def header_bits(bytes128, sec_len, sub):
    """Subscribed columns of the 1024 first-packet header bits as -1 / 0 / 1."""
    b = _c(bytes128, np.uint8); sl = _c(sec_len, np.uint8); sub = _c(sub, np.uint16)
    n = b.shape[0]
    assert b.shape[1] == 128 and sl.shape == (n, 3)
    out = np.empty((n, sub.shape[0]), np.float32)
    lib().sfo_header_bits(_p(b), _p(sl), C.c_uint64(n), _p(sub), C.c_uint32(sub.shape[0]), _p(out))
    return out


def forest_infer(forest, feat, want_leaf_idx=False, threads=1):
    feat = _c(feat, np.float32)
    n, F = feat.shape
    T, d, Cc = forest["T"], forest["depth"], forest["C"]
    fid = _c(forest["fid"], np.uint16)
    thr = _c(forest["thr"], np.float32)
    leaf = _c(forest["leaf"], np.float32)
    li = np.empty((n, T), dtype=np.uint16) if want_leaf_idx else None
    L = lib()
    if forest["kind"] == "rf":
        out = np.empty((n, Cc), dtype=np.float32)

        def work(lo, hi):
            L.sfo_forest_rf(_p(feat[lo:hi]), C.c_uint64(hi - lo), C.c_uint32(F), C.c_uint32(T), C.c_uint32(d),
                            C.c_uint32(Cc), _p(fid), _p(thr), _p(leaf), _p(out[lo:hi]),
                            None if li is None else _p(li[lo:hi]))
    elif forest["kind"] == "gbdt_mc":
        out = np.empty((n, Cc), dtype=np.float32)

        def work(lo, hi):
            L.sfo_forest_gbdt_mc(_p(feat[lo:hi]), C.c_uint64(hi - lo), C.c_uint32(F), C.c_uint32(T), C.c_uint32(d),
                                 C.c_uint32(Cc), _p(fid), _p(thr), _p(leaf), _p(out[lo:hi]),
                                 None if li is None else _p(li[lo:hi]))
    else:
        out = np.empty((n,), dtype=np.float32)

        def work(lo, hi):
            L.sfo_forest_gbdt(_p(feat[lo:hi]), C.c_uint64(hi - lo), C.c_uint32(F), C.c_uint32(T), C.c_uint32(d),
                              _p(fid), _p(thr), _p(leaf), _p(out[lo:hi]),
                              None if li is None else _p(li[lo:hi]))
    _run(work, n, threads)
    return (out, li) if want_leaf_idx else out


def route_lc(prob, tau):
    prob = _c(prob, np.float32)
    n, Cc = prob.shape
    tau = _c(np.broadcast_to(np.asarray(tau, dtype=np.float32), (Cc,)), np.float32)
    score = np.empty(n, np.float32)
    label = np.empty(n, np.uint8)
    dec = np.empty(n, np.uint8)
    ids = np.empty(n, np.uint32)
    k = lib().sfo_route_lc(_p(prob), C.c_uint64(n), C.c_uint32(Cc), _p(tau), _p(score), _p(label),
                           _p(dec), _p(ids), C.c_uint64(n))
    return {"score": score, "label": label, "decision": dec, "esc_ids": ids[:k].copy(), "n_esc": int(k)}


def route_entropy(prob, tau):
    prob = _c(prob, np.float32)
    n, Cc = prob.shape
    tau = _c(np.broadcast_to(np.asarray(tau, dtype=np.float32), (Cc,)), np.float32)
    score = np.empty(n, np.float32)
    label = np.empty(n, np.uint8)
    dec = np.empty(n, np.uint8)
    ids = np.empty(n, np.uint32)
    k = lib().sfo_route_entropy(_p(prob), C.c_uint64(n), C.c_uint32(Cc), _p(tau), _p(score), _p(label),
                                _p(dec), _p(ids), C.c_uint64(n))
    return {"score": score, "label": label, "decision": dec, "esc_ids": ids[:k].copy(), "n_esc": int(k)}


def route_softmax_lc(margin, tau):
    margin = _c(margin, np.float32)
    n, Cc = margin.shape
    tau = _c(np.broadcast_to(np.asarray(tau, dtype=np.float32), (Cc,)), np.float32)
    score = np.empty(n, np.float32)
    label = np.empty(n, np.uint8)
    dec = np.empty(n, np.uint8)
    ids = np.empty(n, np.uint32)
    k = lib().sfo_route_softmax_lc(_p(margin), C.c_uint64(n), C.c_uint32(Cc), _p(tau), _p(score), _p(label),
                                   _p(dec), _p(ids), C.c_uint64(n))
    return {"score": score, "label": label, "decision": dec, "esc_ids": ids[:k].copy(), "n_esc": int(k)}


def route_absmargin(margin, tau_m=TAU_MARGIN):
    margin = _c(margin, np.float32)
    n = margin.shape[0]
    score = np.empty(n, np.float32)
    label = np.empty(n, np.uint8)
    dec = np.empty(n, np.uint8)
    ids = np.empty(n, np.uint32)
    k = lib().sfo_route_absmargin(_p(margin), C.c_uint64(n), C.c_float(tau_m), _p(score), _p(label),
                                  _p(dec), _p(ids), C.c_uint64(n))
    return {"score": score, "label": label, "decision": dec, "esc_ids": ids[:k].copy(), "n_esc": int(k)}


def universal_thresholds(U, q_percent):
    """Algorithm 1 for quantiles q = q_percent[j] / 100."""
    U = _c(U, np.float32)
    q = _c(np.atleast_1d(q_percent), np.uint32)
    out = np.empty(q.shape[0], np.float32)
    lib().sfo_universal_thresholds(_p(U), C.c_uint64(U.shape[0]), _p(q), C.c_uint32(100),
                                   C.c_uint32(q.shape[0]), _p(out))
    return out


def wide_rows(layout, esc_ids, wide, P, to_bf16, n_valid=None, P_real=None, threads=1):
    """layout 0: P x 16 fields (MLP); layout 1: P x 8 channels (CNN)."""
    ids = _c(esc_ids, np.uint32)
    size = _c(wide["size"], np.uint16)
    iat = _c(wide["iat_us"], np.uint32)
    db = _c(wide["dir_bits"], np.uint32)
    hdr = _c(wide["hdr"], np.uint8)
    pitch = size.shape[1]
    H = hdr.shape[2]
    nv = None if n_valid is None else _c(n_valid, np.uint8)
    W = 16 if layout == 0 else 8
    rows = np.empty((ids.shape[0], P * W), dtype=np.float32)
    L = lib()

    def work(lo, hi):
        L.sfo_wide_rows(C.c_int(layout), _p(ids[lo:hi]), C.c_uint64(hi - lo), _p(size), _p(iat), _p(db),
                        _p(hdr), _p(nv), C.c_uint32(pitch), C.c_uint32(H), C.c_uint32(P),
                        C.c_uint32(P if P_real is None else P_real), C.c_int(int(to_bf16)), _p(rows[lo:hi]))
    _run(work, ids.shape[0], threads)
    return rows


def mlp(model, rows, bf16, threads=1):
    rows = _c(rows, np.float32)
    dims = _c(model["dims"], np.uint32)
    nl = len(model["W"])
    Ws = [_c(w, np.float32) for w in model["W"]]
    bs = [_c(b, np.float32) for b in model["b"]]
    Wp = (C.c_void_p * nl)(*[w.ctypes.data for w in Ws])
    bp = (C.c_void_p * nl)(*[b.ctypes.data for b in bs])
    n = rows.shape[0]
    assert rows.shape[1] == int(dims[0])
    logits = np.empty((n, int(dims[-1])), np.float32)
    label = np.empty(n, np.uint8)
    L = lib()

    def work(lo, hi):
        L.sfo_mlp(_p(rows[lo:hi]), C.c_uint64(hi - lo), C.c_uint32(nl), _p(dims), Wp, bp, C.c_int(int(bf16)),
                  _p(logits[lo:hi]), _p(label[lo:hi]))
    _run(work, n, threads)
    return logits, label


def cnn(model, rows, bf16, threads=1):
    rows = _c(rows, np.float32)
    m = model
    n = rows.shape[0]
    assert rows.shape[1] == m["L"] * m["Cin"]
    arrs = [_c(m[k], np.float32) for k in ("w1", "b1", "w2", "b2", "w3", "b3")]
    logits = np.empty((n, m["n_cls"]), np.float32)
    label = np.empty(n, np.uint8)
    L = lib()

    def work(lo, hi):
        L.sfo_cnn(_p(rows[lo:hi]), C.c_uint64(hi - lo), C.c_uint32(m["L"]), C.c_uint32(m["Cin"]),
                  C.c_uint32(m["C1"]), C.c_uint32(m["C2"]), C.c_uint32(m["k"]), C.c_uint32(m["n_cls"]),
                  *[_p(a) for a in arrs], C.c_int(int(bf16)), _p(logits[lo:hi]), _p(label[lo:hi]))
    _run(work, n, threads)
    return logits, label


def merge(label_fast, esc_ids, label_slow):
    lf = _c(label_fast, np.uint8)
    ids = _c(esc_ids, np.uint32)
    ls = _c(label_slow, np.uint8)
    n = lf.shape[0]
    label = np.empty(n, np.uint8)
    stage = np.empty(n, np.uint8)
    lib().sfo_merge(_p(lf), C.c_uint64(n), _p(ids), C.c_uint64(ids.shape[0]), _p(ls), _p(label), _p(stage))
    return label, stage


def serve_batch(cfg, fast_pk, wide_pk, forest, slow_model, tau, threads=1):
    """All stages in order on one batch; returns every intermediate result."""
    feat = extract_features(fast_pk, cfg.N, cfg.F, threads=threads)
    fo = forest_infer(forest, feat, threads=threads)
    r = route_lc(fo, tau) if forest["kind"] == "rf" else route_absmargin(fo, float(np.asarray(tau).ravel()[0]))
    bf16 = cfg.slow_dtype == "bf16"
    layout = 0 if cfg.slow == "mlp" else 1
    rows = wide_rows(layout, r["esc_ids"], wide_pk, cfg.P, bf16, threads=threads)
    if cfg.slow == "mlp":
        logits, label_slow = mlp(slow_model, rows, bf16, threads=threads)
    else:
        logits, label_slow = cnn(slow_model, rows, bf16, threads=threads)
    label, stage = merge(r["label"], r["esc_ids"], label_slow)
    return {"feat": feat, "fast_out": fo, **r, "rows": rows, "logits": logits, "label_slow": label_slow,
            "label_final": label, "stage": stage}


def serve_batch3(cfg, fast_pk, wide_pk, fastest, fast, slow_model, tau1, tau2, threads=1):
    """Three-tier cascade (Sec. 3.1): the fastest model answers what it is sure of; the rest goes to the
    fast model on the SAME features; what that is still unsure of goes to the slow model, which sees more
    packets.  tau1 / tau2 are per-class thresholds (Sec. 3.2).  stage = 1, 2 or 3."""
    feat = extract_features(fast_pk, cfg.N, cfg.F, threads=threads)
    p1 = forest_infer(fastest, feat, threads=threads)
    r1 = route_lc(p1, tau1)
    ids1 = r1["esc_ids"]
    p2 = forest_infer(fast, feat[ids1], threads=threads) if len(ids1) else np.zeros((0, fast["C"]), np.float32)
    route2 = route_softmax_lc if fast["kind"] == "gbdt_mc" else route_lc      # boosted fast model: softmax of its margins
    r2 = route2(p2, tau2) if len(ids1) else {"esc_ids": np.zeros(0, np.uint32), "label": np.zeros(0, np.uint8),
                                               "n_esc": 0, "score": np.zeros(0, np.float32)}
    ids2 = ids1[r2["esc_ids"]]
    bf16 = cfg.slow_dtype == "bf16"
    rows = wide_rows(0 if cfg.slow == "mlp" else 1, ids2, wide_pk, cfg.P, bf16, threads=threads)
    if cfg.slow == "mlp":
        logits, label_slow = mlp(slow_model, rows, bf16, threads=threads)
    else:
        logits, label_slow = cnn(slow_model, rows, bf16, threads=threads)
    n = feat.shape[0]
    label = r1["label"].copy()
    stage = np.ones(n, np.uint8)
    label[ids1] = r2["label"]; stage[ids1] = 2
    label[ids2] = label_slow; stage[ids2] = 3
    return {"feat": feat, "prob1": p1, "ids1": ids1, "prob2": p2, "ids2": ids2, "rows": rows, "logits": logits,
            "label_slow": label_slow, "label_final": label, "stage": stage, "label1": r1["label"], "label2": r2["label"],
            "score2": r2["score"]}

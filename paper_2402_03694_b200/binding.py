"""ctypes binding of libserveflow.so: the same calls as include/serveflow.h.

Argument marshalling only - every step of the serving path runs in the library's
CUDA kernels.  Device buffers are torch tensors (torch is used for memory and
streams, nothing else); host arrays are numpy.  If the shared library is missing
the import fails loudly: there is no fallback path.
"""
import ctypes as C
import os

import numpy as np

_HERE = os.path.dirname(os.path.abspath(__file__))
LIB_PATH = os.path.join(_HERE, "libserveflow.so")

SF_OK = 0
SF_ERR_ARG, SF_ERR_ALLOC, SF_ERR_CUDA, SF_ERR_CAPACITY = -1, -2, -3, -4
SF_ERR_TABLE_FULL, SF_ERR_UNSUPPORTED, SF_ERR_DEVICE_TIMEOUT = -5, -6, -7
SF_ERR_STATIC_LIMIT = -8
SF_NOALLOC_MAX_FLOWS = 4194304
SF_RF, SF_GBDT, SF_GBDT_MC = 0, 1, 2
SF_LC_GT, SF_ABSMARGIN_LT, SF_ENTROPY_GT, SF_SOFTMAX_LC_GT = 0, 1, 2, 3
SF_MLP16, SF_CNN8 = 0, 1
SF_F32, SF_BF16 = 0, 1
SF_TAU_MARGIN_DEFAULT = float.fromhex("0x1.b1d106p-1")


class SfError(RuntimeError):
    def __init__(self, status, where):
        self.status = status
        msg = "%s: %s (%d)" % (where, _lib().sf_strerror(status).decode(), status)
        if status == SF_ERR_CUDA or status == SF_ERR_ALLOC:
            msg += " - " + _lib().sf_last_cuda_error().decode()
        super().__init__(msg)


class sf_counters(C.Structure):
    _fields_ = [("n_flows", C.c_uint64), ("n_fast_done", C.c_uint64), ("n_escalated", C.c_uint64),
                ("n_slow_done", C.c_uint64), ("n_missed", C.c_uint64), ("n_dropped_after_decision", C.c_uint64),
                ("device_error", C.c_int32), ("reserved", C.c_int32)]


class sf_packets(C.Structure):
    _fields_ = [("size", C.c_void_p), ("iat_us", C.c_void_p), ("dir_bits", C.c_void_p), ("hdr", C.c_void_p),
                ("n_valid", C.c_void_p), ("n_flows", C.c_uint32), ("pitch_pkts", C.c_uint32),
                ("hdr_bytes", C.c_uint32)]


class sf_route_cfg(C.Structure):
    _fields_ = [("rule", C.c_int), ("tau", C.c_void_p), ("wide_layout", C.c_int), ("row_dtype", C.c_int),
                ("P", C.c_uint32), ("P_real", C.c_uint32), ("capacity", C.c_uint32)]


class sf_pkt_batch(C.Structure):
    _fields_ = [("src", C.c_void_p), ("dst", C.c_void_p), ("sport", C.c_void_p), ("dport", C.c_void_p),
                ("proto", C.c_void_p), ("dir", C.c_void_p), ("size", C.c_void_p), ("iat_us", C.c_void_p),
                ("hdr", C.c_void_p), ("n", C.c_uint32)]


class sf_batch_result(C.Structure):
    _fields_ = [("n_new_flows", C.c_uint32), ("n_fast_fired", C.c_uint32), ("n_fast_done", C.c_uint32),
                ("n_escalated", C.c_uint32), ("n_slow_fired", C.c_uint32), ("n_dropped_after_decision", C.c_uint32),
                ("n_missed", C.c_uint32), ("reserved", C.c_uint32)]


class sf_key(C.Structure):
    _fields_ = [("src", C.c_uint32), ("dst", C.c_uint32), ("sport", C.c_uint16), ("dport", C.c_uint16),
                ("proto", C.c_uint8), ("pad", C.c_uint8 * 3)]


class sf_flow_result(C.Structure):
    _fields_ = [("found", C.c_uint8), ("stage", C.c_uint8), ("label_fast", C.c_uint8), ("label_slow", C.c_uint8),
                ("n_pkts", C.c_uint32), ("score", C.c_float)]


KEY_DTYPE = np.dtype([("src", "<u4"), ("dst", "<u4"), ("sport", "<u2"), ("dport", "<u2"), ("proto", "u1"),
                      ("pad", "u1", (3,))])
FLOW_RESULT_DTYPE = np.dtype([("found", "u1"), ("stage", "u1"), ("label_fast", "u1"), ("label_slow", "u1"),
                              ("n_pkts", "<u4"), ("score", "<f4")])

EXPORTS = [
    "sf_strerror", "sf_last_cuda_error", "sf_version", "sf_ctx_create", "sf_ctx_destroy", "sf_ctx_poll",
    "sf_ctx_set_timing", "sf_ctx_get_timing",
    "sf_extract_features", "sf_header_bits", "sf_forest_create", "sf_forest_destroy", "sf_fast_infer", "sf_route",
    "sf_route_noalloc",
    "sf_universal_thresholds", "sf_universal_thresholds_dev", "sf_per_class_thresholds", "sf_mlp_create", "sf_cnn_create", "sf_slow_destroy", "sf_slow_infer",
    "sf_serve_batch", "sf_serve_batch3", "sf_serve_batch_host", "sf_serve_batch_intermediates",
    "sf_table_create", "sf_table_destroy", "sf_table_ingest", "sf_table_ingest_host", "sf_table_lookup", "sf_table_set_time", "sf_table_sweep", "sf_table_set_pipelined", "sf_table_flush",
]

_L = None


def _lib():
    global _L
    if _L is None:
        if not os.path.exists(LIB_PATH):
            raise ImportError("libserveflow.so is not built: run `python -m paper_2402_03694_b200.build` "
                              "(there is no CPU fallback)")
        L = C.CDLL(LIB_PATH)
        for name in EXPORTS:
            getattr(L, name)                         # fail loudly on a missing symbol
        for name in ("sf_strerror", "sf_last_cuda_error", "sf_version"):
            getattr(L, name).restype = C.c_char_p
        L.sf_strerror.argtypes = [C.c_int]
        for name in ("sf_ctx_destroy", "sf_forest_destroy", "sf_slow_destroy", "sf_table_destroy"):
            getattr(L, name).restype = None
            getattr(L, name).argtypes = [C.c_void_p]
        V, U32, I = C.c_void_p, C.c_uint32, C.c_int
        L.sf_ctx_create.argtypes = [C.POINTER(V), I, C.c_size_t]
        L.sf_ctx_poll.argtypes = [V, C.POINTER(sf_counters), I, V]
        L.sf_ctx_set_timing.argtypes = [V, I]
        L.sf_ctx_get_timing.argtypes = [V, U32, V, V]
        L.sf_extract_features.argtypes = [V, C.POINTER(sf_packets), U32, U32, V, V]
        L.sf_header_bits.argtypes = [V, V, V, U32, V, U32, V, V]
        L.sf_forest_create.argtypes = [V, I, U32, U32, U32, U32, V, V, V, C.POINTER(V)]
        L.sf_fast_infer.argtypes = [V, V, V, U32, V, V, V]
        L.sf_route.argtypes = [V, C.POINTER(sf_route_cfg), V, U32, U32, C.POINTER(sf_packets), V, V, V, V, V, V, V]
        L.sf_route_noalloc.argtypes = [I, C.POINTER(sf_route_cfg), V, U32, U32, V, V, V, V, V, V, V]
        L.sf_universal_thresholds.argtypes = [V, C.c_uint64, V, U32, U32, V]
        L.sf_universal_thresholds_dev.argtypes = [V, V, U32, V, U32, U32, V, V]
        L.sf_per_class_thresholds.argtypes = [V, V, V, V, U32, U32, U32, U32, U32, V, V, V]
        L.sf_mlp_create.argtypes = [V, I, U32, V, C.POINTER(V), C.POINTER(V), C.POINTER(V)]
        L.sf_cnn_create.argtypes = [V, I, U32, U32, U32, U32, U32, U32, V, V, V, V, V, V, C.POINTER(V)]
        L.sf_slow_infer.argtypes = [V, V, V, V, U32, V, V, V]
        L.sf_serve_batch.argtypes = [V, V, V, C.POINTER(sf_packets), U32, U32, C.POINTER(sf_packets),
                                     C.POINTER(sf_route_cfg), V, V, V, V]
        L.sf_serve_batch_host.argtypes = L.sf_serve_batch.argtypes
        L.sf_serve_batch3.argtypes = [V, V, V, V, C.POINTER(sf_packets), U32, U32, C.POINTER(sf_packets),
                                      C.POINTER(sf_route_cfg), C.POINTER(sf_route_cfg), V, V, V, V]
        L.sf_serve_batch_intermediates.argtypes = [V] + [C.POINTER(V)] * 7
        L.sf_table_create.argtypes = [V, U32, U32, U32, U32, C.POINTER(V)]
        L.sf_table_ingest.argtypes = [V, V, C.POINTER(sf_pkt_batch), V, U32, V, C.POINTER(sf_route_cfg), V, V]
        L.sf_table_ingest_host.argtypes = L.sf_table_ingest.argtypes
        L.sf_table_lookup.argtypes = [V, V, V, U32, V, V]
        L.sf_table_set_pipelined.argtypes = [V, V, I]
        L.sf_table_flush.argtypes = [V, V, V]
        L.sf_table_set_time.argtypes = [V, U32]
        L.sf_table_sweep.argtypes = [V, V, U32, U32, C.c_int, V, V]
        _L = L
    return _L


def _check(status, where):
    if status != SF_OK:
        raise SfError(status, where)


def _dp(t):
    """Device (or host) address of a torch tensor / numpy array / int / None."""
    if t is None:
        return None
    if isinstance(t, int):
        return t
    if isinstance(t, np.ndarray):
        return t.ctypes.data
    return t.data_ptr()


def _stream(stream):
    if stream is None:
        import torch
        return torch.cuda.current_stream().cuda_stream
    return stream if isinstance(stream, int) else stream.cuda_stream


def sf_version():
    return _lib().sf_version().decode()


def sf_strerror(status):
    return _lib().sf_strerror(status).decode()


def make_packets(size, iat_us, dir_bits, hdr=None, n_valid=None, n_flows=None, pitch_pkts=None, hdr_bytes=None):
    """sf_packets from tensors/arrays shaped [n][pitch], [n][pitch], [n][words], [n][pitch][H]."""
    p = sf_packets()
    p.size, p.iat_us, p.dir_bits, p.hdr, p.n_valid = _dp(size), _dp(iat_us), _dp(dir_bits), _dp(hdr), _dp(n_valid)
    p.n_flows = int(size.shape[0] if n_flows is None else n_flows)
    p.pitch_pkts = int(size.shape[1] if pitch_pkts is None else pitch_pkts)
    p.hdr_bytes = int((hdr.shape[2] if hdr is not None else 0) if hdr_bytes is None else hdr_bytes)
    p._keep = (size, iat_us, dir_bits, hdr, n_valid)
    return p


def make_route_cfg(rule, tau, wide_layout, row_dtype, P, capacity, P_real=0):
    c = sf_route_cfg()
    c.rule, c.tau, c.wide_layout, c.row_dtype = rule, _dp(tau), wide_layout, row_dtype
    c.P, c.P_real, c.capacity = int(P), int(P_real), int(capacity)
    c._keep = tau
    return c


def sf_ctx_create(device=0, workspace_bytes=0):
    h = C.c_void_p()
    _check(_lib().sf_ctx_create(C.byref(h), device, workspace_bytes), "sf_ctx_create")
    return h


def sf_ctx_destroy(ctx):
    _lib().sf_ctx_destroy(ctx)


def sf_ctx_poll(ctx, reset=False, stream=None, raise_on_error=True):
    c = sf_counters()
    st = _lib().sf_ctx_poll(ctx, C.byref(c), int(reset), _stream(stream))
    if raise_on_error:
        _check(st, "sf_ctx_poll")
    return c


SF_TIMER_NAMES = ("extract", "forest", "score", "gather", "gemm", "head", "merge", "table", "pull")


def sf_ctx_set_timing(ctx, enable):
    _check(_lib().sf_ctx_set_timing(ctx, int(enable)), "sf_ctx_set_timing")


def sf_ctx_get_timing(ctx, back=0, stream=None):
    """dict name -> milliseconds for the call made `back` calls ago."""
    out = np.zeros(len(SF_TIMER_NAMES), np.float32)
    _check(_lib().sf_ctx_get_timing(ctx, back, out.ctypes.data, _stream(stream)), "sf_ctx_get_timing")
    return {k: float(v) for k, v in zip(SF_TIMER_NAMES, out)}


def sf_extract_features(ctx, pk, N, F, feat_out, stream=None):
    _check(_lib().sf_extract_features(ctx, C.byref(pk), N, F, _dp(feat_out), _stream(stream)), "sf_extract_features")


def sf_header_bits(ctx, bytes128, sec_len, n, sub, m, out, stream=None):
    _check(_lib().sf_header_bits(ctx, _dp(bytes128), _dp(sec_len), n, _dp(sub), m, _dp(out), _stream(stream)),
           "sf_header_bits")


def sf_forest_create(ctx, kind, T, depth, F, Cn, fid, thr, leaf):
    fid = np.ascontiguousarray(fid, np.uint16)
    thr = np.ascontiguousarray(thr, np.float32)
    leaf = np.ascontiguousarray(leaf, np.float32)
    h = C.c_void_p()
    _check(_lib().sf_forest_create(ctx, kind, T, depth, F, Cn, fid.ctypes.data, thr.ctypes.data, leaf.ctypes.data,
                                   C.byref(h)), "sf_forest_create")
    return h


def sf_forest_destroy(forest):
    _lib().sf_forest_destroy(forest)


def sf_fast_infer(ctx, forest, feat, n, out, leaf_idx_out=None, stream=None):
    _check(_lib().sf_fast_infer(ctx, forest, _dp(feat), n, _dp(out), _dp(leaf_idx_out), _stream(stream)),
           "sf_fast_infer")


def sf_route(ctx, cfg, fast_out, n, Cn, wide, esc_ids_out, n_esc_out, rows_out=None, decision_out=None,
             label_fast_out=None, score_out=None, stream=None):
    _check(_lib().sf_route(ctx, C.byref(cfg), _dp(fast_out), n, Cn, C.byref(wide) if wide is not None else None,
                           _dp(esc_ids_out), _dp(n_esc_out), _dp(rows_out), _dp(decision_out), _dp(label_fast_out),
                           _dp(score_out), _stream(stream)), "sf_route")


def sf_route_noalloc(device, cfg, fast_out, n, Cn, esc_ids_out, n_esc_out, decision_out=None, label_fast_out=None,
                     score_out=None, status_out=None, stream=None):
    """Assignment (score, threshold, ascending ids, count) for callers that may not allocate
    device memory: no context, scratch built into the library, n <= SF_NOALLOC_MAX_FLOWS."""
    _check(_lib().sf_route_noalloc(device, C.byref(cfg), _dp(fast_out), n, Cn, _dp(esc_ids_out), _dp(n_esc_out),
                                   _dp(decision_out), _dp(label_fast_out), _dp(score_out), _dp(status_out),
                                   _stream(stream)), "sf_route_noalloc")


def sf_universal_thresholds(scores, q_num, q_den=100):
    scores = np.ascontiguousarray(scores, np.float32)
    q = np.ascontiguousarray(np.atleast_1d(q_num), np.uint32)
    out = np.empty(q.shape[0], np.float32)
    _check(_lib().sf_universal_thresholds(scores.ctypes.data, scores.shape[0], q.ctypes.data, q_den, q.shape[0],
                                          out.ctypes.data), "sf_universal_thresholds")
    return out


def sf_universal_thresholds_dev(ctx, scores, n, q_num, q_den, tau_out, stream=None):
    q = np.ascontiguousarray(np.atleast_1d(q_num), np.uint32)
    _check(_lib().sf_universal_thresholds_dev(ctx, _dp(scores), n, q.ctypes.data, q_den, q.shape[0], _dp(tau_out),
                                              _stream(stream)), "sf_universal_thresholds_dev")


def sf_per_class_thresholds(ctx, scores, label, correct, n, n_classes, Q, a_num, a_den, stream=None):
    tau = np.empty(n_classes, np.float32)
    assigned = C.c_uint64(0)
    _check(_lib().sf_per_class_thresholds(ctx, _dp(scores), _dp(label), _dp(correct), n, n_classes, Q, a_num, a_den,
                                          tau.ctypes.data, C.addressof(assigned), _stream(stream)), "sf_per_class_thresholds")
    return tau, int(assigned.value)


def sf_mlp_create(ctx, dtype, dims, W, b):
    nl = len(W)
    dims = np.ascontiguousarray(dims, np.uint32)
    Ws = [np.ascontiguousarray(w, np.float32) for w in W]
    bs = [np.ascontiguousarray(x, np.float32) for x in b]
    Wp = (C.c_void_p * nl)(*[w.ctypes.data for w in Ws])
    bp = (C.c_void_p * nl)(*[x.ctypes.data for x in bs])
    h = C.c_void_p()
    _check(_lib().sf_mlp_create(ctx, dtype, nl, dims.ctypes.data, Wp, bp, C.byref(h)), "sf_mlp_create")
    return h


def sf_cnn_create(ctx, dtype, m):
    a = [np.ascontiguousarray(m[k], np.float32) for k in ("w1", "b1", "w2", "b2", "w3", "b3")]
    h = C.c_void_p()
    _check(_lib().sf_cnn_create(ctx, dtype, m["L"], m["Cin"], m["C1"], m["C2"], m["k"], m["n_cls"],
                                *[x.ctypes.data for x in a], C.byref(h)), "sf_cnn_create")
    return h


def sf_slow_destroy(slow):
    _lib().sf_slow_destroy(slow)


def sf_slow_infer(ctx, slow, rows, n_rows_dev, capacity, logits_out, label_out=None, stream=None):
    _check(_lib().sf_slow_infer(ctx, slow, _dp(rows), _dp(n_rows_dev), capacity, _dp(logits_out), _dp(label_out),
                                _stream(stream)), "sf_slow_infer")


def sf_serve_batch(ctx, forest, slow, fast_ctx, N, F, slow_ctx, cfg, label_out, stage_out, n_esc_out=None,
                   stream=None):
    _check(_lib().sf_serve_batch(ctx, forest, slow, C.byref(fast_ctx), N, F, C.byref(slow_ctx), C.byref(cfg),
                                 _dp(label_out), _dp(stage_out), _dp(n_esc_out), _stream(stream)), "sf_serve_batch")


def sf_serve_batch3(ctx, fastest, fast, slow, fast_ctx, N, F, slow_ctx, cfg_fastest, cfg_fast, label_out, stage_out,
                    n_esc_out=None, stream=None):
    _check(_lib().sf_serve_batch3(ctx, fastest, fast, slow, C.byref(fast_ctx), N, F, C.byref(slow_ctx), C.byref(cfg_fastest),
                                  C.byref(cfg_fast), _dp(label_out), _dp(stage_out), _dp(n_esc_out), _stream(stream)),
           "sf_serve_batch3")


def sf_serve_batch_host(ctx, forest, slow, fast_ctx_host, N, F, slow_ctx_host, cfg_host_tau, label_host_out,
                        stage_host_out, n_esc_host_out=None, stream=None):
    _check(_lib().sf_serve_batch_host(ctx, forest, slow, C.byref(fast_ctx_host), N, F, C.byref(slow_ctx_host),
                                      C.byref(cfg_host_tau), _dp(label_host_out), _dp(stage_host_out),
                                      _dp(n_esc_host_out), _stream(stream)), "sf_serve_batch_host")


def sf_serve_batch_intermediates(ctx):
    """Device addresses (ints) of the last sf_serve_batch's intermediates."""
    ptrs = [C.c_void_p() for _ in range(7)]
    _check(_lib().sf_serve_batch_intermediates(ctx, *[C.byref(p) for p in ptrs]), "sf_serve_batch_intermediates")
    names = ("feat", "fast_out", "esc_ids", "rows", "logits", "label_fast", "label_slow")
    return {k: p.value for k, p in zip(names, ptrs)}


def sf_table_create(ctx, log2_slots, fast_pkts, slow_pkts, slow_slabs):
    h = C.c_void_p()
    _check(_lib().sf_table_create(ctx, log2_slots, fast_pkts, slow_pkts, slow_slabs, C.byref(h)), "sf_table_create")
    return h


def sf_table_destroy(table):
    _lib().sf_table_destroy(table)


def make_pkt_batch(src, dst, sport, dport, proto, dir_, size, iat_us, hdr, n=None):
    b = sf_pkt_batch()
    b.src, b.dst, b.sport, b.dport, b.proto = _dp(src), _dp(dst), _dp(sport), _dp(dport), _dp(proto)
    b.dir, b.size, b.iat_us, b.hdr = _dp(dir_), _dp(size), _dp(iat_us), _dp(hdr)
    b.n = int(src.shape[0] if n is None else n)
    b._keep = (src, dst, sport, dport, proto, dir_, size, iat_us, hdr)
    return b


def sf_table_ingest(ctx, table, batch, forest, F, slow, cfg, result_dev, stream=None):
    _check(_lib().sf_table_ingest(ctx, table, C.byref(batch), forest, F, slow, C.byref(cfg), _dp(result_dev),
                                  _stream(stream)), "sf_table_ingest")


def sf_table_ingest_host(ctx, table, batch_host, forest, F, slow, cfg, stream=None):
    """batch_host: sf_pkt_batch of HOST planes (numpy or pinned torch tensors); returns the batch's counts."""
    res = sf_batch_result()
    _check(_lib().sf_table_ingest_host(ctx, table, C.byref(batch_host), forest, F, slow, C.byref(cfg), C.addressof(res),
                                       _stream(stream)), "sf_table_ingest_host")
    return res


SWEEP_FIELDS = ("expired_pending", "expired_assigned", "expired_done", "rearmed", "live")     # first 5 of 8 uint32


def sf_table_set_time(table, now):
    _check(_lib().sf_table_set_time(table, now & 0xFFFFFFFF), "sf_table_set_time")


def sf_table_sweep(ctx, table, now, idle_timeout, rearm, result_dev, stream=None):
    _check(_lib().sf_table_sweep(ctx, table, now & 0xFFFFFFFF, idle_timeout, int(bool(rearm)), _dp(result_dev), _stream(stream)),
           "sf_table_sweep")


def sf_table_set_pipelined(ctx, table, on):
    _check(_lib().sf_table_set_pipelined(ctx, table, int(on)), "sf_table_set_pipelined")


def sf_table_flush(ctx, table, stream=None):
    _check(_lib().sf_table_flush(ctx, table, _stream(stream)), "sf_table_flush")


def sf_table_lookup(ctx, table, keys_dev, n, out_dev, stream=None):
    _check(_lib().sf_table_lookup(ctx, table, _dp(keys_dev), n, _dp(out_dev), _stream(stream)), "sf_table_lookup")

"""GPU parity: each stage of the CUDA library, called through the C ABI, against the
CPU oracle on the same seeded inputs.  Integer / index / fast-model outputs must be
bit-exact; slow-model logits within 1e-4 (fp32) or 2e-2 (bf16) absolute."""
import numpy as np
import pytest

import flowgen
import oracle

torch = pytest.importorskip("torch")
pytestmark = pytest.mark.gpu

TOL_F32 = 1e-4
TOL_BF16 = 2e-2


@pytest.fixture(scope="module")
def env():
    if not torch.cuda.is_available():
        pytest.skip("no CUDA device")
    from paper_2402_03694_b200 import build, binding as sf, harness as hz
    build.build()
    ctx = sf.sf_ctx_create(0, 1 << 20)
    yield sf, hz, ctx
    sf.sf_ctx_poll(ctx, raise_on_error=False)
    sf.sf_ctx_destroy(ctx)


def bits(a):
    return np.ascontiguousarray(a, np.float32).view(np.uint32)


# ------------------------------------------------------------------ S1 -------
@pytest.mark.parametrize("N,F,n,pitch", [
    (8, 24, 4096, 8), (16, 48, 5003, 16), (32, 64, 3001, 32), (8, 32, 777, 8),
    (8, 24, 1000, 64),      # window shorter than the row pitch (wide planes)
    (5, 16, 300, 12),       # pitch not a multiple of 8: scalar-load path
    (1, 8, 129, 8), (8, 64, 1, 8),
])
def test_extract_bit_exact(env, N, F, n, pitch):
    sf, hz, ctx = env
    pk = flowgen.gen_packets(500 + N + F, n, pitch, H=0)
    pk["iat_us"][0, :] = 2 ** 32 - 1
    if n > 2:
        pk["iat_us"][1, ::2] = 0
        pk["iat_us"][1, 1::2] = 2 ** 32 - 1
        pk["size"][2, :] = 65535
    ref = oracle.extract_features(pk, N, F)
    d = hz.upload_packets(pk, with_hdr=False)
    out = torch.empty((n, F), dtype=torch.float32, device="cuda")
    sf.sf_extract_features(ctx, d["struct"], N, F, out)
    torch.cuda.synchronize()
    assert np.array_equal(bits(out.cpu().numpy()), bits(ref))


def test_extract_short_flows(env):
    sf, hz, ctx = env
    n, N, F = 2500, 16, 48
    pk = flowgen.gen_packets(41, n, 16, H=0)
    nv = np.random.default_rng(2).integers(0, 20, size=n).astype(np.uint8)
    ref = oracle.extract_features(pk, N, F, n_valid=nv)
    d = hz.upload_packets(pk, n_valid=nv, with_hdr=False)
    out = torch.empty((n, F), dtype=torch.float32, device="cuda")
    sf.sf_extract_features(ctx, d["struct"], N, F, out)
    assert np.array_equal(bits(out.cpu().numpy()), bits(ref))


def test_extract_rejects_bad_arguments(env):
    sf, hz, ctx = env
    pk = flowgen.gen_packets(1, 16, 8, H=0)
    d = hz.upload_packets(pk, with_hdr=False)
    out = torch.empty((16, 24), dtype=torch.float32, device="cuda")
    for N, F in ((0, 24), (33, 24), (9, 24), (8, 20), (8, 72)):
        with pytest.raises(sf.SfError) as e:
            sf.sf_extract_features(ctx, d["struct"], N, F, out)
        assert e.value.status == sf.SF_ERR_ARG


# ------------------------------------------------------------------ S2 -------
def _features(n, N, F, seed):
    pk = flowgen.gen_packets(seed, n, N, H=0)
    return oracle.extract_features(pk, N, F, threads=4)


@pytest.mark.parametrize("kind,T,d,F,C,n", [
    ("rf", 16, 8, 24, 4, 4096),
    ("rf", 10, 12, 48, 8, 3000),     # depth-12 trees: one tree per shared-memory chunk
    ("rf", 7, 10, 64, 16, 1500),
    ("rf", 5, 3, 8, 3, 600),         # class count that is not a multiple of 4
    ("gbdt", 70, 6, 32, 2, 5001),    # 64 trees per chunk + a ragged second chunk
    ("gbdt", 3, 1, 8, 2, 33),
    ("rf", 5, 12, 64, 16, 700),      # largest shapes: 128 KB feature tile, one 32 KB tree per chunk
    ("gbdt", 4, 12, 64, 2, 900),     # 48 KB tree images (nodes + leaves) next to the 128 KB tile
    ("rf", 33, 2, 24, 4, 513),       # many trees per chunk, odd count (ragged group), one flow past a block
])
def test_forest_bit_exact(env, kind, T, d, F, C, n):
    sf, hz, ctx = env
    N = {8: 8, 24: 8, 32: 8, 48: 16, 64: 32}[F]
    feat = _features(n, N, F, 600 + T)
    fo = flowgen.gen_forest(700 + T, kind, T, d, F, C, feat)
    ref, ref_li = oracle.forest_infer(fo, feat, want_leaf_idx=True)
    h = hz.make_forest(ctx, fo)
    fd = hz.dev(feat)
    out = torch.empty((n, C) if kind == "rf" else (n,), dtype=torch.float32, device="cuda")
    li = torch.empty((n, T), dtype=torch.uint16, device="cuda")
    sf.sf_fast_infer(ctx, h, fd, n, out, li)
    torch.cuda.synchronize()
    assert np.array_equal(li.cpu().numpy(), ref_li)
    assert np.array_equal(bits(out.cpu().numpy()), bits(ref))
    out2 = torch.empty_like(out)
    sf.sf_fast_infer(ctx, h, fd, n, out2, None)           # leaf indices are optional
    assert torch.equal(out, out2)
    sf.sf_forest_destroy(h)


def test_forest_summation_order_is_tree_order(env):
    sf, hz, ctx = env
    vals = [2.0 ** 24, 1.0, 1.0, -(2.0 ** 24)]
    fo = {"kind": "gbdt", "T": 4, "depth": 1, "F": 8, "C": 2, "fid": np.zeros((4, 1), np.uint16),
          "thr": np.zeros((4, 1), np.float32), "leaf": np.array([[v, v] for v in vals], np.float32)}
    h = hz.make_forest(ctx, fo)
    out = torch.empty(5, dtype=torch.float32, device="cuda")
    sf.sf_fast_infer(ctx, h, torch.zeros((5, 8), device="cuda"), 5, out)
    assert np.all(out.cpu().numpy() == 0.0)
    sf.sf_forest_destroy(h)


# ------------------------------------------------------------------ S3 -------
def test_route_least_confidence_bit_exact(env):
    sf, hz, ctx = env
    sf.sf_ctx_poll(ctx, reset=True)
    n, C = 10007, 8
    rng = np.random.default_rng(11)
    prob = rng.dirichlet([0.5] * C, size=n).astype(np.float32)
    prob[5] = 1.0 / C                                            # all-equal row: label 0
    tau = rng.uniform(0.3, 0.6, size=C).astype(np.float32)
    prob[7] = 0; prob[7, 3] = 1 - tau[3]; prob[7, 0] = tau[3]    # near the threshold
    ref = oracle.route_lc(prob, tau)
    P, H = 64, 13
    wide = flowgen.gen_packets(12, n, P, H)
    nv = np.full(n, 255, np.uint8); nv[ref["esc_ids"][:50]] = 17
    w = hz.upload_packets(wide, n_valid=nv)
    for dtype in (sf.SF_BF16, sf.SF_F32):
        cfg = sf.make_route_cfg(sf.SF_LC_GT, hz.dev(tau), sf.SF_MLP16, dtype, P, n)
        ids = torch.full((n,), 0xFFFFFFFF, dtype=torch.uint32, device="cuda")
        n_esc = torch.zeros(1, dtype=torch.uint32, device="cuda")
        rows = torch.zeros((n, P * 16), dtype=torch.bfloat16 if dtype == sf.SF_BF16 else torch.float32, device="cuda")
        dec = torch.empty(n, dtype=torch.uint8, device="cuda")
        lab = torch.empty(n, dtype=torch.uint8, device="cuda")
        sc = torch.empty(n, dtype=torch.float32, device="cuda")
        sf.sf_route(ctx, cfg, hz.dev(prob), n, C, w["struct"], ids, n_esc, rows, dec, lab, sc)
        torch.cuda.synchronize()
        k = int(n_esc.cpu().numpy()[0])
        assert k == ref["n_esc"]
        assert np.array_equal(ids.cpu().numpy()[:k], ref["esc_ids"])
        assert np.array_equal(dec.cpu().numpy(), ref["decision"])
        assert np.array_equal(lab.cpu().numpy(), ref["label"])
        assert np.array_equal(bits(sc.cpu().numpy()), bits(ref["score"]))
        ref_rows = oracle.wide_rows(0, ref["esc_ids"], wide, P, dtype == sf.SF_BF16, n_valid=nv, threads=4)
        got = rows[:k].float().cpu().numpy()
        assert np.array_equal(bits(got), bits(ref_rows))
    c = sf.sf_ctx_poll(ctx, reset=True)
    assert c.n_flows == 2 * n and c.n_escalated == 2 * ref["n_esc"] and c.n_fast_done == 2 * (n - ref["n_esc"])


def test_route_absmargin_and_cnn_layout(env):
    sf, hz, ctx = env
    n, P, H = 6001, 128, 5
    rng = np.random.default_rng(13)
    margin = (rng.normal(size=n) * 2.24).astype(np.float32)
    margin[3] = np.float32(oracle.TAU_MARGIN)          # equal to the threshold: strict < keeps it
    margin[4] = -np.float32(oracle.TAU_MARGIN)
    ref = oracle.route_absmargin(margin)
    wide = flowgen.gen_packets(14, n, P, H)
    w = hz.upload_packets(wide)
    tau = hz.dev(np.array([sf.SF_TAU_MARGIN_DEFAULT], np.float32))
    assert np.float32(sf.SF_TAU_MARGIN_DEFAULT) == np.float32(oracle.TAU_MARGIN)
    cfg = sf.make_route_cfg(sf.SF_ABSMARGIN_LT, tau, sf.SF_CNN8, sf.SF_BF16, P, n)
    ids = torch.zeros(n, dtype=torch.uint32, device="cuda")
    n_esc = torch.zeros(1, dtype=torch.uint32, device="cuda")
    rows = torch.zeros((n, P * 8), dtype=torch.bfloat16, device="cuda")
    dec = torch.empty(n, dtype=torch.uint8, device="cuda")
    lab = torch.empty(n, dtype=torch.uint8, device="cuda")
    sf.sf_route(ctx, cfg, hz.dev(margin), n, 2, w["struct"], ids, n_esc, rows, dec, lab, None)
    k = int(n_esc.cpu().numpy()[0])
    assert k == ref["n_esc"] and ref["decision"][3] == 0 and ref["decision"][4] == 0
    assert np.array_equal(ids.cpu().numpy()[:k], ref["esc_ids"])
    assert np.array_equal(dec.cpu().numpy(), ref["decision"]) and np.array_equal(lab.cpu().numpy(), ref["label"])
    ref_rows = oracle.wide_rows(1, ref["esc_ids"], wide, P, True, threads=4)
    assert np.array_equal(bits(rows[:k].float().cpu().numpy()), bits(ref_rows))
    sf.sf_ctx_poll(ctx, reset=True)


@pytest.mark.parametrize("layout,H,P,n,shift", [(0, 13, 9, 7, 0), (0, 13, 9, 7, 1), (0, 13, 9, 7, 2), (1, 13, 11, 5, 0), (1, 5, 7, 3, 3)])
def test_route_header_bytes_odd_planes(env, layout, H, P, n, shift):
    """The gather reads a packet's header bytes as the aligned 32-bit words that contain them.  Planes whose
    size is not a multiple of four (the last word is partial), a header stride wider than the bytes used, and a
    header plane that does not start on a 4-byte boundary (byte loads instead) must all give the oracle's rows."""
    sf, hz, ctx = env
    C = 4
    rng = np.random.default_rng(41 + shift)
    prob = rng.dirichlet([0.5] * C, size=n).astype(np.float32)
    tau = np.full(C, -1.0, np.float32)                     # every flow is assigned
    wide = flowgen.gen_packets(42, n, P, H)
    t = {k: hz.dev(wide[k]) for k in ("size", "iat_us", "dir_bits")}
    buf = torch.zeros(n * P * H + 8, dtype=torch.uint8, device="cuda")
    hv = buf[shift:shift + n * P * H].view(n, P, H)
    hv.copy_(hz.dev(wide["hdr"]))
    assert hv.data_ptr() % 4 == shift % 4
    st = sf.make_packets(t["size"], t["iat_us"], t["dir_bits"], hv, None)
    W = 16 if layout == 0 else 8
    cfg = sf.make_route_cfg(sf.SF_LC_GT, hz.dev(tau), sf.SF_MLP16 if layout == 0 else sf.SF_CNN8, sf.SF_BF16, P, n)
    ids = torch.zeros(n, dtype=torch.uint32, device="cuda")
    n_esc = torch.zeros(1, dtype=torch.uint32, device="cuda")
    rows = torch.zeros((n, P * W), dtype=torch.bfloat16, device="cuda")
    sf.sf_route(ctx, cfg, hz.dev(prob), n, C, st, ids, n_esc, rows)
    assert int(n_esc.cpu().numpy()[0]) == n
    ref_rows = oracle.wide_rows(layout, np.arange(n, dtype=np.uint32), wide, P, True)
    assert np.array_equal(bits(rows.float().cpu().numpy()), bits(ref_rows))
    sf.sf_ctx_poll(ctx, reset=True)


def test_route_zero_padding_and_empty_and_overflow(env):
    sf, hz, ctx = env
    n, C = 3000, 4
    rng = np.random.default_rng(15)
    prob = rng.dirichlet([0.5] * C, size=n).astype(np.float32)
    tau = np.full(C, 0.4, np.float32)
    ref = oracle.route_lc(prob, tau)
    wide = flowgen.gen_packets(16, n, 64, 13)
    w = hz.upload_packets(wide)
    # 64 real packets in a 128-packet row
    cfg = sf.make_route_cfg(sf.SF_LC_GT, hz.dev(tau), sf.SF_MLP16, sf.SF_BF16, 128, n, P_real=64)
    ids = torch.zeros(n, dtype=torch.uint32, device="cuda")
    n_esc = torch.zeros(1, dtype=torch.uint32, device="cuda")
    rows = torch.ones((n, 2048), dtype=torch.bfloat16, device="cuda")
    sf.sf_route(ctx, cfg, hz.dev(prob), n, C, w["struct"], ids, n_esc, rows)
    k = int(n_esc.cpu().numpy()[0])
    ref_rows = oracle.wide_rows(0, ref["esc_ids"], wide, 128, True, P_real=64, threads=4)
    assert k == ref["n_esc"] and np.array_equal(bits(rows[:k].float().cpu().numpy()), bits(ref_rows))
    # nothing assigned
    cfg0 = sf.make_route_cfg(sf.SF_LC_GT, hz.dev(np.full(C, 2.0, np.float32)), sf.SF_MLP16, sf.SF_BF16, 64, n)
    sf.sf_route(ctx, cfg0, hz.dev(prob), n, C, None, ids, n_esc)
    assert int(n_esc.cpu().numpy()[0]) == 0
    # empty batch
    sf.sf_route(ctx, cfg0, hz.dev(prob), 0, C, None, ids, n_esc)
    assert int(n_esc.cpu().numpy()[0]) == 0
    assert sf.sf_ctx_poll(ctx, reset=True).device_error == 0
    # capacity overflow: count saturates, the prefix is still right, the error word says so
    cap = ref["n_esc"] // 2
    cfgc = sf.make_route_cfg(sf.SF_LC_GT, hz.dev(tau), sf.SF_MLP16, sf.SF_BF16, 64, cap)
    ids2 = torch.full((n,), 0xFFFFFFFF, dtype=torch.uint32, device="cuda")
    sf.sf_route(ctx, cfgc, hz.dev(prob), n, C, None, ids2, n_esc)
    assert int(n_esc.cpu().numpy()[0]) == cap
    got = ids2.cpu().numpy()
    assert np.array_equal(got[:cap], ref["esc_ids"][:cap]) and np.all(got[cap:] == 0xFFFFFFFF)
    c = sf.sf_ctx_poll(ctx, reset=True, raise_on_error=False)
    assert c.device_error == sf.SF_ERR_CAPACITY
    assert sf.sf_ctx_poll(ctx).device_error == 0


# ------------------------------------------------------------------ S4 -------
def _run_slow(sf, hz, ctx, handle, rows_t, n_rows, cap, n_cls):
    cnt = hz.dev(np.array([n_rows], np.uint32))
    logits = torch.full((cap, n_cls), float("nan"), dtype=torch.float32, device="cuda")
    label = torch.full((cap,), 255, dtype=torch.uint8, device="cuda")
    sf.sf_ctx_poll(ctx, reset=True)
    sf.sf_slow_infer(ctx, handle, rows_t, cnt, cap, logits, label)
    torch.cuda.synchronize()
    c = sf.sf_ctx_poll(ctx, reset=True)
    assert c.device_error == 0 and c.n_slow_done == n_rows
    return logits.cpu().numpy(), label.cpu().numpy()


def _check_labels(ref_logits, ref_label, got_label, tol):
    s = np.sort(ref_logits, axis=1)
    clear = (s[:, -1] - s[:, -2]) >= 2 * tol if ref_logits.shape[1] > 1 else np.ones(len(ref_label), bool)
    assert np.array_equal(got_label[clear], ref_label[clear])


def test_mlp_fp32(env):
    sf, hz, ctx = env
    m = flowgen.gen_mlp(21, (1024, 256, 256, 4))
    n_rows, cap = 1000, 1100
    rows = np.random.default_rng(3).uniform(0, 1, size=(cap, 1024)).astype(np.float32)
    ref, ref_label = oracle.mlp(m, rows[:n_rows], False, threads=8)
    h = sf.sf_mlp_create(ctx, sf.SF_F32, m["dims"], m["W"], m["b"])
    logits, label = _run_slow(sf, hz, ctx, h, hz.dev(rows), n_rows, cap, 4)
    assert np.max(np.abs(logits[:n_rows] - ref)) <= TOL_F32
    assert np.all(np.isnan(logits[n_rows:])) and np.all(label[n_rows:] == 255)     # rows past the count untouched
    _check_labels(ref, ref_label, label[:n_rows], TOL_F32)
    sf.sf_slow_destroy(h)


@pytest.mark.parametrize("dims,n_rows,cap", [
    ((64, 64, 4), 128, 128),              # one tile, one K slice
    ((128, 128, 8), 300, 384),            # ragged last tile
    ((256, 256, 256, 2), 130, 1000),      # BN = 256, count far below capacity
    ((192, 320, 64, 16), 515, 600),       # BN = 64 path, K not a power of two
    ((256, 256, 256, 2), 1, 1000),        # sixteen rows or fewer: served on CUDA cores inside the same launches
    ((192, 320, 64, 16), 7, 600),
    ((2048, 1024, 8), 16, 64),
    ((2048, 1024, 8), 17, 64),            # one row more: back on the tensor cores
    # capacities beyond 65,536 rows: the head is folded into the last hidden layer's epilogue (row panels per CTA)
    ((256, 512, 512, 8), 777, 66000),     # two 256-column tiles per panel, 8 logits per row
    ((256, 512, 512, 8), 66000, 66000),   # every panel of every CTA, ragged last panel
    ((192, 320, 384, 16), 1500, 70000),   # three 128-column tiles per panel, 16 logits per row
    ((128, 192, 5), 300, 66001),          # three 64-column tiles per panel, odd class count
    ((256, 512, 512, 4), 900, 66000),     # four logits kept per row
    ((256, 512, 512, 3), 515, 66000),     # three classes in the four-logit form
    ((256, 512, 512, 2), 515, 66000),     # two logits kept per row
    ((128, 256, 3), 300, 66001),          # a single column tile per panel: the head keeps its own launch
])
def test_mlp_bf16_small_integers_are_exact(env, dims, n_rows, cap):
    """Integer-valued bf16 operands with small sums: every product and partial sum is
    exactly representable, so the tensor-core result must equal integer arithmetic."""
    sf, hz, ctx = env
    rng = np.random.default_rng(sum(dims))
    nl = len(dims) - 1
    W = [rng.integers(-2, 3, size=(dims[l + 1], dims[l])).astype(np.float32) for l in range(nl)]
    b = [rng.integers(-3, 4, size=dims[l + 1]).astype(np.float32) for l in range(nl)]
    # sparsify so that activations stay below 256 (exact in bf16)
    for l in range(nl):
        W[l] *= (rng.random(W[l].shape) < 8.0 / dims[l])
    x = rng.integers(0, 3, size=(cap, dims[0])).astype(np.float32)
    h = x[:n_rows].astype(np.int64)
    for l in range(nl):
        h = h @ W[l].astype(np.int64).T + b[l].astype(np.int64)
        if l + 1 < nl:
            h = np.maximum(h, 0)
            assert h.max() < 256
    m = {"dims": dims, "W": W, "b": b}
    o_logits, _ = oracle.mlp(m, x[:n_rows], True, threads=4)
    assert np.array_equal(o_logits, h.astype(np.float32))
    hd = sf.sf_mlp_create(ctx, sf.SF_BF16, dims, W, b)
    logits, label = _run_slow(sf, hz, ctx, hd, hz.dev(x).to(torch.bfloat16), n_rows, cap, dims[-1])
    assert np.array_equal(logits[:n_rows], h.astype(np.float32))
    assert np.array_equal(label[:n_rows], np.argmax(h, axis=1).astype(np.uint8))
    assert np.all(np.isnan(logits[n_rows:]))
    sf.sf_slow_destroy(hd)


@pytest.mark.parametrize("dims,n_rows,extra", [((1024, 512, 512, 2), 700, 57), ((2048, 1024, 1024, 1024, 8), 400, 57), ((2048, 1024, 1024, 1024, 8), 11, 57),
                                               ((2048, 1024, 1024, 1024, 8), 3000, 70000), ((1024, 512, 512, 2), 2500, 70000)])
def test_mlp_bf16_within_tolerance(env, dims, n_rows, extra):
    sf, hz, ctx = env
    m = flowgen.gen_mlp(33, dims)
    wide = flowgen.gen_packets(34, n_rows, dims[0] // 16, 13)
    rows = oracle.wide_rows(0, np.arange(n_rows, dtype=np.uint32), wide, dims[0] // 16, True, threads=4)
    ref, ref_label = oracle.mlp(m, rows, True, threads=8)
    hd = sf.sf_mlp_create(ctx, sf.SF_BF16, m["dims"], m["W"], m["b"])
    cap = n_rows + extra             # beyond 65,536 rows of capacity the head runs inside the last hidden layer's launch
    rt = torch.zeros((cap, dims[0]), dtype=torch.bfloat16, device="cuda")
    rt[:n_rows] = hz.dev(rows).to(torch.bfloat16)
    logits, label = _run_slow(sf, hz, ctx, hd, rt, n_rows, cap, dims[-1])
    assert np.max(np.abs(logits[:n_rows] - ref)) <= TOL_BF16
    _check_labels(ref, ref_label, label[:n_rows], TOL_BF16)
    # zero rows: nothing is written
    logits0, _ = _run_slow(sf, hz, ctx, hd, rt, 0, cap, dims[-1])
    assert np.all(np.isnan(logits0))
    sf.sf_slow_destroy(hd)


@pytest.mark.parametrize("arch", ["mlp_f32", "mlp_bf16", "cnn"])
def test_slow_model_row_count_above_capacity_is_clamped(env, arch):
    """The row count is a device word of the caller.  A value above `capacity` must not make the
    kernels read or write past the buffers: the first `capacity` rows are answered, nothing
    beyond them is touched, and the context reports SF_ERR_CAPACITY."""
    sf, hz, ctx = env
    cap, guard = 150, 64
    if arch == "cnn":
        m = flowgen.gen_cnn(5, 128, 8, 64, 128, 5, 16)
        rows = _cnn_rows(cap + guard, 9)
        ref, _ = oracle.cnn(m, rows[:cap], True, threads=8)
        h = sf.sf_cnn_create(ctx, sf.SF_BF16, m)
        rt, n_cls, tol = hz.dev(rows).to(torch.bfloat16), 16, TOL_BF16
    else:
        bf = arch == "mlp_bf16"
        dims = (256, 128, 128, 4)
        m = flowgen.gen_mlp(6, dims)
        rows = np.random.default_rng(4).uniform(0, 1, size=(cap + guard, dims[0])).astype(np.float32)
        if bf:
            rows = torch.from_numpy(rows).to(torch.bfloat16).float().numpy()      # exactly representable inputs
        ref, _ = oracle.mlp(m, rows[:cap], bf, threads=8)
        h = sf.sf_mlp_create(ctx, sf.SF_BF16 if bf else sf.SF_F32, m["dims"], m["W"], m["b"])
        rt = hz.dev(rows).to(torch.bfloat16) if bf else hz.dev(rows)
        n_cls, tol = 4, (TOL_BF16 if bf else TOL_F32)
    cnt = hz.dev(np.array([cap + 5], np.uint32))
    logits = torch.full((cap + guard, n_cls), float("nan"), dtype=torch.float32, device="cuda")
    label = torch.full((cap + guard,), 255, dtype=torch.uint8, device="cuda")
    sf.sf_ctx_poll(ctx, reset=True)
    sf.sf_slow_infer(ctx, h, rt, cnt, cap, logits, label)
    torch.cuda.synchronize()
    c = sf.sf_ctx_poll(ctx, reset=True, raise_on_error=False)
    assert c.device_error == sf.SF_ERR_CAPACITY and c.n_slow_done == cap
    lg, lb = logits.cpu().numpy(), label.cpu().numpy()
    assert np.max(np.abs(lg[:cap] - ref)) <= tol
    assert np.all(np.isnan(lg[cap:])) and np.all(lb[cap:] == 255)
    assert sf.sf_ctx_poll(ctx).device_error == 0
    sf.sf_slow_destroy(h)


def test_create_rejects_unsupported_shapes(env):
    sf, hz, ctx = env
    W = [np.zeros((48, 100), np.float32), np.zeros((4, 48), np.float32)]
    b = [np.zeros(48, np.float32), np.zeros(4, np.float32)]
    with pytest.raises(sf.SfError) as e:
        sf.sf_mlp_create(ctx, sf.SF_BF16, (100, 48, 4), W, b)
    assert e.value.status == sf.SF_ERR_UNSUPPORTED
    with pytest.raises(sf.SfError):
        sf.sf_forest_create(ctx, sf.SF_RF, 1, 13, 8, 2, np.zeros((1, 8191)), np.zeros((1, 8191)), np.zeros((1, 8192, 2)))
    with pytest.raises(sf.SfError):      # feature id out of range
        sf.sf_forest_create(ctx, sf.SF_RF, 1, 1, 8, 2, np.full((1, 1), 9), np.zeros((1, 1)), np.zeros((1, 2, 2)))


# ------------------------------------------------------------------ S4: CNN --
def _cnn_rows(n_rows, seed):
    wide = flowgen.gen_packets(seed, n_rows, 128, 5)
    return oracle.wide_rows(1, np.arange(n_rows, dtype=np.uint32), wide, 128, True, threads=4)


def test_cnn_tap_alignment_with_delta_kernels(env):
    """conv kernels that are a single shifted tap: any error in how the shifted operands
    are addressed (row shift, zero padding at both ends) shows up at once."""
    sf, hz, ctx = env
    n_rows, cap = 5, 8
    rows = _cnn_rows(cap, 71)
    for t1, t2 in ((2, 2), (0, 2), (4, 2), (2, 0), (2, 4), (1, 3)):
        m = flowgen.gen_cnn(72, 128, 8, 64, 128, 5, 16)
        mix1 = m["w1"][:, 2, :].copy(); mix2 = m["w2"][:, 2, :].copy()
        m["w1"][:] = 0; m["w1"][:, t1, :] = mix1
        m["w2"][:] = 0; m["w2"][:, t2, :] = mix2
        ref, _ = oracle.cnn(m, rows[:n_rows], True)
        h = sf.sf_cnn_create(ctx, sf.SF_BF16, m)
        logits, _ = _run_slow(sf, hz, ctx, h, hz.dev(rows).to(torch.bfloat16), n_rows, cap, 16)
        assert np.max(np.abs(logits[:n_rows] - ref)) <= TOL_BF16, (t1, t2)
        sf.sf_slow_destroy(h)


# 6,001 rows: about 40 flows (20 pairs, some odd counts) per persistent block, so every ring and barrier phase wraps several times
@pytest.mark.parametrize("n_rows,cap,n_cls", [(0, 4, 16), (1, 1, 16), (2, 2, 16), (3, 4, 16), (300, 333, 16), (1000, 1000, 7), (6001, 6100, 16)])
def test_cnn_within_tolerance(env, n_rows, cap, n_cls):
    sf, hz, ctx = env
    m = flowgen.gen_cnn(73, 128, 8, 64, 128, 5, n_cls)
    rows = _cnn_rows(cap, 74)
    ref, ref_label = oracle.cnn(m, rows[:n_rows], True, threads=8)
    h = sf.sf_cnn_create(ctx, sf.SF_BF16, m)
    rt = hz.dev(rows).to(torch.bfloat16)
    logits, label = _run_slow(sf, hz, ctx, h, rt, n_rows, cap, n_cls)
    assert np.all(np.isnan(logits[n_rows:])) and np.all(label[n_rows:] == 255)      # rows past the count untouched
    if n_rows:
        assert np.max(np.abs(logits[:n_rows] - ref)) <= TOL_BF16
        _check_labels(ref, ref_label, label[:n_rows], TOL_BF16)
    logits2, label2 = _run_slow(sf, hz, ctx, h, rt, n_rows, cap, n_cls)      # run-to-run identical bits
    assert np.array_equal(logits[:n_rows], logits2[:n_rows]) and np.array_equal(label[:n_rows], label2[:n_rows])
    sf.sf_slow_destroy(h)


def test_route_entropy_within_tolerance(env):
    """Entropy score (Sec. 3.2): fp32 logf on the device against the double-precision oracle."""
    sf, hz, ctx = env
    n, C = 20011, 8
    rng = np.random.default_rng(23)
    prob = rng.dirichlet([0.5] * C, size=n).astype(np.float32)
    prob[3] = 0; prob[3, 1] = 1.0
    tau = rng.uniform(0.6, 1.4, C).astype(np.float32)
    ref = oracle.route_entropy(prob, tau)
    cfg = sf.make_route_cfg(sf.SF_ENTROPY_GT, hz.dev(tau), sf.SF_MLP16, sf.SF_BF16, 64, n)
    ids = torch.zeros(n, dtype=torch.uint32, device="cuda"); n_esc = torch.zeros(1, dtype=torch.uint32, device="cuda")
    dec = torch.empty(n, dtype=torch.uint8, device="cuda"); lab = torch.empty(n, dtype=torch.uint8, device="cuda")
    sc = torch.empty(n, dtype=torch.float32, device="cuda")
    sf.sf_route(ctx, cfg, hz.dev(prob), n, C, None, ids, n_esc, None, dec, lab, sc)
    torch.cuda.synchronize()
    sf.sf_ctx_poll(ctx, reset=True)
    score = sc.cpu().numpy(); d = dec.cpu().numpy()
    assert np.max(np.abs(score - ref["score"])) <= 2e-6 and score[3] == 0.0
    assert np.array_equal(lab.cpu().numpy(), ref["label"])
    away = np.abs(ref["score"] - tau[ref["label"]]) > 1e-5
    assert np.array_equal(d[away], ref["decision"][away])
    k = int(n_esc.cpu().numpy()[0])
    assert k == int(d.sum()) and np.array_equal(ids.cpu().numpy()[:k], np.nonzero(d)[0])      # the list is consistent with its own decisions
    assert abs(k - ref["n_esc"]) <= int((~away).sum())


# ------------------------------------------------------- first-packet header bits ---
@pytest.mark.parametrize("n,m", [(5000, 64), (77, 1024), (1, 1), (130, 37)])
def test_header_bits_bit_exact_and_feed_a_first_packet_tree(env, n, m):
    sf, hz, ctx = env
    b, sl = flowgen.gen_first_packet_headers(31 + n, n)
    rng = np.random.default_rng(m)
    sub = np.sort(rng.choice(1024, size=m, replace=False)).astype(np.uint16)
    ref = oracle.header_bits(b, sl, sub)
    out = torch.full((n, m), 9.0, dtype=torch.float32, device="cuda")
    sf.sf_header_bits(ctx, hz.dev(b), hz.dev(sl), n, hz.dev(sub), m, out)
    torch.cuda.synchronize()
    assert np.array_equal(out.cpu().numpy(), ref)
    if m == 64:        # the paper's fastest model: one decision tree on first-packet bits
        fo = flowgen.gen_forest(55, "rf", 1, 8, 64, 4, ref)
        h = hz.make_forest(ctx, fo)
        p = torch.empty((n, 4), dtype=torch.float32, device="cuda")
        sf.sf_fast_infer(ctx, h, out, n, p)
        assert np.array_equal(bits(p.cpu().numpy()), bits(oracle.forest_infer(fo, ref)))
        sf.sf_forest_destroy(h)


# ------------------------------------------------------- threshold calibration on the device ---
@pytest.mark.parametrize("n", [1, 255, 4096, 4097, 300007])
def test_algorithm_1_on_device_scores(env, n):
    sf, hz, ctx = env
    rng = np.random.default_rng(n)
    u = rng.random(n).astype(np.float32)
    u[rng.integers(0, n, n // 3)] = np.float32(0.25)            # many ties
    if n > 10:
        u[:5] = [0.0, 1.0, 3e38, 1e-40, 0.5]                    # zero, a huge value, a subnormal
    q = [0, 1, 50, 75, 76, 99, 100]
    ref = oracle.universal_thresholds(u, q)
    tau = torch.zeros(len(q), dtype=torch.float32, device="cuda")
    sf.sf_universal_thresholds_dev(ctx, hz.dev(u), n, q, 100, tau)
    torch.cuda.synchronize()
    assert np.array_equal(bits(tau.cpu().numpy()), bits(ref))
    assert np.array_equal(bits(sf.sf_universal_thresholds(u, q)), bits(ref))


def test_algorithm_1_on_device_orders_negative_scores(env):
    sf, hz, ctx = env
    u = np.random.default_rng(5).normal(size=20000).astype(np.float32)
    ref = oracle.universal_thresholds(u, [10, 50, 90])
    tau = torch.zeros(3, dtype=torch.float32, device="cuda")
    sf.sf_universal_thresholds_dev(ctx, hz.dev(u), 20000, [10, 50, 90], 100, tau)
    torch.cuda.synchronize()
    assert np.array_equal(bits(tau.cpu().numpy()), bits(ref))


@pytest.mark.parametrize("n,C,Q", [(50000, 8, 100), (3000, 16, 1000), (9, 2, 4), (120000, 3, 20)])
def test_algorithm_2_per_class_thresholds(env, n, C, Q):
    from oracle.calibrate import per_class_thresholds
    sf, hz, ctx = env
    rng = np.random.default_rng(n + C)
    u = rng.random(n).astype(np.float32)
    u[rng.integers(0, n, n // 4)] = np.float32(0.5)
    pred = rng.integers(0, max(C - 1, 1), n).astype(np.uint8)   # the last class is never predicted (when C > 1)
    slope = rng.uniform(0.2, 1.0, C)
    correct = (rng.random(n) > u * slope[pred]).astype(np.uint8)
    for a in (0, 24, 70, 100):
        ref_tau, ref_assigned, _ = per_class_thresholds(u, pred, correct, C, Q, a, 100)
        tau, assigned = sf.sf_per_class_thresholds(ctx, hz.dev(u), hz.dev(pred), hz.dev(correct), n, C, Q, a, 100)
        assert np.array_equal(bits(tau), bits(ref_tau)) and assigned == ref_assigned
        assert assigned == int(np.count_nonzero(u > tau[pred]))


# ------------------------------------------------------- multi-class boosted trees ---
@pytest.mark.parametrize("C,rounds,depth,F,n", [(1, 9, 5, 24, 700), (2, 30, 6, 32, 5000), (3, 11, 4, 24, 1537),
                                                 (5, 40, 6, 48, 4099), (8, 25, 8, 48, 3000), (11, 20, 6, 64, 2500),
                                                 (16, 12, 7, 64, 1111), (7, 3, 9, 16, 513)])
def test_gbdt_multiclass_margins_bit_exact(env, C, rounds, depth, F, n):
    sf, hz, ctx = env
    rng = np.random.default_rng(C * 100 + depth)
    feat = rng.normal(size=(n, F)).astype(np.float32)
    fo = flowgen.gen_forest(7 + C, "gbdt_mc", rounds * C, depth, F, C, feat, sigma=0.3)
    ref, ref_li = oracle.forest_infer(fo, feat, want_leaf_idx=True, threads=4)
    h = hz.make_forest(ctx, fo)
    out = torch.full((n, C), 7.0, dtype=torch.float32, device="cuda")
    li = torch.zeros((n, rounds * C), dtype=torch.uint16, device="cuda")
    sf.sf_fast_infer(ctx, h, hz.dev(feat), n, out, li)
    torch.cuda.synchronize()
    assert sf.sf_ctx_poll(ctx, reset=True).device_error == 0
    assert np.array_equal(li.cpu().numpy(), ref_li)
    assert np.array_equal(bits(out.cpu().numpy()), bits(ref))
    sf.sf_forest_destroy(h)


def test_gbdt_multiclass_round_too_large_for_a_chunk_is_refused(env):
    sf, hz, ctx = env
    feat = np.random.default_rng(1).normal(size=(64, 16)).astype(np.float32)
    fo = flowgen.gen_forest(3, "gbdt_mc", 4, 12, 16, 4, feat)          # 4 trees x 48 KB per round > 64 KB chunk
    h = hz.make_forest(ctx, fo)
    out = torch.zeros((64, 4), dtype=torch.float32, device="cuda")
    with pytest.raises(Exception) as e:
        sf.sf_fast_infer(ctx, h, hz.dev(feat), 64, out)
    assert "unsupported" in str(e.value).lower() or "-6" in str(e.value)
    sf.sf_forest_destroy(h)


def test_route_softmax_least_confidence_within_tolerance(env):
    sf, hz, ctx = env
    n, C = 30011, 11
    rng = np.random.default_rng(29)
    m = (rng.normal(size=(n, C)) * rng.uniform(0.2, 3.0, (n, 1))).astype(np.float32)
    m[5] = 0.25                                                  # all equal: LC = 1 - 1/C, label 0
    tau = rng.uniform(0.3, 0.7, C).astype(np.float32)
    ref = oracle.route_softmax_lc(m, tau)
    cfg = sf.make_route_cfg(sf.SF_SOFTMAX_LC_GT, hz.dev(tau), sf.SF_MLP16, sf.SF_BF16, 64, n)
    ids = torch.zeros(n, dtype=torch.uint32, device="cuda"); n_esc = torch.zeros(1, dtype=torch.uint32, device="cuda")
    dec = torch.empty(n, dtype=torch.uint8, device="cuda"); lab = torch.empty(n, dtype=torch.uint8, device="cuda")
    sc = torch.empty(n, dtype=torch.float32, device="cuda")
    sf.sf_route(ctx, cfg, hz.dev(m), n, C, None, ids, n_esc, None, dec, lab, sc)
    torch.cuda.synchronize()
    sf.sf_ctx_poll(ctx, reset=True)
    score = sc.cpu().numpy(); d = dec.cpu().numpy()
    assert np.max(np.abs(score - ref["score"])) <= 2e-6 and abs(score[5] - (1 - 1 / C)) <= 2e-6
    assert np.array_equal(lab.cpu().numpy(), ref["label"]) and lab.cpu().numpy()[5] == 0
    away = np.abs(ref["score"] - tau[ref["label"]]) > 1e-5
    assert np.array_equal(d[away], ref["decision"][away])
    k = int(n_esc.cpu().numpy()[0])
    assert k == int(d.sum()) and np.array_equal(ids.cpu().numpy()[:k], np.nonzero(d)[0])
    assert abs(k - ref["n_esc"]) <= int((~away).sum())


@pytest.mark.parametrize("kind", ["rf", "gbdt", "gbdt_mc"])
def test_forest_threshold_edge_cases_bit_exact(env, kind):
    """Values equal to thresholds, one float apart from them, signed zeros, infinities and negative values:
    the cases where a comparison that is not the plain fp32 `x <= thr` of the definition would go wrong."""
    sf, hz, ctx = env
    rng = np.random.default_rng(77)
    base = np.concatenate([rng.normal(size=40) * 10.0 ** rng.integers(-3, 9, 40), [0.0, -0.0, 1.0, -1.0, 40.0, 1500.0, 3e38, -3e38,
                                                                                    1e-40, -1e-40, 2.0 ** 32, 16777216.0]]).astype(np.float32)
    up = np.nextafter(base, np.float32(np.inf)); dn = np.nextafter(base, np.float32(-np.inf))
    far_up = (base.view(np.uint32) + np.uint32(63)).view(np.float32)      # same 64-key cell or the next one
    pool_x = np.concatenate([base, up, dn, far_up]).astype(np.float32)
    pool_x = pool_x[np.isfinite(pool_x)]
    pool_t = np.concatenate([pool_x, [np.inf, -np.inf]]).astype(np.float32)
    n, F, C, depth, T = 3000, 8, 4, 7, 24
    feat = pool_x[rng.integers(0, len(pool_x), (n, F))]
    fo = flowgen.gen_forest(5, kind, T, depth, F, C, feat, sigma=0.5)
    fo["thr"] = np.ascontiguousarray(pool_t[rng.integers(0, len(pool_t), fo["thr"].shape)])
    ref, ref_li = oracle.forest_infer(fo, feat, want_leaf_idx=True, threads=4)
    assert len(np.unique(ref_li)) > 20
    h = hz.make_forest(ctx, fo)
    out = torch.zeros(ref.shape, dtype=torch.float32, device="cuda")
    li = torch.zeros((n, T), dtype=torch.uint16, device="cuda")
    sf.sf_fast_infer(ctx, h, hz.dev(feat), n, out, li)
    torch.cuda.synchronize()
    assert sf.sf_ctx_poll(ctx, reset=True).device_error == 0
    assert np.array_equal(li.cpu().numpy(), ref_li)
    assert np.array_equal(bits(out.cpu().numpy()), bits(ref))
    sf.sf_forest_destroy(h)

"""GPU parity of the whole cascade (sf_serve_batch and its host-pointer variant)
against the oracle's staged evaluation."""
import dataclasses

import numpy as np
import pytest

import flowgen
import oracle
from workload import make_workload

torch = pytest.importorskip("torch")
pytestmark = pytest.mark.gpu


@pytest.fixture(scope="module")
def env():
    if not torch.cuda.is_available():
        pytest.skip("no CUDA device")
    from paper_2402_03694_b200 import build, binding as sf, harness as hz
    build.build()
    ctx = sf.sf_ctx_create(0, 0)
    yield sf, hz, ctx
    sf.sf_ctx_destroy(ctx)


def bits(a):
    return np.ascontiguousarray(a, np.float32).view(np.uint32)


def run_and_check(sf, hz, ctx, wl, capacity=None):
    cfg, n = wl["cfg"], wl["n"]
    tol = 2e-2 if cfg.slow_dtype == "bf16" else 1e-4
    ref = oracle.serve_batch(cfg, wl["fast"], wl["wide"], wl["forest"], wl["slow"], wl["tau"], threads=8)
    forest = hz.make_forest(ctx, wl["forest"])
    slow = hz.make_slow(ctx, cfg, wl["slow"])
    fast_d = hz.upload_packets(wl["fast"], with_hdr=False)
    wide_d = hz.upload_packets(wl["wide"])
    cap = n if capacity is None else capacity
    rcfg = hz.route_cfg_for(cfg, hz.dev(wl["tau"]), cap)
    label = torch.full((n,), 255, dtype=torch.uint8, device="cuda")
    stage = torch.zeros(n, dtype=torch.uint8, device="cuda")
    n_esc = torch.zeros(1, dtype=torch.uint32, device="cuda")
    sf.sf_ctx_poll(ctx, reset=True)
    sf.sf_serve_batch(ctx, forest, slow, fast_d["struct"], cfg.N, cfg.F, wide_d["struct"], rcfg, label, stage, n_esc)
    torch.cuda.synchronize()
    c = sf.sf_ctx_poll(ctx, reset=True)
    k = int(n_esc.cpu().numpy()[0])
    assert k == ref["n_esc"] and c.n_flows == n and c.n_escalated == k and c.n_slow_done == k
    p = sf.sf_serve_batch_intermediates(ctx)
    Cf = 1 if cfg.kind == "gbdt" else cfg.C
    feat = hz.ptr_tensor(p["feat"], (n, cfg.F), torch.float32).cpu().numpy()
    fo = hz.ptr_tensor(p["fast_out"], (n, Cf), torch.float32).cpu().numpy()
    ids = hz.ptr_tensor(p["esc_ids"], (k,), torch.uint32).cpu().numpy()
    D = cfg.D
    rows = hz.ptr_tensor(p["rows"], (k, D), torch.bfloat16 if cfg.slow_dtype == "bf16" else torch.float32).float().cpu().numpy()
    logits = hz.ptr_tensor(p["logits"], (k, cfg.n_slow_classes), torch.float32).cpu().numpy()
    assert np.array_equal(bits(feat), bits(ref["feat"]))
    assert np.array_equal(bits(fo.reshape(ref["fast_out"].shape)), bits(ref["fast_out"]))
    assert np.array_equal(ids, ref["esc_ids"])
    assert np.array_equal(bits(rows), bits(ref["rows"]))
    assert np.max(np.abs(logits - ref["logits"])) <= tol
    st = stage.cpu().numpy()
    lab = label.cpu().numpy()
    assert np.array_equal(st, ref["stage"])
    fastm = st == 1
    assert np.array_equal(lab[fastm], ref["label_final"][fastm])
    s = np.sort(ref["logits"], axis=1)
    clear = (s[:, -1] - s[:, -2]) >= 2 * tol
    assert np.array_equal(lab[ref["esc_ids"]][clear], ref["label_slow"][clear])
    assert np.array_equal(lab[ref["esc_ids"]], hz.ptr_tensor(p["label_slow"], (k,), torch.uint8).cpu().numpy())
    # the composite call folds the assignment into the tree kernel: the staged calls must give the same bits
    lab_fast = hz.ptr_tensor(p["label_fast"], (n,), torch.uint8).cpu().numpy()
    feat_s = torch.empty((n, cfg.F), dtype=torch.float32, device="cuda")
    fo_s = torch.empty((n, Cf), dtype=torch.float32, device="cuda")
    ids_s = torch.full((max(cap, 1),), 0xFFFFFFFF, dtype=torch.uint32, device="cuda")
    ne_s = torch.zeros(1, dtype=torch.uint32, device="cuda")
    dec_s = torch.zeros(n, dtype=torch.uint8, device="cuda")
    lab_s = torch.zeros(n, dtype=torch.uint8, device="cuda")
    sf.sf_extract_features(ctx, fast_d["struct"], cfg.N, cfg.F, feat_s)
    sf.sf_fast_infer(ctx, forest, feat_s, n, fo_s)
    sf.sf_route(ctx, rcfg, fo_s, n, Cf if cfg.kind != "gbdt" else 1, None, ids_s, ne_s, None, dec_s, lab_s, None)
    torch.cuda.synchronize()
    sf.sf_ctx_poll(ctx, reset=True)
    assert np.array_equal(bits(fo_s.cpu().numpy().reshape(fo.shape)), bits(fo))
    assert int(ne_s.cpu().numpy()[0]) == k and np.array_equal(ids_s.cpu().numpy()[:k], ids)
    assert np.array_equal(dec_s.cpu().numpy(), (st >= 2).astype(np.uint8)) and np.array_equal(lab_s.cpu().numpy(), lab_fast)
    # host-pointer entry point gives the same answers
    fast_h = hz.pinned_packets(wl["fast"], with_hdr=False)
    wide_h = hz.pinned_packets(wl["wide"])
    rcfg_h = hz.route_cfg_for(cfg, np.ascontiguousarray(wl["tau"]), cap)
    lab_h = np.zeros(n, np.uint8); st_h = np.zeros(n, np.uint8); ne_h = np.zeros(1, np.uint32)
    sf.sf_serve_batch_host(ctx, forest, slow, fast_h["struct"], cfg.N, cfg.F, wide_h["struct"], rcfg_h, lab_h, st_h, ne_h)
    assert int(ne_h[0]) == k and np.array_equal(lab_h, lab) and np.array_equal(st_h, st)
    # pageable host planes take the staged route (host-side compaction into the library's pinned buffer)
    fast_p = hz.pinned_packets(wl["fast"], with_hdr=False, pinned=False)
    wide_p = hz.pinned_packets(wl["wide"], pinned=False)
    lab_p = np.zeros(n, np.uint8); st_p = np.zeros(n, np.uint8); ne_p = np.zeros(1, np.uint32)
    sf.sf_serve_batch_host(ctx, forest, slow, fast_p["struct"], cfg.N, cfg.F, wide_p["struct"], rcfg_h, lab_p, st_p, ne_p)
    assert int(ne_p[0]) == k and np.array_equal(lab_p, lab) and np.array_equal(st_p, st)
    sf.sf_serve_batch_host(ctx, forest, slow, fast_h["struct"], cfg.N, cfg.F, wide_h["struct"], rcfg_h, lab_h, st_h, ne_h)   # and back
    assert int(ne_h[0]) == k and np.array_equal(lab_h, lab) and np.array_equal(st_h, st)
    sf.sf_ctx_poll(ctx, reset=True)
    sf.sf_slow_destroy(slow)
    sf.sf_forest_destroy(forest)
    return ref


def test_c1_full(env):
    sf, hz, ctx = env
    wl = make_workload(flowgen.get_config(1))
    ref = run_and_check(sf, hz, ctx, wl)
    assert 0.2 < ref["n_esc"] / wl["n"] < 0.3


def test_c2_shapes_reduced_flow_count(env):
    """Config 2's model shapes (100 depth-12 trees, 2048-wide bf16 MLP) on 6,000 flows:
    several 512-flow tiles plus a ragged tail, ~1,400 assigned rows (11 GEMM row tiles)."""
    sf, hz, ctx = env
    wl = make_workload(flowgen.get_config(2), n=6000)
    run_and_check(sf, hz, ctx, wl)


def test_c3_shapes_reduced_flow_count(env):
    sf, hz, ctx = env
    wl = make_workload(flowgen.get_config(3), n=9000)
    run_and_check(sf, hz, ctx, wl)


def test_shared_planes_and_ragged_sizes(env):
    """fast_ctx and slow_ctx alias the same wide planes (pitch = P), odd flow count."""
    sf, hz, ctx = env
    cfg = dataclasses.replace(flowgen.get_config(1), n=1237)
    wl = make_workload(cfg, n=1237)
    wl["fast"] = wl["wide"]
    run_and_check(sf, hz, ctx, wl)


def test_c4_shapes_reduced_flow_count(env):
    """Config 4: 64 depth-10 trees over 64 features of 32 packets, 16 classes, fused 1-D CNN."""
    sf, hz, ctx = env
    wl = make_workload(flowgen.get_config(4), n=5000)
    run_and_check(sf, hz, ctx, wl)


@pytest.mark.parametrize("c,n", [(1, 3000), (2, 5000)])
def test_three_tier_cascade(env, c, n):
    """fastest (one decision tree) -> fast (forest) -> slow, per-class thresholds at both tiers."""
    sf, hz, ctx = env
    cfg = dataclasses.replace(flowgen.get_config(c), n=n)
    wl = make_workload(cfg, n=n)
    feat = oracle.extract_features(wl["fast"], cfg.N, cfg.F, threads=8)
    fastest = flowgen.gen_forest(4242, "rf", 1, 7, cfg.F, cfg.C, feat)
    rng = np.random.default_rng(c)
    tau1 = rng.uniform(0.2, 0.7, cfg.C).astype(np.float32)
    tau2 = (wl["tau"] + rng.uniform(-0.05, 0.05, cfg.C)).astype(np.float32)
    ref = oracle.serve_batch3(cfg, wl["fast"], wl["wide"], fastest, wl["forest"], wl["slow"], tau1, tau2, threads=8)
    tol = 2e-2 if cfg.slow_dtype == "bf16" else 1e-4
    h1 = hz.make_forest(ctx, fastest); h2 = hz.make_forest(ctx, wl["forest"]); hs = hz.make_slow(ctx, cfg, wl["slow"])
    fast_d = hz.upload_packets(wl["fast"], with_hdr=False); wide_d = hz.upload_packets(wl["wide"])
    cfg1 = sf.make_route_cfg(sf.SF_LC_GT, hz.dev(tau1), sf.SF_MLP16, sf.SF_BF16, cfg.P, n)
    cfg2 = hz.route_cfg_for(cfg, hz.dev(tau2), n)
    label = torch.full((n,), 255, dtype=torch.uint8, device="cuda")
    stage = torch.zeros(n, dtype=torch.uint8, device="cuda")
    cnt = torch.zeros(2, dtype=torch.uint32, device="cuda")
    sf.sf_ctx_poll(ctx, reset=True)
    sf.sf_serve_batch3(ctx, h1, h2, hs, fast_d["struct"], cfg.N, cfg.F, wide_d["struct"], cfg1, cfg2, label, stage, cnt)
    torch.cuda.synchronize()
    c_ = sf.sf_ctx_poll(ctx, reset=True)
    k1, k2 = [int(x) for x in cnt.cpu().numpy()]
    assert (k1, k2) == (len(ref["ids1"]), len(ref["ids2"])) and 0 < k2 < k1 < n
    assert c_.device_error == 0 and c_.n_flows == n + k1 and c_.n_escalated == k1 + k2 and c_.n_slow_done == k2
    st = stage.cpu().numpy(); lab = label.cpu().numpy()
    assert np.array_equal(st, ref["stage"])
    assert np.array_equal(lab[st < 3], ref["label_final"][st < 3])
    p = sf.sf_serve_batch_intermediates(ctx)
    assert np.array_equal(hz.ptr_tensor(p["esc_ids"], (k2,), torch.uint32).cpu().numpy(), ref["ids2"])
    logits = hz.ptr_tensor(p["logits"], (k2, cfg.n_slow_classes), torch.float32).cpu().numpy()
    assert np.max(np.abs(logits - ref["logits"])) <= tol
    s = np.sort(ref["logits"], axis=1)
    clear = (s[:, -1] - s[:, -2]) >= 2 * tol
    assert np.array_equal(lab[ref["ids2"]][clear], ref["label_slow"][clear])
    # with a cfg_fastest that lets nothing through the fastest model, every flow is stage 1
    never = sf.make_route_cfg(sf.SF_LC_GT, hz.dev(np.full(cfg.C, 2.0, np.float32)), sf.SF_MLP16, sf.SF_BF16, cfg.P, n)
    sf.sf_serve_batch3(ctx, h1, h2, hs, fast_d["struct"], cfg.N, cfg.F, wide_d["struct"], never, cfg2, label, stage, cnt)
    torch.cuda.synchronize()
    assert cnt.cpu().numpy().tolist() == [0, 0] and bool((stage == 1).all())
    sf.sf_ctx_poll(ctx, reset=True)
    sf.sf_slow_destroy(hs); sf.sf_forest_destroy(h2); sf.sf_forest_destroy(h1)


def test_empty_batch_and_nothing_assigned(env):
    sf, hz, ctx = env
    cfg = dataclasses.replace(flowgen.get_config(1), n=700)
    wl = make_workload(cfg, n=700)
    forest = hz.make_forest(ctx, wl["forest"]); slow = hz.make_slow(ctx, cfg, wl["slow"])
    fast_d = hz.upload_packets(wl["fast"], with_hdr=False); wide_d = hz.upload_packets(wl["wide"])
    label = torch.full((700,), 255, dtype=torch.uint8, device="cuda"); stage = torch.zeros(700, dtype=torch.uint8, device="cuda")
    n_esc = torch.full((1,), 7, dtype=torch.uint32, device="cuda")
    # thresholds nobody exceeds: the slow model sees zero rows and every flow keeps its fast answer
    never = hz.route_cfg_for(cfg, hz.dev(np.full(cfg.C, 2.0, np.float32)), 700)
    sf.sf_ctx_poll(ctx, reset=True)
    sf.sf_serve_batch(ctx, forest, slow, fast_d["struct"], cfg.N, cfg.F, wide_d["struct"], never, label, stage, n_esc)
    torch.cuda.synchronize()
    ref = oracle.route_lc(oracle.forest_infer(wl["forest"], oracle.extract_features(wl["fast"], cfg.N, cfg.F)), 2.0)
    assert int(n_esc.cpu().numpy()[0]) == 0 and bool((stage == 1).all()) and np.array_equal(label.cpu().numpy(), ref["label"])
    c = sf.sf_ctx_poll(ctx, reset=True)
    assert c.device_error == 0 and c.n_slow_done == 0 and c.n_fast_done == 700
    # an empty batch is accepted and touches nothing
    fast0 = sf.make_packets(fast_d["size"], fast_d["iat_us"], fast_d["dir_bits"], None, None, n_flows=0)
    wide0 = sf.make_packets(wide_d["size"], wide_d["iat_us"], wide_d["dir_bits"], wide_d["hdr"], None, n_flows=0)
    zero_cap = hz.route_cfg_for(cfg, hz.dev(wl["tau"]), 0)
    sf.sf_serve_batch(ctx, forest, slow, fast0, cfg.N, cfg.F, wide0, zero_cap, label, stage, n_esc)
    torch.cuda.synchronize()
    assert int(n_esc.cpu().numpy()[0]) == 0 and sf.sf_ctx_poll(ctx, reset=True).device_error == 0
    sf.sf_slow_destroy(slow); sf.sf_forest_destroy(forest)


def test_three_tier_with_boosted_fast_model(env):
    """fastest (one decision tree, least confidence) -> fast (multi-class boosted trees, least confidence of the
    softmax of their margins) -> slow.  The softmax is fp32 on the device, so flows whose tier-2 score lies within
    1e-5 of its threshold may legitimately differ; everything else must match."""
    sf, hz, ctx = env
    n = 6000
    cfg = dataclasses.replace(flowgen.get_config(2), n=n)
    wl = make_workload(cfg, n=n)
    feat = oracle.extract_features(wl["fast"], cfg.N, cfg.F, threads=8)
    fastest = flowgen.gen_forest(4243, "rf", 1, 7, cfg.F, cfg.C, feat)
    fast = flowgen.gen_forest(4244, "gbdt_mc", 30 * cfg.C, 6, cfg.F, cfg.C, feat, sigma=0.25)
    rng = np.random.default_rng(9)
    tau1 = rng.uniform(0.2, 0.6, cfg.C).astype(np.float32)
    tau2 = rng.uniform(0.55, 0.7, cfg.C).astype(np.float32)
    ref = oracle.serve_batch3(cfg, wl["fast"], wl["wide"], fastest, fast, wl["slow"], tau1, tau2, threads=8)
    band = np.zeros(n, bool)
    band[ref["ids1"]] = np.abs(ref["score2"] - tau2[ref["label2"]]) <= 1e-5
    h1 = hz.make_forest(ctx, fastest); h2 = hz.make_forest(ctx, fast); hs = hz.make_slow(ctx, cfg, wl["slow"])
    fast_d = hz.upload_packets(wl["fast"], with_hdr=False); wide_d = hz.upload_packets(wl["wide"])
    cfg1 = sf.make_route_cfg(sf.SF_LC_GT, hz.dev(tau1), sf.SF_MLP16, sf.SF_BF16, cfg.P, n)
    cfg2 = sf.make_route_cfg(sf.SF_SOFTMAX_LC_GT, hz.dev(tau2), sf.SF_MLP16, sf.SF_BF16, cfg.P, n)
    label = torch.full((n,), 255, dtype=torch.uint8, device="cuda")
    stage = torch.zeros(n, dtype=torch.uint8, device="cuda")
    cnt = torch.zeros(2, dtype=torch.uint32, device="cuda")
    sf.sf_ctx_poll(ctx, reset=True)
    sf.sf_serve_batch3(ctx, h1, h2, hs, fast_d["struct"], cfg.N, cfg.F, wide_d["struct"], cfg1, cfg2, label, stage, cnt)
    torch.cuda.synchronize()
    assert sf.sf_ctx_poll(ctx, reset=True).device_error == 0
    k1, k2 = [int(x) for x in cnt.cpu().numpy()]
    assert k1 == len(ref["ids1"]) and abs(k2 - len(ref["ids2"])) <= int(band.sum()) and 0 < k2 < k1 < n
    assert len(ref["ids2"]) > 200 and band.sum() < 20
    st = stage.cpu().numpy(); lab = label.cpu().numpy()
    ok = ~band
    assert np.array_equal(st[ok], ref["stage"][ok])
    sel = ok & (st < 3)
    assert np.array_equal(lab[sel], ref["label_final"][sel])
    s = np.sort(ref["logits"], axis=1)
    clear = ((s[:, -1] - s[:, -2]) >= 4e-2) & ok[ref["ids2"]]
    assert np.array_equal(lab[ref["ids2"]][clear], ref["label_slow"][clear])
    sf.sf_slow_destroy(hs); sf.sf_forest_destroy(h2); sf.sf_forest_destroy(h1)

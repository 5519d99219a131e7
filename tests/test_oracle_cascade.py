"""The oracle's stages chained as the cascade (Sec. 3.1): all flows through the
fast model, only the uncertain ones through the slow model."""
import numpy as np

import flowgen
import oracle


def test_c1_cascade_escalates_about_a_quarter():
    cfg = flowgen.get_config(1)
    wide = flowgen.gen_packets(cfg.seed_data, cfg.n, cfg.P, cfg.H)
    fast = flowgen.fast_view(wide, cfg.N)
    val = flowgen.fast_view(flowgen.gen_packets(cfg.seed_val, cfg.n_val, cfg.N, 0), cfg.N)
    feat = oracle.extract_features(fast, cfg.N, cfg.F)
    forest = flowgen.gen_forest(cfg.seed_model, cfg.kind, cfg.T, cfg.depth, cfg.F, cfg.C, feat[:65536])
    u_val = oracle.route_lc(oracle.forest_infer(forest, oracle.extract_features(val, cfg.N, cfg.F)), 2.0)["score"]
    tau = oracle.universal_thresholds(u_val, [cfg.q_percent])[0]
    # on the validation set itself the assigned share is 1 - q up to ties (Algorithm 1)
    assert abs((u_val > tau).mean() - (1 - cfg.q_percent / 100)) < 2e-3
    model = flowgen.gen_mlp(cfg.seed_model, cfg.dims)
    out = oracle.serve_batch(cfg, fast, wide, forest, model, tau, threads=4)
    e = out["n_esc"] / cfg.n
    assert 0.20 < e < 0.30
    assert out["n_esc"] == int(out["decision"].sum()) == out["rows"].shape[0] == out["logits"].shape[0]
    assert int((out["stage"] == 2).sum()) == out["n_esc"]
    keep = out["stage"] == 1
    assert np.array_equal(out["label_final"][keep], out["label"][keep])
    assert np.array_equal(out["label_final"][out["esc_ids"]], out["label_slow"])
    assert np.array_equal(out["feat"], feat)


def _three_tier_setup(n=1500):
    import dataclasses
    cfg = dataclasses.replace(flowgen.get_config(1), n=n)
    wide = flowgen.gen_packets(cfg.seed_data, n, cfg.P, cfg.H)
    fast = flowgen.fast_view(wide, cfg.N)
    feat = oracle.extract_features(fast, cfg.N, cfg.F)
    fastest = flowgen.gen_forest(77, "rf", 1, 6, cfg.F, cfg.C, feat)              # one decision tree
    fastf = flowgen.gen_forest(cfg.seed_model, "rf", cfg.T, cfg.depth, cfg.F, cfg.C, feat)
    model = flowgen.gen_mlp(cfg.seed_model, cfg.dims)
    return cfg, wide, fast, fastest, fastf, model


def test_three_tier_reduces_to_known_cases():
    """Special thresholds turn the three-tier cascade into paths that are pinned elsewhere."""
    cfg, wide, fast, fastest, fastf, model = _three_tier_setup()
    C = cfg.C
    never, always = np.full(C, 2.0, np.float32), np.full(C, -1.0, np.float32)
    tau = np.full(C, 0.55, np.float32)
    # the fastest model answers everything: stage 1 everywhere, labels = its argmax
    o = oracle.serve_batch3(cfg, fast, wide, fastest, fastf, model, never, tau)
    assert np.all(o["stage"] == 1) and len(o["ids1"]) == 0 and o["logits"].shape[0] == 0
    assert np.array_equal(o["label_final"], oracle.forest_infer(fastest, o["feat"]).argmax(1).astype(np.uint8))
    # the fastest model answers nothing: identical to the two-tier cascade with the fast model
    o3 = oracle.serve_batch3(cfg, fast, wide, fastest, fastf, model, always, tau)
    o2 = oracle.serve_batch(cfg, fast, wide, fastf, model, tau)
    assert np.array_equal(o3["ids2"], o2["esc_ids"]) and np.array_equal(o3["logits"], o2["logits"])
    assert np.array_equal(o3["label_final"], o2["label_final"]) and np.array_equal(o3["stage"], o2["stage"] + 1)
    # nothing is ever sure: every flow ends at the slow model
    o = oracle.serve_batch3(cfg, fast, wide, fastest, fastf, model, always, always)
    assert np.all(o["stage"] == 3) and np.array_equal(o["label_final"], o["label_slow"])
    # general case: nested id sets, per-class thresholds honoured at both tiers
    t1 = np.array([0.2, 0.6, 0.4, 2.0], np.float32)
    o = oracle.serve_batch3(cfg, fast, wide, fastest, fastf, model, t1, tau)
    assert set(o["ids2"]) <= set(o["ids1"]) and 0 < len(o["ids2"]) < len(o["ids1"]) < cfg.n
    s1 = np.float32(1) - o["prob1"].max(1)
    assert np.array_equal(np.nonzero(s1 > t1[o["label1"]])[0], o["ids1"])
    assert not np.any(o["label1"][o["ids1"]] == 3)                 # class 3's threshold can never be exceeded
    assert np.array_equal(np.bincount(o["stage"], minlength=4)[1:], [cfg.n - len(o["ids1"]), len(o["ids1"]) - len(o["ids2"]), len(o["ids2"])])

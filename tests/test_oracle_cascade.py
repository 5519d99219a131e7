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

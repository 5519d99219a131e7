"""Test-side construction of a config's inputs, models and threshold, with the
ORACLE supplying the feature sample (for split thresholds) and the validation
scores (for Algorithm 1).  Nothing here comes from the CUDA path."""
import numpy as np

import flowgen
import oracle


def make_workload(cfg, n=None, threads=8):
    n = cfg.n if n is None else int(n)
    wide = flowgen.gen_packets(cfg.seed_data, n, cfg.P, cfg.H)
    fast = flowgen.fast_view(wide, cfg.N)
    m = min(n, 65536)
    feat_sample = oracle.extract_features({k: v[:m] for k, v in fast.items()}, cfg.N, cfg.F, threads=threads)
    forest = flowgen.gen_forest(cfg.seed_model, cfg.kind, cfg.T, cfg.depth, cfg.F, cfg.C, feat_sample, cfg.gbdt_sigma)
    if cfg.kind == "rf":
        nv = min(n, cfg.n_val)
        val = flowgen.gen_packets(cfg.seed_val, nv, cfg.N, 0)
        pv = oracle.forest_infer(forest, oracle.extract_features(val, cfg.N, cfg.F, threads=threads), threads=threads)
        u = oracle.route_lc(pv, 2.0)["score"]
        tau = np.full(cfg.C, oracle.universal_thresholds(u, [cfg.q_percent])[0], np.float32)
    else:
        tau = np.array([oracle.TAU_MARGIN], np.float32)
    if cfg.slow == "mlp":
        slow = flowgen.gen_mlp(cfg.seed_model, cfg.dims)
    else:
        slow = flowgen.gen_cnn(cfg.seed_model, *cfg.cnn)
    return {"cfg": cfg, "n": n, "wide": wide, "fast": fast, "forest": forest, "tau": tau, "slow": slow}

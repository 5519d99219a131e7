"""Pins for the oracle's tree-ensemble, scoring, threshold and wide-row stages."""
import ctypes as C
import math
from fractions import Fraction

import numpy as np
import pytest

import flowgen
import oracle


def _forest(kind, T, d, F, C, fid, thr, leaf):
    return {"kind": kind, "T": T, "depth": d, "F": F, "C": C,
            "fid": np.asarray(fid, np.uint16), "thr": np.asarray(thr, np.float32),
            "leaf": np.asarray(leaf, np.float32)}


@pytest.mark.parametrize("d", [1, 2, 3])
def test_brute_force_path_conjunctions(d):
    """For every leaf, evaluate the conjunction of its path predicates directly
    (no traversal loop): exactly one leaf's conjunction holds, and it is the leaf
    the oracle reports."""
    rng = np.random.default_rng(d)
    F, T, n = 5, 7, 400
    n_int, n_leaf = 2 ** d - 1, 2 ** d
    x = rng.integers(0, 4, size=(n, F)).astype(np.float32)      # few values -> equality happens
    fid = rng.integers(0, F, size=(T, n_int))
    thr = rng.integers(0, 4, size=(T, n_int)).astype(np.float32)
    leaf = rng.normal(size=(T, n_leaf)).astype(np.float32)
    _, li = oracle.forest_infer(_forest("gbdt", T, d, F, 1, fid, thr, leaf), x, want_leaf_idx=True)
    for f in range(n):
        for t in range(T):
            holds = []
            for l in range(n_leaf):
                node, ok = 0, True
                bits = [(l >> (d - 1 - k)) & 1 for k in range(d)]      # 0 = left, 1 = right
                for b in bits:
                    left = x[f, fid[t, node]] <= thr[t, node]
                    ok = ok and (left if b == 0 else not left)
                    node = 2 * node + 1 + b
                holds.append(ok)
            assert sum(holds) == 1 and holds.index(True) == li[f, t]


def test_infinite_thresholds_and_equality_goes_left():
    d, F, T = 4, 3, 2
    x = np.random.default_rng(0).normal(size=(50, F)).astype(np.float32)
    fid = np.zeros((T, 15), np.uint16)
    leaf = np.zeros((T, 16), np.float32)
    _, li = oracle.forest_infer(_forest("gbdt", T, d, F, 1, fid, np.full((T, 15), np.inf), leaf), x, True)
    assert np.all(li == 0)
    _, li = oracle.forest_infer(_forest("gbdt", T, d, F, 1, fid, np.full((T, 15), -np.inf), leaf), x, True)
    assert np.all(li == 15)
    xe = np.full((1, F), 2.5, np.float32)
    _, li = oracle.forest_infer(_forest("gbdt", T, d, F, 1, fid, np.full((T, 15), 2.5), leaf), xe, True)
    assert np.all(li == 0)                       # x == thr goes left
    _, li = oracle.forest_infer(_forest("gbdt", T, d, F, 1, fid, np.full((T, 15), np.nextafter(np.float32(2.5), np.float32(0))), leaf), xe, True)
    assert np.all(li == 15)


def test_single_tree_one_hot_is_a_decision_tree():
    d, F, C = 3, 4, 3
    rng = np.random.default_rng(2)
    x = rng.normal(size=(100, F)).astype(np.float32)
    fid = rng.integers(0, F, size=(1, 7))
    thr = rng.normal(size=(1, 7)).astype(np.float32)
    cls = rng.integers(0, C, size=8)
    leaf = np.eye(C, dtype=np.float32)[cls][None]
    p, li = oracle.forest_infer(_forest("rf", 1, d, F, C, fid, thr, leaf), x, True)
    assert np.array_equal(p, np.eye(C, dtype=np.float32)[cls[li[:, 0]]])


def test_equal_leaves_give_sequential_sum_over_T():
    T, d, C = 100, 2, 2
    v = np.float32(0.1)
    leaf = np.full((T, 4, C), v, np.float32)
    p = oracle.forest_infer(_forest("rf", T, d, 1, C, np.zeros((T, 3)), np.zeros((T, 3)), leaf),
                            np.zeros((1, 1), np.float32))
    acc = np.float32(0)
    for _ in range(T):
        acc = np.float32(acc + v)
    assert p[0, 0] == np.float32(acc / np.float32(T))


def test_tree_order_of_summation_is_sequential():
    """Leaf values 2^24, 1, 1, -2^24 in tree order: the sequential fp32 sum is 0
    ((2^24+1) rounds back to 2^24 twice); any pairwise or reversed order gives 2 or 1."""
    vals = [2.0 ** 24, 1.0, 1.0, -(2.0 ** 24)]
    T = 4
    leaf = np.array([[v, v] for v in vals], np.float32)            # depth 1, both leaves equal
    m = oracle.forest_infer(_forest("gbdt", T, 1, 1, 1, np.zeros((T, 1)), np.zeros((T, 1)), leaf),
                            np.zeros((1, 1), np.float32))
    assert m[0] == 0.0
    leafc = np.repeat(leaf[:, :, None], 2, axis=2)
    p = oracle.forest_infer(_forest("rf", T, 1, 1, 2, np.zeros((T, 1)), np.zeros((T, 1)), leafc),
                            np.zeros((1, 1), np.float32))
    assert p[0, 0] == 0.0 and p[0, 1] == 0.0


def test_rf_probabilities_are_a_distribution():
    cfg = flowgen.get_config(1)
    w = flowgen.gen_packets(cfg.seed_data, 1024, cfg.N, H=0)
    feat = oracle.extract_features(w, cfg.N, cfg.F)
    fo = flowgen.gen_forest(cfg.seed_model, "rf", cfg.T, cfg.depth, cfg.F, cfg.C, feat)
    p = oracle.forest_infer(fo, feat)
    assert np.all(p >= 0) and np.all(p <= 1) and np.allclose(p.sum(1), 1, atol=1e-5)
    # float64 mean of the gathered leaves agrees to rounding
    _, li = oracle.forest_infer(fo, feat, True)
    ref = fo["leaf"][np.arange(cfg.T)[None, :], li.astype(np.int64)].astype(np.float64).mean(1)
    assert np.allclose(p, ref, atol=1e-6)


# ---------------------------------------------------------------- routing ----

def test_least_confidence_value():
    # Sec. 3.2: LC = 1 - max P
    assert np.float32(oracle.least_confidence([0.7, 0.2, 0.1, 0.0])) == np.float32(1) - np.float32(0.7)
    assert oracle.least_confidence([0.25, 0.25, 0.25, 0.25]) == 0.75
    assert oracle.least_confidence([0.0, 1.0]) == 0.0


def test_entropy_closed_forms():
    for C in (2, 4, 8):
        assert abs(oracle.entropy([1.0 / C] * C) - math.log(C)) < 1e-6
    assert oracle.entropy([1.0, 0.0, 0.0]) == 0.0


def test_algorithm1_toy_and_portion():
    U = np.array([0.3, 0.1, 0.4, 0.2], np.float32)
    assert oracle.universal_thresholds(U, [50])[0] == np.float32(0.2)       # 1-based U[ceil(.5*4)]
    assert oracle.universal_thresholds(U, [25, 75, 100, 1]).tolist() == [np.float32(0.1), np.float32(0.3), np.float32(0.4), np.float32(0.1)]
    rng = np.random.default_rng(4)
    U = rng.random(10000).astype(np.float32)                            # distinct with prob ~1
    for q in (10, 50, 76, 99):
        tau = oracle.universal_thresholds(U, [q])[0]
        assert int((U > tau).sum()) == 10000 - math.ceil(q * 10000 / 100)


def test_route_count_equals_direct_count_and_ids_sorted():
    rng = np.random.default_rng(6)
    p = rng.dirichlet([0.5] * 5, size=5000).astype(np.float32)
    tau = np.array([0.3, 0.4, 0.5, 0.2, 0.35], np.float32)
    r = oracle.route_lc(p, tau)
    direct = 0
    ids = []
    for f in range(5000):
        a = int(np.argmax(p[f]))                    # numpy argmax: first maximum
        if np.float32(1) - p[f, a] > tau[a]:
            direct += 1
            ids.append(f)
    assert r["n_esc"] == direct and r["esc_ids"].tolist() == ids
    assert np.all(np.diff(r["esc_ids"].astype(np.int64)) > 0)
    assert np.array_equal(r["decision"].nonzero()[0], r["esc_ids"])
    # strictness: a score equal to tau is NOT assigned
    r = oracle.route_lc(np.array([[0.75, 0.25]], np.float32), 0.25)
    assert r["n_esc"] == 0
    r = oracle.route_lc(np.array([[0.5, 0.5]], np.float32), 0.25)
    assert r["n_esc"] == 1 and r["label"][0] == 0      # tie -> lowest index


def test_margin_rule_matches_probability_rule():
    """|p - 0.5| < 0.2 with p = sigmoid(m)  <=>  |m| < ln(0.7/0.3)."""
    assert abs(oracle.TAU_MARGIN - math.log(7 / 3)) < 1e-7
    rng = np.random.default_rng(7)
    m = (rng.normal(size=20000) * 2.24).astype(np.float32)
    r = oracle.route_absmargin(m)
    p = 1.0 / (1.0 + np.exp(-m.astype(np.float64)))
    away = np.abs(np.abs(m.astype(np.float64)) - math.log(7 / 3)) > 1e-5
    assert np.array_equal((np.abs(p - 0.5) < 0.2)[away], r["decision"].astype(bool)[away])
    assert np.array_equal(r["label"], (m > 0).astype(np.uint8))
    assert r["n_esc"] == int(r["decision"].sum()) == len(r["esc_ids"])
    # two-class least confidence: LC = 0.5 - |p - 0.5|
    for mm in (-3.0, -0.2, 0.0, 0.9, 4.0):
        pp = oracle.sigmoid(mm)
        assert abs((1 - max(pp, 1 - pp)) - (0.5 - abs(pp - 0.5))) < 1e-12


def test_sigmoid_closed_forms():
    """The class-1 probability of a boosted binary model: values that are known in closed form, the
    symmetry sigma(m) + sigma(-m) = 1, and monotonicity (a sign error or a dropped minus fails all three)."""
    assert oracle.sigmoid(0.0) == 0.5
    assert abs(oracle.sigmoid(math.log(3.0)) - 0.75) < 1e-15          # 1 / (1 + 1/3)
    assert abs(oracle.sigmoid(-math.log(3.0)) - 0.25) < 1e-15
    assert abs(oracle.sigmoid(math.log(7.0 / 3.0)) - 0.7) < 1e-15     # the 0.2 band of the binary rule
    for m in (-20.0, -3.0, -0.5, 0.25, 2.0, 11.0):
        assert abs(oracle.sigmoid(m) + oracle.sigmoid(-m) - 1.0) < 1e-15
    xs = [-8.0, -1.0, -0.1, 0.0, 0.1, 1.0, 8.0]
    ys = [oracle.sigmoid(x) for x in xs]
    assert all(a < b for a, b in zip(ys, ys[1:])) and 0.0 < ys[0] and ys[-1] < 1.0


def test_bf16_rounding_ties():
    assert oracle.bf16_round(1 + 2 ** -8) == 1.0                 # tie -> even (down)
    assert oracle.bf16_round(1 + 3 * 2 ** -8) == 1 + 2 ** -6     # tie -> even (up)
    assert oracle.bf16_round(1 + 2 ** -8 + 2 ** -20) == 1 + 2 ** -7
    assert oracle.bf16_round(0.0) == 0.0 and oracle.bf16_round(-1.0 - 2 ** -8) == -1.0
    assert oracle.bf16_round(1395.0 / 2048) == float(np.float32(0.6796875))   # 0.68115 -> 8 bits


def test_integer_log():
    assert [oracle.ilog(a) for a in (0, 1, 2, 3, 4, 7, 2 ** 32 - 1)] == [0, 4, 6, 8, 9, 12, 128]
    rng = np.random.default_rng(8)
    for a in [int(x) for x in rng.integers(0, 2 ** 32, size=300)] + list(range(0, 70)):
        v = a + 1
        e = v.bit_length() - 1
        frac = Fraction(v, 2 ** e) - 1                  # in [0,1)
        assert oracle.ilog(a) == 4 * e + math.floor(4 * frac)
        assert 0 <= math.log2(v) - oracle.ilog(a) / 4 < 0.34             # under-estimates log2 by < 1/4 + 0.086
    ls = [oracle.ilog(a) for a in range(0, 5000)]
    assert all(b >= a for a, b in zip(ls, ls[1:]))     # monotone


@pytest.mark.parametrize("layout,H,P", [(0, 13, 64), (1, 5, 128)])
def test_wide_rows_field_by_field(layout, H, P):
    w = flowgen.gen_packets(31, 40, P, H=H)
    ids = np.array([0, 3, 17, 39], np.uint32)
    nv = np.full(40, 255, np.uint8)
    nv[3] = 10
    for bf in (False, True):
        rows = oracle.wide_rows(layout, ids, w, P, bf, n_valid=nv)
        W = 16 if layout == 0 else 8
        rows = rows.reshape(len(ids), P, W)
        for r, f in enumerate(ids):
            for i in range(P):
                if i >= nv[f]:
                    assert np.all(rows[r, i] == 0)
                    continue
                exp = [float(w["size"][f, i]) / 2048.0, oracle.ilog(w["iat_us"][f, i]) / 128.0,
                       float((int(w["dir_bits"][f, i // 32]) >> (i % 32)) & 1)]
                exp += [float(b) / 256.0 for b in w["hdr"][f, i, :(13 if layout == 0 else 5)]]
                if bf:
                    exp = [oracle.bf16_round(v) for v in exp]
                assert rows[r, i].tolist() == [float(np.float32(v)) for v in exp]
    # zero padding beyond the real packet count (streaming: 64 real, 128 wide)
    if layout == 0:
        w64 = flowgen.gen_packets(31, 40, 64, H=H)
        r = oracle.wide_rows(0, ids, w64, 128, True, P_real=64).reshape(len(ids), 128, 16)
        assert np.all(r[:, 64:] == 0)
        assert np.array_equal(r[:, :64].reshape(len(ids), -1), oracle.wide_rows(0, ids, w64, 64, True))


def test_merge():
    lf = np.array([1, 2, 3, 0, 1], np.uint8)
    label, stage = oracle.merge(lf, np.array([1, 4], np.uint32), np.array([7, 9], np.uint8))
    assert label.tolist() == [1, 7, 3, 0, 9] and stage.tolist() == [1, 2, 1, 1, 2]


def test_entropy_rule_matches_direct_evaluation():
    rng = np.random.default_rng(21)
    p = rng.dirichlet([0.5] * 6, size=3000).astype(np.float32)
    p[0] = 0; p[0, 2] = 1.0                                   # a certain prediction: H = 0
    tau = rng.uniform(0.4, 1.2, 6).astype(np.float32)
    r = oracle.route_entropy(p, tau)
    pd = p.astype(np.float64)
    with np.errstate(divide="ignore", invalid="ignore"):
        h = -np.where(pd > 0, pd * np.log(pd), 0.0).sum(1)     # Sec. 3.2
    assert np.allclose(r["score"], h, atol=1e-6) and r["score"][0] == 0.0
    lab = p.argmax(1)
    assert np.array_equal(r["label"], lab)
    away = np.abs(h - tau[lab]) > 1e-5
    assert np.array_equal(r["decision"].astype(bool)[away], (h > tau[lab])[away])
    assert r["n_esc"] == int(r["decision"].sum()) and np.array_equal(r["esc_ids"], np.nonzero(r["decision"])[0])
    # entropy and least confidence order two-class predictions the same way
    q = np.stack([np.linspace(0.5, 0.99, 50), 1 - np.linspace(0.5, 0.99, 50)], 1).astype(np.float32)
    he = oracle.route_entropy(q, 9.0)["score"]; lc = oracle.route_lc(q, 9.0)["score"]
    assert np.all(np.diff(he) < 0) and np.all(np.diff(lc) < 0)


# ---- multi-class boosted trees and the softmax least-confidence rule ----
def test_gbdt_mc_equals_the_scalar_model_on_each_class_subensemble():
    rng = np.random.default_rng(41)
    F, C, rounds, depth, n = 12, 5, 7, 4, 300
    feat = rng.normal(size=(n, F)).astype(np.float32)
    fo = flowgen.gen_forest(42, "gbdt_mc", rounds * C, depth, F, C, feat, sigma=0.3)
    m, li = oracle.forest_infer(fo, feat, want_leaf_idx=True)
    assert m.shape == (n, C)
    for c in range(C):
        sub = {"kind": "gbdt", "T": rounds, "depth": depth, "F": F, "C": 1, "fid": fo["fid"][c::C].copy(),
               "thr": fo["thr"][c::C].copy(), "leaf": fo["leaf"][c::C].copy()}
        mc, lic = oracle.forest_infer(sub, feat, want_leaf_idx=True)
        assert np.array_equal(m[:, c].view(np.uint32), mc.view(np.uint32)) and np.array_equal(li[:, c::C], lic)
    one = dict(fo, C=1, kind="gbdt_mc")
    assert np.array_equal(oracle.forest_infer(one, feat)[:, 0].view(np.uint32),
                          oracle.forest_infer(dict(fo, kind="gbdt", C=1), feat).view(np.uint32))


def test_softmax_least_confidence_closed_forms():
    L = oracle.lib()
    def lc(m):
        a = np.asarray(m, np.float32)
        return L.sfo_softmax_lc(a.ctypes.data_as(C.c_void_p), C.c_uint32(len(a)))
    assert abs(lc([0.3] * 7) - (1 - 1 / 7)) < 1e-15                   # equal margins: uniform
    assert lc([50.0, -50.0, -50.0]) < 1e-40 and lc([50.0, -50.0, -50.0]) >= 0
    assert abs(lc([1.0, 2.0, 3.0]) - lc([-9.0, -8.0, -7.0])) < 1e-15   # shift invariance
    assert abs(lc([0.0, np.log(3.0)]) - 0.25) < 1e-7                   # two classes: 1 - sigmoid(gap) = 1 - 3/4
    m = np.array([[0.2, 1.5, -0.3]], np.float32)
    p = np.exp(m[0].astype(np.float64)); p /= p.sum()
    r = oracle.route_softmax_lc(m, [0.0, 0.9, 0.0])
    assert abs(float(r["score"][0]) - (1 - p.max())) < 1e-7 and r["label"][0] == 1 and r["decision"][0] == 0
    r = oracle.route_softmax_lc(np.array([[1.0, 1.0, 0.0]], np.float32), 0.5)
    assert r["label"][0] == 0 and r["decision"][0] == 1                # tie -> lowest index; LC = 1 - e/(2e+1) > 0.5

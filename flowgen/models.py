"""Seeded random model parameters (stand-ins for trained models).

Tree ensembles are complete binary trees in heap order.  A split's feature id is
uniform over the F features; its threshold is an order statistic, at a uniform
random quantile, of that feature over a sample of feature rows that the CALLER
supplies (this module computes no features).  Random-forest leaves are
Dirichlet(0.5) class-probability vectors; boosted-tree leaves are N(0, sigma)
scalars.  Dense layers are Xavier-uniform with U(-0.1, 0.1) biases.
"""
import numpy as np


def gen_forest(seed, kind, T, depth, F, C, feat_sample, sigma=0.1):
    """Return dict(fid uint16[T][2^d-1], thr float32[T][2^d-1], leaf float32[T][2^d][C] | [T][2^d])."""
    rng = np.random.Generator(np.random.PCG64(np.random.SeedSequence(int(seed))))
    n_int = (1 << depth) - 1
    n_leaf = 1 << depth
    feat_sample = np.asarray(feat_sample, dtype=np.float32)
    m = feat_sample.shape[0]
    assert feat_sample.shape[1] == F and m >= 1
    col_sorted = np.sort(feat_sample, axis=0)            # [m][F], each column ascending
    fid = rng.integers(0, F, size=(T, n_int), dtype=np.int64)
    q = rng.random(size=(T, n_int))
    rank = np.floor(q * (m - 1)).astype(np.int64)
    thr = col_sorted[rank, fid].astype(np.float32)
    if kind == "rf":
        g = rng.standard_gamma(0.5, size=(T, n_leaf, C))
        g = np.maximum(g, 1e-300)
        leaf = (g / g.sum(axis=2, keepdims=True)).astype(np.float32)
    elif kind in ("gbdt", "gbdt_mc"):       # gbdt_mc: tree t belongs to class t mod C (T a multiple of C)
        assert kind == "gbdt" or T % C == 0
        leaf = rng.normal(0.0, sigma, size=(T, n_leaf)).astype(np.float32)
    else:
        raise ValueError(kind)
    return {"kind": kind, "T": T, "depth": depth, "F": F, "C": C,
            "fid": fid.astype(np.uint16), "thr": np.ascontiguousarray(thr),
            "leaf": np.ascontiguousarray(leaf)}


def _xavier(rng, shape, fan_in, fan_out):
    a = np.sqrt(6.0 / (fan_in + fan_out))
    return rng.uniform(-a, a, size=shape).astype(np.float32)


def gen_mlp(seed, dims):
    """Return dict(dims, W=[float32[out][in]...], b=[float32[out]...])."""
    rng = np.random.Generator(np.random.PCG64(np.random.SeedSequence(int(seed) + 50_000)))
    W, b = [], []
    for l in range(len(dims) - 1):
        W.append(_xavier(rng, (dims[l + 1], dims[l]), dims[l], dims[l + 1]))
        b.append(rng.uniform(-0.1, 0.1, size=(dims[l + 1],)).astype(np.float32))
    return {"dims": tuple(int(d) for d in dims), "W": W, "b": b}


def gen_cnn(seed, L, Cin, C1, C2, k, n_cls):
    """Return dict with w1[C1][k][Cin], w2[C2][k][C1], w3[n_cls][C2] and biases."""
    rng = np.random.Generator(np.random.PCG64(np.random.SeedSequence(int(seed) + 60_000)))
    w1 = _xavier(rng, (C1, k, Cin), k * Cin, k * C1)
    b1 = rng.uniform(-0.1, 0.1, size=(C1,)).astype(np.float32)
    w2 = _xavier(rng, (C2, k, C1), k * C1, k * C2)
    b2 = rng.uniform(-0.1, 0.1, size=(C2,)).astype(np.float32)
    w3 = _xavier(rng, (n_cls, C2), C2, n_cls)
    b3 = rng.uniform(-0.1, 0.1, size=(n_cls,)).astype(np.float32)
    return {"L": L, "Cin": Cin, "C1": C1, "C2": C2, "k": k, "n_cls": n_cls,
            "w1": w1, "b1": b1, "w2": w2, "b2": b2, "w3": w3, "b3": b3}

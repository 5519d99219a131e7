"""Pins for the oracle's slow models: naive loops, special weights, exact
small-integer cases, padding behaviour and an im2col reformulation."""
import numpy as np
import pytest

import flowgen
import oracle


def _naive_mlp(model, rows, bf16):
    """Triple loop in Python floats (double), written independently."""
    rb = oracle.bf16_round if bf16 else (lambda v: float(np.float32(v)))
    out = []
    for r in rows:
        h = [rb(float(v)) for v in r]
        nl = len(model["W"])
        for l in range(nl):
            W, b = model["W"][l], model["b"][l]
            g = []
            for o in range(W.shape[0]):
                acc = 0.0
                for k in range(W.shape[1]):
                    acc += (rb(float(W[o, k])) if bf16 else float(W[o, k])) * h[k]
                v = float(np.float32(acc + float(b[o])))
                if l + 1 < nl:
                    v = max(v, 0.0)
                    if bf16:
                        v = oracle.bf16_round(v)
                g.append(v)
            h = g
        out.append(h)
    return np.array(out, np.float32)


@pytest.mark.parametrize("bf16", [False, True])
def test_mlp_matches_naive_triple_loop(bf16):
    m = flowgen.gen_mlp(5, (12, 7, 9, 3))
    rows = np.random.default_rng(0).normal(size=(6, 12)).astype(np.float32)
    logits, label = oracle.mlp(m, rows, bf16)
    ref = _naive_mlp(m, rows, bf16)
    assert np.allclose(logits, ref, rtol=0, atol=1e-6)
    assert np.array_equal(label, ref.argmax(1).astype(np.uint8))


def test_mlp_zero_weights_give_bias_and_integers_are_exact():
    dims = (8, 5, 4)
    m = {"dims": dims, "W": [np.zeros((5, 8), np.float32), np.zeros((4, 5), np.float32)],
         "b": [np.arange(5, dtype=np.float32), np.array([0.5, -1, 2, 2], np.float32)]}
    logits, label = oracle.mlp(m, np.ones((3, 8), np.float32), True)
    assert np.all(logits == m["b"][1]) and np.all(label == 2)        # tie 2,3 -> lowest index
    rng = np.random.default_rng(1)
    m = {"dims": dims, "W": [rng.integers(-3, 4, (5, 8)).astype(np.float32), rng.integers(-3, 4, (4, 5)).astype(np.float32)],
         "b": [rng.integers(-2, 3, 5).astype(np.float32), rng.integers(-2, 3, 4).astype(np.float32)]}
    x = rng.integers(-4, 5, (10, 8)).astype(np.float32)
    logits, _ = oracle.mlp(m, x, True)
    h = np.maximum(x.astype(np.int64) @ m["W"][0].astype(np.int64).T + m["b"][0].astype(np.int64), 0)
    ref = h @ m["W"][1].astype(np.int64).T + m["b"][1].astype(np.int64)
    assert np.all(np.abs(h) < 256)                       # exactly representable in bf16
    assert np.array_equal(logits, ref.astype(np.float32))


def test_mlp_transposed_weights_would_fail():
    """A [in][out] reading of W gives different logits: guards the operand order."""
    m = flowgen.gen_mlp(6, (6, 6, 6))
    rows = np.random.default_rng(2).normal(size=(4, 6)).astype(np.float32)
    a, _ = oracle.mlp(m, rows, False)
    ref = np.maximum(rows.astype(np.float64) @ m["W"][0].astype(np.float64).T + m["b"][0], 0) @ m["W"][1].astype(np.float64).T + m["b"][1]
    assert np.allclose(a, ref, atol=1e-5)
    mt = {"dims": m["dims"], "W": [w.T.copy() for w in m["W"]], "b": m["b"]}
    b, _ = oracle.mlp(mt, rows, False)
    assert not np.allclose(a, b, atol=1e-3)


def _cnn(L=16, Cin=3, C1=4, C2=5, k=5, n_cls=3, seed=3):
    return flowgen.gen_cnn(seed, L, Cin, C1, C2, k, n_cls)


def test_cnn_centre_tap_delta_is_channel_mixing():
    m = _cnn()
    L, Cin, C1, C2 = m["L"], m["Cin"], m["C1"], m["C2"]
    rng = np.random.default_rng(4)
    mix1 = rng.normal(size=(C1, Cin)).astype(np.float32)
    mix2 = rng.normal(size=(C2, C1)).astype(np.float32)
    m["w1"] = np.zeros_like(m["w1"]); m["w1"][:, 2, :] = mix1
    m["w2"] = np.zeros_like(m["w2"]); m["w2"][:, 2, :] = mix2
    x = rng.normal(size=(2, L, Cin)).astype(np.float32)
    logits, _ = oracle.cnn(m, x.reshape(2, -1), False)
    h1 = np.maximum(x.astype(np.float64) @ mix1.T + m["b1"], 0).astype(np.float32)
    h2 = np.maximum(h1.astype(np.float64) @ mix2.T + m["b2"], 0).astype(np.float32)
    ref = h2.astype(np.float64).mean(1) @ m["w3"].T + m["b3"]
    assert np.allclose(logits, ref, atol=1e-5)


def test_cnn_zero_padding_edges_and_constant_pool():
    # all-ones input, all-ones first kernel, zero bias: position p sees 3,4,5,...,5,4,3 taps
    L, Cin, C1, C2, k, n_cls = 8, 2, 1, 1, 5, 1
    m = {"L": L, "Cin": Cin, "C1": C1, "C2": C2, "k": k, "n_cls": n_cls,
         "w1": np.ones((C1, k, Cin), np.float32), "b1": np.zeros(C1, np.float32),
         "w2": np.zeros((C2, k, C1), np.float32), "b2": np.zeros(C2, np.float32),
         "w3": np.ones((n_cls, C2), np.float32), "b3": np.zeros(n_cls, np.float32)}
    m["w2"][0, 2, 0] = 1.0                               # identity second conv
    x = np.ones((1, L * Cin), np.float32)
    logits, _ = oracle.cnn(m, x, False)
    taps = [3, 4, 5, 5, 5, 5, 4, 3]
    assert logits[0, 0] == np.float32(sum(t * Cin for t in taps) / L)
    # a constant after the second conv pools to that constant
    m["w1"][:] = 0; m["w2"][:] = 0; m["b2"][:] = 0.375
    logits, _ = oracle.cnn(m, x, True)
    assert logits[0, 0] == np.float32(0.375)


@pytest.mark.parametrize("bf16", [False, True])
def test_cnn_equals_im2col_plus_dense(bf16):
    """Second formulation: explicit im2col patches (zero padded) times the flattened
    kernel, through plain numpy float64 products."""
    m = _cnn(L=12, Cin=3, C1=6, C2=4, k=5, n_cls=3, seed=9)
    rng = np.random.default_rng(10)
    x = rng.normal(size=(3, m["L"], m["Cin"])).astype(np.float32)
    rb = np.vectorize(oracle.bf16_round) if bf16 else (lambda a: a)
    if bf16:
        x = rb(x).astype(np.float32)

    def conv(h, w, b):
        n, L, Ci = h.shape
        Co, k, _ = w.shape
        hp = np.zeros((n, L + k - 1, Ci)); hp[:, 2:2 + L] = h
        patches = np.stack([hp[:, p:p + k].reshape(n, k * Ci) for p in range(L)], axis=1)   # [n][L][k*Ci]
        y = patches @ np.asarray(rb(w), np.float64).reshape(Co, k * Ci).T + b
        y = np.maximum(y.astype(np.float32), 0)
        return np.asarray(rb(y), np.float32)

    h1 = conv(x.astype(np.float64), m["w1"], m["b1"])
    h2 = conv(h1.astype(np.float64), m["w2"], m["b2"])
    ref = h2.astype(np.float64).mean(1) @ np.asarray(rb(m["w3"]), np.float64).T + m["b3"]
    logits, label = oracle.cnn(m, x.reshape(3, -1), bf16)
    assert np.allclose(logits, ref, atol=2e-3 if bf16 else 1e-5)
    if not bf16:
        assert np.array_equal(label, ref.argmax(1))

"""Pins for the oracle's feature stage: hand values, the 128-bit case, invariants,
and an independent evaluation in Python integers with brute-force rounding."""
import os
from fractions import Fraction

import numpy as np
import pytest

import flowgen
import oracle

GOLD = os.path.join(os.path.dirname(__file__), "golden", "features_hand.txt")


def _pk(size, iat, dirs):
    size = np.asarray(size, np.uint16).reshape(1, -1)
    iat = np.asarray(iat, np.uint32).reshape(1, -1)
    P = size.shape[1]
    words = (P + 31) // 32
    db = np.zeros((1, words), np.uint32)
    for i, d in enumerate(dirs):
        if d:
            db[0, i // 32] |= np.uint32(1 << (i % 32))
    return {"size": size, "iat_us": iat, "dir_bits": db}


def nearest_f32(v):
    """Brute-force round-to-nearest-even of a non-negative Python int: bracket it
    between adjacent float32 values and compare exact distances."""
    v = int(v)
    if v == 0:
        return np.float32(0.0)
    approx = np.float32(float(v))          # a nearby float32 (possibly double-rounded)
    cands = {approx, np.nextafter(approx, np.float32(0)), np.nextafter(approx, np.float32(np.inf)),
             np.nextafter(np.nextafter(approx, np.float32(0)), np.float32(0))}
    best = None
    for c in cands:
        ci = int(Fraction(float(c)))       # float32 values above 2^24 are integers
        if Fraction(float(c)) != ci:
            dist = abs(Fraction(float(c)) - v)
        else:
            dist = abs(ci - v)
        even = (np.array([c]).view(np.uint32)[0] & 1) == 0
        key = (dist, 0 if even else 1)
        if best is None or key < best[0]:
            best = (key, c)
    return best[1]


def test_hand_values_all_groups():
    exp = {}
    for line in open(GOLD):
        if line.startswith("g"):
            t = line.split()
            exp[int(t[0][1:])] = [float(x) for x in t[1:]]
    pk = _pk([100, 200, 300, 400], [10, 20, 30, 40], [0, 1, 1, 0])
    feat = oracle.extract_features(pk, 4, 64)[0]
    for g in range(8):
        assert feat[8 * g:8 * g + 8].tolist() == exp[g], g


def test_128_bit_variance_case():
    U = 2 ** 32 - 1
    pk = _pk([1, 1, 1, 1], [0, 0, U, U], [0, 0, 0, 0])
    f = oracle.extract_features(pk, 4, 16)[0]
    # V = 4*2U^2 - (2U)^2 = 4U^2 (needs > 64 bits); var = U^2/4 -> 2^62 in fp32
    assert f[8 + 1] == np.float32(2.0 ** 33)
    assert f[8 + 5] == np.float32(2.0 ** 62)
    assert f[8 + 4] == np.float32(2.0 ** 31)


def test_u128_to_f32_matches_brute_force():
    rng = np.random.default_rng(5)
    vals = [0, 1, (1 << 24) - 1, 1 << 24, (1 << 24) + 1, (1 << 24) + 2, (1 << 24) + 3,
            (1 << 25) + 2, (1 << 25) + 6, (1 << 64) - 1, 1 << 64, (1 << 64) + (1 << 40),
            (3 << 62) + (1 << 39), (1 << 74) + (1 << 50), (1 << 74) + (3 << 50), (1 << 100) - 1]
    for _ in range(300):
        bits = int(rng.integers(1, 110))
        vals.append(int(rng.integers(0, 1 << 62)) << max(0, bits - 62) | int(rng.integers(0, 1 << 20)))
    for v in vals:
        assert np.float32(oracle.u128_to_f32(v)) == nearest_f32(v), v


def _py_features(size, iat, dirs, N, F, m=None):
    """Differently written evaluation: Python ints and Fractions per subset list."""
    m = N if m is None else min(N, m)
    idx = list(range(m))
    subsets = {
        0: idx, 1: idx,
        2: [i for i in idx if dirs[i] == 0], 4: [i for i in idx if dirs[i] == 0],
        3: [i for i in idx if dirs[i] == 1], 5: [i for i in idx if dirs[i] == 1],
        6: [i for i in idx if i >= 1 and dirs[i] != dirs[i - 1]],
    }
    subsets[7] = subsets[6]
    out = []
    for g in range(F // 8):
        q = size if g in (0, 2, 3, 6) else iat
        xs = [int(q[i]) for i in subsets[g]]
        if not xs:
            out += [np.float32(0)] * 8
            continue
        c = len(xs)
        s1 = sum(xs)
        V = c * sum(x * x for x in xs) - s1 * s1
        out += [nearest_f32(c), nearest_f32(s1), nearest_f32(min(xs)), nearest_f32(max(xs)),
                nearest_f32(s1) / nearest_f32(c), nearest_f32(V) / nearest_f32(c * c),
                nearest_f32(xs[0]), nearest_f32(xs[-1])]
    return np.array(out, np.float32)


@pytest.mark.parametrize("N,F", [(8, 24), (16, 48), (32, 64), (8, 32)])
def test_cross_check_python_ints(N, F):
    w = flowgen.gen_packets(77 + N, 300, 32, H=0)
    w["iat_us"][5, :] = 2 ** 32 - 1          # extreme values
    w["iat_us"][6, ::2] = 0
    w["iat_us"][6, 1::2] = 2 ** 32 - 1
    pk = flowgen.fast_view(w, N)
    nv = np.random.default_rng(1).integers(0, N + 3, size=300).astype(np.uint8)
    feat = oracle.extract_features(pk, N, F)
    feat_nv = oracle.extract_features(pk, N, F, n_valid=nv)
    for f in range(300):
        dirs = [(int(pk["dir_bits"][f, 0]) >> i) & 1 for i in range(N)]
        ref = _py_features(pk["size"][f], pk["iat_us"][f], dirs, N, F)
        assert np.array_equal(feat[f].view(np.uint32), ref.view(np.uint32)), f
        ref = _py_features(pk["size"][f], pk["iat_us"][f], dirs, N, F, m=int(nv[f]))
        assert np.array_equal(feat_nv[f].view(np.uint32), ref.view(np.uint32)), f


def test_invariants():
    N, F = 16, 64
    w = flowgen.gen_packets(123, 2000, 16, H=0)
    feat = oracle.extract_features(w, N, F).reshape(2000, 8, 8)
    cnt, s, mn, mx, mean, var = (feat[:, :, k] for k in range(6))
    ok = cnt > 0
    assert np.all(mn[ok] <= mean[ok] * (1 + 1e-6)) and np.all(mean[ok] <= mx[ok] * (1 + 1e-6))
    assert np.all(var >= 0)
    assert np.all((var == 0) == ((mn == mx) | ~ok))
    assert np.all(cnt[:, 2] + cnt[:, 3] == N) and np.all(cnt[:, 0] == N)
    assert np.all(cnt[:, 6] <= N - 1)
    # integer sums of the direction subsets add up to the whole (sizes are small: exact in fp32)
    assert np.all(s[:, 2] + s[:, 3] == s[:, 0])
    assert not np.isnan(feat).any() and not np.isinf(feat).any()


def test_direction_flip_swaps_groups():
    N, F = 16, 48
    w = flowgen.gen_packets(9, 500, 16, H=0)
    a = oracle.extract_features(w, N, F).reshape(500, 6, 8)
    w2 = dict(w)
    w2["dir_bits"] = w["dir_bits"] ^ np.uint32(0xFFFF)
    b = oracle.extract_features(w2, N, F).reshape(500, 6, 8)
    assert np.array_equal(a[:, 2], b[:, 3]) and np.array_equal(a[:, 3], b[:, 2])
    assert np.array_equal(a[:, 4], b[:, 5]) and np.array_equal(a[:, 0], b[:, 0])


def test_permutation_inside_subset_keeps_order_free_slots():
    N, F = 8, 16
    rng = np.random.default_rng(3)
    w = flowgen.gen_packets(10, 200, 8, H=0)
    perm = rng.permutation(8)
    w2 = {"size": w["size"][:, perm].copy(), "iat_us": w["iat_us"][:, perm].copy(),
          "dir_bits": np.zeros_like(w["dir_bits"])}
    w["dir_bits"][:] = 0
    a = oracle.extract_features(w, N, F).reshape(200, 2, 8)
    b = oracle.extract_features(w2, N, F).reshape(200, 2, 8)
    assert np.array_equal(a[:, :, :6], b[:, :, :6])


def test_empty_window_and_short_flows():
    w = flowgen.gen_packets(11, 4, 8, H=0)
    nv = np.array([0, 1, 8, 200], np.uint8)
    f = oracle.extract_features(w, 8, 24, n_valid=nv)
    assert np.all(f[0] == 0)
    assert f[1, 0] == 1 and f[1, 5] == 0 and f[1, 2] == f[1, 3] == f[1, 6] == f[1, 7] == w["size"][1, 0]
    full = oracle.extract_features(w, 8, 24)
    assert np.array_equal(f[2], full[2]) and np.array_equal(f[3], full[3])


def test_pitch_larger_than_window():
    w = flowgen.gen_packets(12, 64, 64, H=0)
    a = oracle.extract_features(w, 8, 24)                       # pitch 64, window 8
    b = oracle.extract_features(flowgen.fast_view(w, 8), 8, 24)  # pitch 8
    assert np.array_equal(a, b)


def test_header_bits_hand_example_and_masks():
    """First-packet header bits (Sec. 4.1): hand-built rows."""
    b = np.zeros((3, 128), np.uint8)
    sl = np.array([[20, 20, 0], [24, 0, 8], [60, 60, 8]], np.uint8)
    b[0, 0] = 0x45                      # version 4, IHL 5: bits 0100 0101
    b[0, 9] = 6                         # protocol TCP: 0000 0110 -> columns 72..79
    b[0, 60 + 13] = 0x12                # TCP flags SYN+ACK at TCP byte 13: 0001 0010
    b[1, 120 + 2] = 0x80                # first bit of UDP byte 2
    b[1, 30] = 0xFF                     # noise beyond the 24-byte IPv4 header: must be masked
    sub = np.array([0, 1, 2, 3, 4, 5, 6, 7, 77, 78, 79, 480 + 13 * 8 + 3, 480 + 13 * 8 + 6, 960 + 16, 240, 20 * 8 - 1, 20 * 8, 1023], np.uint16)
    o = oracle.header_bits(b, sl, sub)
    assert o[0].tolist() == [0, 1, 0, 0, 0, 1, 0, 1,  1, 1, 0,  1, 1,  -1,  -1, 0, -1, -1]
    assert o[1, 13] == 1 and o[1, 14] == -1 and o[1, 11] == -1       # UDP present, byte 30 masked, no TCP section
    assert o[1, 15] == 0 and o[1, 16] == 0                           # bytes 19 and 20 are inside a 24-byte header
    assert not np.any(o[2] == -1)                                    # everything present
    # all 1024 columns: the count of -1 columns follows from the lengths; present bits reproduce the bytes
    bb, ll = flowgen.gen_first_packet_headers(5, 200)
    full = oracle.header_bits(bb, ll, np.arange(1024, dtype=np.uint16))
    assert np.array_equal((full == -1).sum(1), 8 * (128 - ll.astype(np.int64).sum(1)))
    bits = np.unpackbits(bb, axis=1).astype(np.float32)              # numpy unpacks MSB first
    assert np.array_equal(full[full >= 0], bits[full >= 0])

"""Pins for the sequential streaming reference: hand-counted tiny streams and the exact
invariant that a flow's streaming answer equals the batch answer on its own first packets."""
import numpy as np

import flowgen
import oracle
from oracle.stream import simulate_stream


def _tiny_models(F=24, C=3, seed=5):
    w = flowgen.gen_packets(seed, 512, 8, 0)
    feat = oracle.extract_features(w, 8, F)
    forest = flowgen.gen_forest(seed, "rf", 6, 4, F, C, feat)
    slow = flowgen.gen_mlp(seed, (64, 16, 3))            # 4 packets x 16 fields
    return forest, slow


def _batch(keys, seed):
    """keys: list of flow numbers, one per packet, in arrival order."""
    rng = np.random.default_rng(seed)
    m = len(keys)
    k = np.asarray(keys, np.uint32)
    return {"src": k + 10, "dst": k + 20, "sport": (k + 1).astype(np.uint16), "dport": (k + 2).astype(np.uint16),
            "proto": (k % 7).astype(np.uint8), "dir": rng.integers(0, 2, m).astype(np.uint8),
            "size": rng.integers(40, 1500, m).astype(np.uint16), "iat_us": rng.integers(0, 10 ** 6, m).astype(np.uint32),
            "hdr": rng.integers(0, 256, (m, 13)).astype(np.uint8)}


def test_hand_counted_stream_never_assigned():
    forest, slow = _tiny_models()
    # flow 0: 5 + 4 = 9 packets, flow 1: 2 + 1 = 3 packets, flow 2: 3 + 5 = 8; two batches, interleaved
    b1 = _batch([0, 1, 0, 2, 0, 0, 2, 2, 1, 0], 1)
    b2 = _batch([2, 2, 0, 0, 2, 2, 0, 0, 1, 2], 2)
    per, cnt = simulate_stream([b1, b2], 8, 12, 24, forest, np.full(3, 2.0, np.float32), slow, 4)   # tau 2: nothing assigned
    assert cnt == {"new_flows": 3, "fast_fired": 2, "fast_done": 2, "escalated": 0, "slow_fired": 0,
                   "dropped_after_decision": 1}                       # flow 0's ninth packet
    n = {k[0] - 10: v for k, v in per.items()}
    assert (n[0]["n_pkts"], n[0]["stage"]) == (9, 1) and (n[1]["n_pkts"], n[1]["stage"]) == (3, 0)
    assert (n[2]["n_pkts"], n[2]["stage"]) == (8, 1)


def test_hand_counted_stream_always_assigned():
    forest, slow = _tiny_models()
    keys = [0] * 3 + [1] * 5 + [0] * 4 + [1] * 2        # flow 0: 7 packets, flow 1: 7 packets
    per, cnt = simulate_stream([_batch(keys, 3)], 2, 4, 24, forest, np.full(3, -1.0, np.float32), slow, 4)
    # both flows fire fast at 2 packets, are assigned (tau -1), fire slow at 4, then 3 late packets each
    assert cnt == {"new_flows": 2, "fast_fired": 2, "fast_done": 0, "escalated": 2, "slow_fired": 2,
                   "dropped_after_decision": 6}
    assert all(v["stage"] == 3 and v["label_slow"] is not None for v in per.values())


def test_streaming_answer_equals_batch_answer_on_first_packets():
    forest, slow = _tiny_models()
    src = flowgen.StreamSource(11, 300, 1.1)
    batches = [src.batch(b, 1500) for b in range(6)]
    tau = np.full(3, 0.45, np.float32)
    per, cnt = simulate_stream(batches, 8, 12, 24, forest, tau, flowgen.gen_mlp(5, (12 * 16, 16, 3)), 12, threads=2)
    # rebuild every flow's packet list independently and run the batch oracle on it
    flows = {}
    for b in batches:
        for i in range(len(b["size"])):
            k = (int(b["src"][i]), int(b["dst"][i]), int(b["sport"][i]), int(b["dport"][i]), int(b["proto"][i]))
            flows.setdefault(k, []).append((int(b["size"][i]), int(b["iat_us"][i]), int(b["dir"][i])))
    assert cnt["new_flows"] == len(flows) and sum(v["n_pkts"] for v in per.values()) == 6 * 1500
    checked = 0
    for k, pk in flows.items():
        r = per[k]
        assert r["n_pkts"] == len(pk)
        if len(pk) < 8:
            assert r["stage"] == 0
            continue
        size = np.array([[p[0] for p in pk[:8]]], np.uint16)
        iat = np.array([[p[1] for p in pk[:8]]], np.uint32)
        db = np.array([[sum(p[2] << i for i, p in enumerate(pk[:8]))]], np.uint32)
        prob = oracle.forest_infer(forest, oracle.extract_features({"size": size, "iat_us": iat, "dir_bits": db}, 8, 24))
        rt = oracle.route_lc(prob, tau)
        assert r["label_fast"] == int(rt["label"][0]) and (r["stage"] >= 2) == bool(rt["decision"][0])
        assert r["stage"] == (1 if not rt["decision"][0] else (3 if len(pk) >= 12 else 2))
        checked += 1
    assert checked > 50
    late = sum(max(0, len(pk) - (8 if per[k]["stage"] == 1 else 12)) for k, pk in flows.items() if per[k]["stage"] in (1, 3))
    assert cnt["dropped_after_decision"] == late


# ---- table lifecycle: idle timeout and re-arming (Sec. 3.1 / 4.1 discard after a timeout; continuous inference) ----
def test_lifecycle_without_sweeps_equals_the_plain_stream():
    from oracle.lifecycle import simulate_lifecycle
    forest, slow = _tiny_models()
    src = flowgen.StreamSource(12, 200, 1.1)
    batches = [src.batch(b, 800) for b in range(5)]
    tau = np.full(3, 0.45, np.float32)
    slow12 = flowgen.gen_mlp(5, (12 * 16, 16, 3))
    per, cnt = simulate_stream(batches, 8, 12, 24, forest, tau, slow12, 12, threads=2)
    per2, tot, sweeps = simulate_lifecycle([("batch", b, 7) for b in batches], 8, 12, 24, forest, tau, slow12, 12)
    assert tot == cnt and sweeps == [] and per.keys() == per2.keys()
    for k in per:
        a, b = per[k], per2[k]
        assert (a["n_pkts"], a["stage"]) == (b["n_pkts"], b["stage"])
        if a["stage"] >= 1:
            assert a["label_fast"] == b["label_fast"] and a["score"] == b["score"]
        if a["stage"] == 3:
            assert a["label_slow"] == b["label_slow"] and np.array_equal(a["logits"], b["logits"])


def test_lifecycle_hand_counted_timeouts_and_rearm():
    from oracle.lifecycle import simulate_lifecycle
    forest, slow = _tiny_models()
    never = np.full(3, 2.0, np.float32)          # nothing assigned
    always = np.full(3, -1.0, np.float32)        # everything assigned
    # t=10: flow 0 gets 2 packets (answered at 2), flow 1 gets 1 (pending).  t=20: flow 2 gets 2.
    ev = [("batch", _batch([0, 1, 0], 1), 10), ("batch", _batch([2, 2], 2), 20),
          ("sweep", 25, 10, False),              # idle: f0 15, f1 15, f2 5 -> f0 (done) and f1 (pending) go
          ("batch", _batch([0, 2, 0, 0], 3), 30)]      # f0 returns as a NEW flow: answered at 2, third packet late; f2 late
    per, tot, sw = simulate_lifecycle(ev, 2, 4, 24, forest, never, slow, 4)
    assert sw == [{"expired_pending": 1, "expired_assigned": 0, "expired_done": 1, "rearmed": 0, "live": 1}]
    assert tot == {"new_flows": 4, "fast_fired": 3, "fast_done": 3, "escalated": 0, "slow_fired": 0, "dropped_after_decision": 2}
    n = {k[0] - 10: v for k, v in per.items()}
    assert set(n) == {0, 2} and (n[0]["n_pkts"], n[0]["stage"]) == (3, 1) and (n[2]["n_pkts"], n[2]["stage"]) == (3, 1)
    # an assigned flow that never gets its slow context is what the timeout is for
    ev = [("batch", _batch([0, 0, 0], 4), 0), ("sweep", 100, 50, False)]
    per, tot, sw = simulate_lifecycle(ev, 2, 4, 24, forest, always, slow, 4)
    assert sw[0]["expired_assigned"] == 1 and per == {} and tot["escalated"] == 1 and tot["slow_fired"] == 0
    # exactly at the limit the flow stays (strictly greater), and the difference wraps in 32 bits
    ev = [("batch", _batch([0], 5), 0xFFFFFFF0), ("sweep", 0x10, 0x20, False), ("sweep", 0x11, 0x20, False)]
    _, _, sw = simulate_lifecycle(ev, 2, 4, 24, forest, never, slow, 4)
    assert [s["live"] for s in sw] == [1, 0]
    # re-arming: every answered flow starts a new window, so a long-lived flow is inferred once per window
    ev = []
    for w in range(3):
        ev += [("batch", _batch([0, 0, 0, 1], 10 + w), w), ("sweep", w, 100, True)]
    per, tot, sw = simulate_lifecycle(ev, 2, 4, 24, forest, never, slow, 4)
    assert tot["fast_fired"] == 4 and tot["dropped_after_decision"] == 3       # flow 0 three times, flow 1 once (2 packets by window 2)
    assert [s["rearmed"] for s in sw] == [1, 2, 1]


def test_lifecycle_rearmed_window_equals_batch_answer_on_that_windows_packets():
    from oracle.lifecycle import simulate_lifecycle
    forest, slow = _tiny_models()
    tau = np.full(3, 2.0, np.float32)
    b1, b2 = _batch([0] * 8, 21), _batch([0] * 8, 22)
    per, tot, _ = simulate_lifecycle([("batch", b1, 0), ("sweep", 1, 100, True), ("batch", b2, 2)], 8, 12, 24, forest, tau, slow, 4)
    db = np.array([[sum(int(b2["dir"][i] & 1) << i for i in range(8))]], np.uint32)
    feat = oracle.extract_features({"size": b2["size"][None, :], "iat_us": b2["iat_us"][None, :], "dir_bits": db}, 8, 24)
    rt = oracle.route_lc(oracle.forest_infer(forest, feat), tau)
    r = list(per.values())[0]
    assert r["label_fast"] == int(rt["label"][0]) and np.float32(r["score"]) == rt["score"][0] and tot["fast_fired"] == 2

"""Test infrastructure: the streaming path with its table lifecycle, packet by packet.

Sec. 3.1 says that data waiting in the queues without a match is discarded after a
timeout, Sec. 4.1 that unrequested packet features are purged after a time threshold,
and the QoE task (Sec. 5.1) needs continuous inference: a monitored flow is inferred
again and again.  Reading, stated as a dictionary keyed by the 5-tuple:

  * events are either ("batch", packets, now) or ("sweep", now, timeout, rearm);
    every packet of a batch carries the batch's time stamp; last_seen[flow] = time stamp
    of the last batch that held one of its packets.
  * a flow collects fast_pkts packets, the fast model runs (features -> trees ->
    least-confidence rule); an answered flow ignores later packets; an assigned flow keeps
    collecting until slow_pkts packets, then the slow model runs; later packets are ignored.
  * sweep: a flow with now - last_seen > timeout (unsigned 32-bit difference) is discarded
    whatever its stage (its key may come back later as a new flow); with rearm, every
    other flow that has its answer (stage 1 or 3) starts a new window: packet count 0,
    stage 0, the old labels stay readable until the next answer overwrites them.
"""
import numpy as np

from . import extract_features, forest_infer, route_lc, wide_rows, mlp


def _fast(rec, fast_pkts, F, forest, tau):
    size = np.array([rec["size"][:fast_pkts]], np.uint16)
    iat = np.array([rec["iat"][:fast_pkts]], np.uint32)
    dirb = np.zeros((1, 1), np.uint32)
    for p in range(fast_pkts):
        dirb[0, 0] |= np.uint32(rec["dir"][p] << p)
    feat = extract_features({"size": size, "iat_us": iat, "dir_bits": dirb}, fast_pkts, F)
    rt = route_lc(forest_infer(forest, feat), tau)
    return int(rt["label"][0]), float(rt["score"][0]), bool(rt["decision"][0])


def _slow(rec, slow_pkts, slow_model, P_model, bf16):
    words = (slow_pkts + 31) // 32
    dirb = np.zeros((1, words), np.uint32)
    for p in range(slow_pkts):
        dirb[0, p // 32] |= np.uint32(rec["dir"][p] << (p % 32))
    planes = {"size": np.array([rec["size"][:slow_pkts]], np.uint16), "iat_us": np.array([rec["iat"][:slow_pkts]], np.uint32),
              "dir_bits": dirb, "hdr": np.array([np.stack(rec["hdr"][:slow_pkts])], np.uint8)}
    rows = wide_rows(0, np.zeros(1, np.uint32), planes, P_model, bf16, P_real=slow_pkts)
    logits, label = mlp(slow_model, rows, bf16)
    return int(label[0]), logits[0]


def simulate_lifecycle(events, fast_pkts, slow_pkts, F, forest, tau, slow_model, P_model, bf16=True):
    """Returns (per_key dict of the flows alive at the end, totals dict, list of per-sweep dicts)."""
    flows = {}
    tot = {"new_flows": 0, "fast_fired": 0, "fast_done": 0, "escalated": 0, "slow_fired": 0, "dropped_after_decision": 0}
    sweeps = []
    for ev in events:
        if ev[0] == "batch":
            _, b, now = ev
            for i in range(len(b["size"])):
                key = (int(b["src"][i]), int(b["dst"][i]), int(b["sport"][i]), int(b["dport"][i]), int(b["proto"][i]))
                r = flows.get(key)
                if r is None:
                    r = {"size": [], "iat": [], "dir": [], "hdr": [], "n": 0, "stage": 0, "label_fast": 0, "score": 0.0,
                         "label_slow": 0, "logits": None}
                    flows[key] = r
                    tot["new_flows"] += 1
                r["last_seen"] = now
                if r["stage"] in (1, 3):
                    tot["dropped_after_decision"] += 1
                    r["n"] += 1
                    continue
                r["size"].append(int(b["size"][i])); r["iat"].append(int(b["iat_us"][i]))
                r["dir"].append(int(b["dir"][i]) & 1); r["hdr"].append(np.asarray(b["hdr"][i], np.uint8))
                r["n"] += 1
                if r["stage"] == 0 and r["n"] == fast_pkts:
                    r["label_fast"], r["score"], assigned = _fast(r, fast_pkts, F, forest, tau)
                    tot["fast_fired"] += 1
                    r["stage"] = 2 if assigned else 1
                    tot["escalated" if assigned else "fast_done"] += 1
                if r["stage"] == 2 and r["n"] == slow_pkts:
                    r["label_slow"], r["logits"] = _slow(r, slow_pkts, slow_model, P_model, bf16)
                    r["stage"] = 3
                    tot["slow_fired"] += 1
        else:
            _, now, timeout, rearm = ev
            s = {"expired_pending": 0, "expired_assigned": 0, "expired_done": 0, "rearmed": 0, "live": 0}
            for key in list(flows.keys()):
                r = flows[key]
                if ((now - r["last_seen"]) & 0xFFFFFFFF) > timeout:
                    s[{0: "expired_pending", 2: "expired_assigned", 1: "expired_done", 3: "expired_done"}[r["stage"]]] += 1
                    del flows[key]
                elif rearm and r["stage"] in (1, 3):
                    r.update(size=[], iat=[], dir=[], hdr=[], n=0, stage=0)
                    s["rearmed"] += 1
                    s["live"] += 1
                else:
                    s["live"] += 1
            sweeps.append(s)
    per_key = {k: {"n_pkts": r["n"], "stage": r["stage"], "label_fast": r["label_fast"], "score": r["score"],
                   "label_slow": r["label_slow"], "logits": r["logits"]} for k, r in flows.items()}
    return per_key, tot, sweeps

"""Sequential reference for the streaming workload (test infrastructure, like the rest
of this package).

The paper's server joins a flow's later packets with its escalation by flow id (Sec. 3.1:
Queue 2 and Queue 3 are combined "based on flow ID"; Sec. 4.1).  The plain statement of
that behaviour is a packet-by-packet loop over a dictionary keyed by the 5-tuple:

  * a flow collects its first `fast_pkts` packets; with the fast_pkts-th packet the fast
    model runs (features of those packets -> tree ensemble -> least-confidence rule);
  * an answered flow ignores every later packet (counted as arriving after the decision);
  * an assigned flow keeps collecting until `slow_pkts` packets, then the slow model runs
    on the wide row of those packets (zero padded to the model's width); later packets
    are again counted as arriving after the decision.

A flow's decisions depend only on its own first packets, so they are evaluated in bulk
with the batch oracle before the sequential pass (same values as deciding inside the loop).
"""
import numpy as np

from . import extract_features, forest_infer, route_lc, wide_rows, mlp


def simulate_stream(batches, fast_pkts, slow_pkts, F, forest, tau, slow_model, P_model, bf16=True, threads=4):
    """batches: list of dicts with src, dst, sport, dport, proto, dir, size, iat_us, hdr arrays.
    Returns (per_key dict key->record, counters dict)."""
    flows = {}
    order = []
    for b in batches:
        for i in range(len(b["size"])):
            key = (int(b["src"][i]), int(b["dst"][i]), int(b["sport"][i]), int(b["dport"][i]), int(b["proto"][i]))
            rec = flows.get(key)
            if rec is None:
                rec = {"size": [], "iat": [], "dir": [], "hdr": [], "n": 0}
                flows[key] = rec
                order.append(key)
            if rec["n"] < slow_pkts:
                rec["size"].append(int(b["size"][i])); rec["iat"].append(int(b["iat_us"][i]))
                rec["dir"].append(int(b["dir"][i]) & 1); rec["hdr"].append(np.asarray(b["hdr"][i], np.uint8))
            rec["n"] += 1

    # bulk fast decisions for the flows that reached fast_pkts packets
    fired = [k for k in order if flows[k]["n"] >= fast_pkts]
    if fired:
        size = np.array([flows[k]["size"][:fast_pkts] for k in fired], np.uint16)
        iat = np.array([flows[k]["iat"][:fast_pkts] for k in fired], np.uint32)
        dirb = np.zeros((len(fired), 1), np.uint32)
        for r, k in enumerate(fired):
            for p in range(fast_pkts):
                dirb[r, 0] |= np.uint32(flows[k]["dir"][p] << p)
        feat = extract_features({"size": size, "iat_us": iat, "dir_bits": dirb}, fast_pkts, F, threads=threads)
        prob = forest_infer(forest, feat, threads=threads)
        rt = route_lc(prob, tau)
        for r, k in enumerate(fired):
            flows[k].update(label_fast=int(rt["label"][r]), score=float(rt["score"][r]), assigned=bool(rt["decision"][r]))
    # bulk slow decisions for assigned flows that reached slow_pkts packets
    slow_fired = [k for k in fired if flows[k]["assigned"] and flows[k]["n"] >= slow_pkts]
    if slow_fired:
        words = (slow_pkts + 31) // 32
        size = np.array([flows[k]["size"][:slow_pkts] for k in slow_fired], np.uint16)
        iat = np.array([flows[k]["iat"][:slow_pkts] for k in slow_fired], np.uint32)
        hdr = np.array([np.stack(flows[k]["hdr"][:slow_pkts]) for k in slow_fired], np.uint8)
        dirb = np.zeros((len(slow_fired), words), np.uint32)
        for r, k in enumerate(slow_fired):
            for p in range(slow_pkts):
                dirb[r, p // 32] |= np.uint32(flows[k]["dir"][p] << (p % 32))
        planes = {"size": size, "iat_us": iat, "dir_bits": dirb, "hdr": hdr}
        rows = wide_rows(0, np.arange(len(slow_fired), dtype=np.uint32), planes, P_model, bf16, P_real=slow_pkts, threads=threads)
        logits, label_slow = mlp(slow_model, rows, bf16, threads=threads)
        for r, k in enumerate(slow_fired):
            flows[k].update(label_slow=int(label_slow[r]), logits=logits[r])

    # the sequential pass: stage reached and counters, packet by packet
    cnt = {"new_flows": len(order), "fast_fired": 0, "fast_done": 0, "escalated": 0, "slow_fired": 0,
           "dropped_after_decision": 0}
    state = {}
    for b in batches:
        for i in range(len(b["size"])):
            key = (int(b["src"][i]), int(b["dst"][i]), int(b["sport"][i]), int(b["dport"][i]), int(b["proto"][i]))
            s = state.setdefault(key, {"n": 0, "stage": 0})
            if s["stage"] in (1, 3):
                cnt["dropped_after_decision"] += 1
            s["n"] += 1
            if s["stage"] == 0 and s["n"] == fast_pkts:
                cnt["fast_fired"] += 1
                if flows[key]["assigned"]:
                    s["stage"] = 2; cnt["escalated"] += 1
                else:
                    s["stage"] = 1; cnt["fast_done"] += 1
            if s["stage"] == 2 and s["n"] == slow_pkts:
                s["stage"] = 3; cnt["slow_fired"] += 1
    per_key = {}
    for k in order:
        r = flows[k]
        per_key[k] = {"n_pkts": state[k]["n"], "stage": state[k]["stage"], "label_fast": r.get("label_fast"),
                      "score": r.get("score"), "label_slow": r.get("label_slow"), "logits": r.get("logits")}
    return per_key, cnt

"""Seeded interleaved packet stream for the streaming workload.

n_keys distinct flows keyed by a random 5-tuple (uint32 src/dst address, uint16
ports, uint8 protocol).  Each packet picks its flow by a bounded Zipf(s) law over
flow ranks (rank r has weight r^-s) and draws size / inter-arrival / direction /
header bytes from the same distributions as the batch workloads.  Packets come in
batches; a batch is a struct of arrays:
    src, dst uint32[m] · sport, dport uint16[m] · proto, dir uint8[m]
    size uint16[m] · iat_us uint32[m] · hdr uint8[m][13]
"""
import numpy as np


def gen_keys(seed, n_keys):
    rng = np.random.Generator(np.random.PCG64(np.random.SeedSequence(int(seed) + 70_000)))
    return {
        "src": rng.integers(0, 1 << 32, size=n_keys, dtype=np.uint32),
        "dst": rng.integers(0, 1 << 32, size=n_keys, dtype=np.uint32),
        "sport": rng.integers(0, 1 << 16, size=n_keys, dtype=np.uint16),
        "dport": rng.integers(0, 1 << 16, size=n_keys, dtype=np.uint16),
        "proto": rng.integers(0, 256, size=n_keys, dtype=np.uint8),
    }


class StreamSource:
    """Draws batches of packets; batch b depends only on (seed, b)."""

    def __init__(self, seed, n_keys, zipf_s=1.1, H=13):
        self.seed = int(seed)
        self.n_keys = int(n_keys)
        self.H = H
        self.keys = gen_keys(seed, n_keys)
        w = np.arange(1, self.n_keys + 1, dtype=np.float64) ** (-float(zipf_s))
        self.cdf = np.cumsum(w)
        self.cdf /= self.cdf[-1]

    def batch(self, b, m):
        ss = np.random.SeedSequence(entropy=self.seed, spawn_key=(1_000_000 + int(b),))
        r = [np.random.Generator(np.random.PCG64(k)) for k in ss.spawn(7)]
        u = r[0].random(size=m)
        flow = np.minimum(np.searchsorted(self.cdf, u, side="left"), self.n_keys - 1)
        small = r[1].integers(40, 101, size=m, dtype=np.uint16)
        large = r[2].integers(1200, 1501, size=m, dtype=np.uint16)
        pick = r[3].random(size=m, dtype=np.float32) < np.float32(0.6)
        size = np.where(pick, small, large).astype(np.uint16)
        iat = np.clip(np.rint(r[4].lognormal(8.0, 2.5, size=m)), 0.0, 4294967295.0).astype(np.uint32)
        d = r[5].integers(0, 2, size=m, dtype=np.uint8)
        hdr = r[6].integers(0, 256, size=(m, self.H), dtype=np.uint8)
        k = self.keys
        return {
            "flow": flow.astype(np.int64),            # generator-side rank, not given to the library
            "src": k["src"][flow], "dst": k["dst"][flow],
            "sport": k["sport"][flow], "dport": k["dport"][flow], "proto": k["proto"][flow],
            "dir": d, "size": size, "iat_us": iat, "hdr": hdr,
        }


def gen_stream_batch(seed, n_keys, b, m, zipf_s=1.1):
    return StreamSource(seed, n_keys, zipf_s).batch(b, m)

"""Seeded packet-header planes.

Per packet: a uint16 size from a bimodal mixture (60 % uniform 40..100 bytes,
40 % uniform 1200..1500 bytes, both inclusive), a uint32 inter-arrival time in
microseconds = rint(lognormal(mu=8, sigma=2.5)) clipped to the uint32 range, one
direction bit (Bernoulli 0.5) and H uniform header bytes.

Layout (row pitch = P packets):
    size     uint16[n][P]
    iat_us   uint32[n][P]
    dir_bits uint32[n][ceil(P/32)]   bit (i % 32) of word (i // 32) = direction of packet i
    hdr      uint8 [n][P][H]

Flows are generated in chunks of CHUNK_FLOWS, each from its own child seed, so the
first k flows of a large batch equal a batch of k flows with the same seed.
"""
import os
from concurrent.futures import ThreadPoolExecutor

import numpy as np

CHUNK_FLOWS = 65536


def gen_packets(seed, n, P, H=13, workers=None):
    """Return dict(size, iat_us, dir_bits, hdr) for n flows of P packets each.  Chunks are
    independent, so `workers` threads (default: the host's cores, at most 16) draw them side
    by side; the bytes do not depend on the number of workers."""
    n = int(n)
    words = (P + 31) // 32
    size = np.empty((n, P), dtype=np.uint16)
    iat = np.empty((n, P), dtype=np.uint32)
    dir_bits = np.empty((n, words), dtype=np.uint32)
    hdr = np.empty((n, P, H), dtype=np.uint8)
    n_chunks = (n + CHUNK_FLOWS - 1) // CHUNK_FLOWS

    def one(ci):
        lo = ci * CHUNK_FLOWS
        m = min(CHUNK_FLOWS, n - lo)
        ss = np.random.SeedSequence(entropy=int(seed), spawn_key=(ci,))
        s, a, d, h = _chunk_prefix(ss, m, P, H)
        size[lo:lo + m] = s
        iat[lo:lo + m] = a
        dir_bits[lo:lo + m] = d
        hdr[lo:lo + m] = h

    if workers is None:
        workers = min(16, os.cpu_count() or 1)
    workers = max(1, min(int(workers), n_chunks))
    if workers == 1:
        for ci in range(n_chunks):
            one(ci)
    else:
        with ThreadPoolExecutor(max_workers=workers) as ex:
            list(ex.map(one, range(n_chunks)))
    return {"size": size, "iat_us": iat, "dir_bits": dir_bits, "hdr": hdr}


def _chunk_prefix(ss, m, P, H):
    """Rows [0, m) of a chunk.  Each plane has its own child stream, so a shorter
    chunk is a prefix of a longer one drawn from the same seed."""
    kids = ss.spawn(6)
    r = [np.random.Generator(np.random.PCG64(k)) for k in kids]
    small = r[0].integers(40, 101, size=(m, P), dtype=np.uint16)
    large = r[1].integers(1200, 1501, size=(m, P), dtype=np.uint16)
    pick = r[2].random(size=(m, P), dtype=np.float32) < np.float32(0.6)
    size = np.where(pick, small, large).astype(np.uint16)
    ln = r[3].lognormal(mean=8.0, sigma=2.5, size=(m, P))
    iat = np.clip(np.rint(ln), 0.0, 4294967295.0).astype(np.uint32)
    words = (P + 31) // 32
    dir_bits = r[4].integers(0, 1 << 32, size=(m, words), dtype=np.uint32)
    if P % 32:
        dir_bits[:, -1] &= np.uint32((1 << (P % 32)) - 1)
    hdr = r[5].integers(0, 256, size=(m, P, H), dtype=np.uint8) if H > 0 \
        else np.zeros((m, P, 0), dtype=np.uint8)
    return size, iat, dir_bits, hdr


def fast_view(wide, N):
    """Contiguous planes of the first N packets (pitch N) cut from wide planes."""
    words = (N + 31) // 32
    d = np.ascontiguousarray(wide["dir_bits"][:, :words]).copy()
    if N % 32:
        d[:, -1] &= np.uint32((1 << (N % 32)) - 1)
    return {
        "size": np.ascontiguousarray(wide["size"][:, :N]),
        "iat_us": np.ascontiguousarray(wide["iat_us"][:, :N]),
        "dir_bits": d,
        "hdr": np.ascontiguousarray(wide["hdr"][:, :N]),
    }


def gen_first_packet_headers(seed, n):
    """Synthetic first-packet header bytes: [n][128] = IPv4 (60) | TCP (60) | UDP (8), and the number
    of bytes present in each section: IPv4 20..60 in steps of 4; 70 % TCP (20..60 in steps of 4, no UDP),
    30 % UDP (8 bytes, no TCP).  Bytes beyond a section's length are filled with noise on purpose
    (a reader must mask them by the lengths)."""
    rng = np.random.Generator(np.random.PCG64(np.random.SeedSequence(int(seed) + 80_000)))
    b = rng.integers(0, 256, size=(n, 128), dtype=np.uint8)
    ip_len = (20 + 4 * rng.integers(0, 11, size=n)).astype(np.uint8)
    is_tcp = rng.random(n) < 0.7
    tcp_len = np.where(is_tcp, 20 + 4 * rng.integers(0, 11, size=n), 0).astype(np.uint8)
    udp_len = np.where(is_tcp, 0, 8).astype(np.uint8)
    return b, np.stack([ip_len, tcp_len, udp_len], axis=1).astype(np.uint8)

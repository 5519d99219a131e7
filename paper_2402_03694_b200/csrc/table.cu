// S0: device-resident per-flow state for the streaming workload.
//
// The paper's server joins first-packet features, later packets and escalations by flow id
// through message queues (Sec. 3.1, Sec. 4.1).  Here one open-addressing hash table in HBM,
// keyed by the 5-tuple, holds every flow's state, and a batch of interleaved packets is
// ingested by a short chain of kernels on one stream:
//   probe     one thread per packet: 128-bit compare-and-swap on the 16-byte key slot
//             (claims an empty slot or recognises its own key; bounded linear probing)
//   sort      key = arrival index of the flow's first packet in the batch (16 bits, unique per
//             flow); stable LSD radix sort (2 passes of 8 bits, tiles of 1024, one kernel per pass)
//             puts each flow's packets together in ARRIVAL order; rank = position minus start of the run
//   apply1    packets that fall into a flow's first `fast_pkts` positions are written to its
//             fast context; flows that just reached fast_pkts packets are listed
//   fast path S1 reads the listed flows' packets in place (through the slot list), S2 runs as the
//             tree-sliced leaf-index kernel for small batches (flow count read on the device)
//   finish    leaf sums in tree order, least-confidence score and decision, then the table update:
//             answered flows are marked, assigned flows get a slab for their slow context
//   apply2    later packets go to the slab of an assigned flow (or are counted as arriving
//             after the decision); flows that just reached slow_pkts packets are listed
//   slow path wide rows of the listed slabs (zero-padded to the model's width) -> S4 -> labels
//   sweep     (on request) one thread per slot: a flow idle for longer than the timeout is discarded
//             (Sec. 3.1 / 4.1: unmatched data is purged after a timeout): its slot becomes a tombstone
//             that a later insertion may claim, its slab goes back to the free list; optionally every
//             answered flow is re-armed for a new window (continuous inference on long-lived flows)
// Slabs are also returned when the slow model has answered.
// Every loop is bounded; a key that finds no slot within the probe limit is counted as missed
// and SF_ERR_TABLE_FULL is recorded in the context's error word.
#include "common.cuh"
#include <algorithm>
#include <new>
#include <string.h>

namespace {

constexpr uint32_t kMaxBatch = 65536;
constexpr uint32_t kProbeLimit = 64;
constexpr uint32_t kHdr = 13;
constexpr uint32_t kMiss = 0xFFFFFFFFu;

struct TableDev {
    // per slot
    ulonglong2* keys; uint32_t* cnt; uint8_t* stage; uint8_t* label_fast; uint8_t* label_slow; float* score; uint32_t* slab;
    uint16_t* f_size; uint32_t* f_iat; uint32_t* f_dir; uint8_t* f_hdr;
    // per slab
    uint16_t* s_size; uint32_t* s_iat; uint32_t* s_dir; uint8_t* s_hdr;
    uint32_t* slab_next;          // bump allocator for slabs never used before
    uint32_t* slab_free; int* slab_free_n;      // stack of returned slabs
    uint32_t* last_seen;          // per slot: time stamp of the last batch that held a packet of the flow
    uint32_t now;                 // time stamp of the batch being ingested
    uint32_t* first;              // per slot: arrival index of the flow's first packet in the current batch (else ~0)
    uint32_t mask, n_slots, fast_pkts, slow_pkts, slow_slabs;
};

}  // namespace

struct sf_table {
    sf_ctx* ctx;
    TableDev d;
    uint32_t log2_slots;
    // per-batch scratch with fixed addresses
    uint32_t* key_a; uint32_t* key_b; uint32_t* idx_a; uint32_t* idx_b; uint32_t* rank; uint32_t* pos;
    uint32_t* fire1_slot; uint32_t* fire2_slab; uint32_t* fire2_slot;
    uint32_t* run0;                   // [key] position where the run of the flow with that sort key starts in the sorted batch
    uint32_t* counts;                 // [0] n_fire1, [1] n_fire2
    uint32_t* pkt_slot; uint32_t* hist;
    void* all;                        // one allocation behind everything above
    // Pipelined ingest (off by default): the look-up and sort of batch b+1 (caller's stream) overlap the fast / slow model work
    // of batch b (the table's own stream).  What the two halves of consecutive batches would share exists twice and is used in
    // turn: sort keys, indices, run starts, packet slots, digit counts, and the per-slot `first` array.
    struct SortSet { uint32_t* key_a; uint32_t* key_b; uint32_t* idx_a; uint32_t* idx_b; uint32_t* run0; uint32_t* pkt_slot; uint32_t* hist; uint32_t* first; };
    SortSet set[2];
    void* all2;                       // the second set's allocation
    int pipelined;
    uint64_t n_batches;               // batches ingested in pipelined mode (selects the set)
    cudaStream_t model_stream;
    cudaEvent_t ev_sorted[2], ev_done[2];
    bool outstanding;                 // model-phase work may still be running on model_stream
};

namespace {

constexpr uint64_t kTomb = ~0ull;      // both halves all ones: no real key (bits 40..62 of the high half are zero)

__device__ __forceinline__ void cas128(void* p, uint64_t clo, uint64_t chi, uint64_t nlo, uint64_t nhi, uint64_t& olo, uint64_t& ohi) {
    // compare with (clo, chi), swap in the key; returns what was there
    asm volatile(
        "{\n"
        ".reg .b128 c, s, d;\n"
        "mov.b128 c, {%2, %3};\n"
        "mov.b128 s, {%4, %5};\n"
        "atom.global.cas.b128 d, [%6], c, s;\n"
        "mov.b128 {%0, %1}, d;\n"
        "}\n"
        : "=l"(olo), "=l"(ohi) : "l"(clo), "l"(chi), "l"(nlo), "l"(nhi), "l"(p) : "memory");
}

__device__ __forceinline__ uint64_t mix64(uint64_t x) {
    x ^= x >> 30; x *= 0xbf58476d1ce4e5b9ull;
    x ^= x >> 27; x *= 0x94d049bb133111ebull;
    x ^= x >> 31;
    return x;
}
__device__ __forceinline__ void make_key(uint32_t src, uint32_t dst, uint32_t sport, uint32_t dport, uint32_t proto,
                                         uint64_t& lo, uint64_t& hi) {
    lo = (uint64_t)src | ((uint64_t)dst << 32);
    hi = (uint64_t)sport | ((uint64_t)dport << 16) | ((uint64_t)proto << 32) | (1ull << 63);     // never zero
}
__device__ __forceinline__ uint32_t hash_key(uint64_t lo, uint64_t hi, uint32_t mask) {
    return (uint32_t)mix64(lo ^ mix64(hi)) & mask;
}

__global__ void probe_kernel(TableDev t, sf_pkt_batch b, uint32_t* __restrict__ pkt_slot,
                             sf_batch_result* res, sf_dev_state* st)
{
    const uint32_t i = blockIdx.x * blockDim.x + threadIdx.x;
    const bool valid = i < b.n;                      // every lane stays to the end: the counters are added up per warp
    const uint32_t lane = threadIdx.x & 31u;
    uint64_t lo = 0, hi = 0;
    if (valid) make_key(b.src[i], b.dst[i], b.sport[i], b.dport[i], b.proto[i], lo, hi);
    uint32_t slot = t.n_slots;                       // "missed" sorts after every real slot
    bool is_new = false;
    // Walk the whole probe chain: the key may sit behind a tombstone.  If it is absent, claim the
    // first tombstone seen, else the empty slot that ends the chain.  Every thread with this key
    // walks the same chain and slots only ever change from free to taken during a batch, so all
    // of them end at one slot.  A lost race against another key restarts the walk (bounded).
    for (uint32_t attempt = 0; valid && attempt < 16 && slot == t.n_slots; attempt++) {
        uint32_t h = hash_key(lo, hi, t.mask), cand = t.n_slots;
        bool cand_tomb = false;
        for (uint32_t p = 0; p < kProbeLimit; p++) {
            const ulonglong2 cur = __ldcg(&t.keys[h]);       // from L2: another SM may just have claimed it
            if (cur.x == lo && cur.y == hi) { slot = h; break; }
            if (cur.x == kTomb && cur.y == kTomb) { if (cand == t.n_slots) { cand = h; cand_tomb = true; } }
            else if (cur.x == 0 && cur.y == 0) { if (cand == t.n_slots) cand = h; break; }
            h = (h + 1) & t.mask;
        }
        if (slot != t.n_slots) break;
        if (cand == t.n_slots) break;                // no free slot within the probe limit
        uint64_t olo, ohi;
        const uint64_t c = cand_tomb ? kTomb : 0ull;
        cas128(&t.keys[cand], c, c, lo, hi, olo, ohi);
        if (olo == c && ohi == c) { slot = cand; is_new = true; }
        else if (olo == lo && ohi == hi) slot = cand;
    }
    // One atomic per warp and counter, and one atomicMin per warp and flow: a heavy flow puts thousands of packets of a
    // batch on one slot, and same-address atomics are served one after the other.
    const bool missed = valid && slot == t.n_slots;
    const uint32_t m_new = __ballot_sync(0xFFFFFFFFu, is_new), m_miss = __ballot_sync(0xFFFFFFFFu, missed);
    if (lane == 0 && m_new) atomicAdd(&res->n_new_flows, (uint32_t)__popc(m_new));
    if (lane == 0 && m_miss) {
        atomicAdd(&res->n_missed, (uint32_t)__popc(m_miss));
        atomicAdd((unsigned long long*)&st->counters.n_missed, (unsigned long long)__popc(m_miss));
        sf_dev_set_error(st, SF_ERR_TABLE_FULL);
    }
    // lanes hold consecutive arrival indices, so the lowest lane among those with the same slot holds their minimum
    const uint32_t peers = __match_any_sync(0xFFFFFFFFu, (valid && !missed) ? slot : (0xFFFFFFC0u + lane));
    if (valid && !missed && (peers & ((1u << lane) - 1u)) == 0) atomicMin(&t.first[slot], i);
    if (valid) pkt_slot[i] = slot;
}

// Sort key of a packet = arrival index of its flow's first packet in this batch: 16 bits,
// unique per flow; a packet that found no slot is a run of its own.  The block also counts its keys' first radix
// digit (shared-memory counters, then one add per digit into hist0[tile][digit]; the caller zeroed hist0).
constexpr uint32_t kTile = 1024;
constexpr uint32_t kMaxTiles = kMaxBatch / kTile;            // 64
constexpr uint32_t kHistWords = 256 * kMaxTiles;             // one pass: [tile][digit]
__global__ void __launch_bounds__(256)
key_kernel(TableDev t, const uint32_t* __restrict__ pkt_slot, uint32_t n,
           uint32_t* __restrict__ key, uint32_t* __restrict__ idx, uint32_t* __restrict__ hist0)
{
    sf_chain_enter();
    __shared__ uint32_t c[256];
    c[threadIdx.x] = 0;
    __syncthreads();
    const uint32_t i = blockIdx.x * blockDim.x + threadIdx.x;
    if (i < n) {
        const uint32_t slot = pkt_slot[i];
        const uint32_t k = (slot < t.n_slots) ? t.first[slot] : i;
        key[i] = k;
        idx[i] = i;
        atomicAdd(&c[k & 255u], 1u);
    }
    __syncthreads();
    if (c[threadIdx.x]) atomicAdd(&hist0[((blockIdx.x * 256u) / kTile) * 256u + threadIdx.x], c[threadIdx.x]);
}

// Stable LSD radix sort of the 16-bit keys: two passes of 8-bit digits, tiles of 1024 items, one kernel per pass.
// A block turns the pass's per-tile digit counts hist[tile][digit] into the output position of its own tile's first
// item of every digit (thread d: items of smaller digits in all tiles + items of digit d in earlier tiles), then takes
// its tile 256 items at a time in index order; an item's place among the items of its digit = (earlier rounds) +
// (earlier warps of this round) + (lower lanes of its warp with the same digit, by match.any).  While moving the
// items it counts the NEXT pass's digit of every item under the tile the item lands in (16-bit counters in shared
// memory, two per word: a block moves at most 1024 items; then one add per non-zero counter into next_hist, which the
// caller zeroed), so no pass needs a counting kernel of its own.
__global__ void __launch_bounds__(256)
radix8_scatter_kernel(const uint32_t* __restrict__ kin, const uint32_t* __restrict__ iin, uint32_t* __restrict__ kout,
                      uint32_t* __restrict__ iout, uint32_t n, uint32_t shift, const uint32_t* __restrict__ hist, uint32_t nblk,
                      uint32_t* __restrict__ next_hist, uint32_t* __restrict__ run_start_of)
{
    sf_chain_enter();
    __shared__ uint32_t base[256];
    __shared__ uint32_t wc[8][256];
    __shared__ uint32_t wsum[8];
    __shared__ uint32_t nh[256 * (kMaxTiles / 2)];       // next pass: [digit][output tile pair]
    const uint32_t tid = threadIdx.x, lane = tid & 31u, warp = tid >> 5;
    if (next_hist) for (uint32_t i = tid; i < 256 * (kMaxTiles / 2); i += 256) nh[i] = 0;
    {
        uint32_t tot = 0, part = 0;
        for (uint32_t t = 0; t < nblk; t++) { const uint32_t v = hist[t * 256u + tid]; tot += v; if (t < blockIdx.x) part += v; }
        uint32_t x = tot;
#pragma unroll
        for (uint32_t o = 1; o < 32; o <<= 1) { const uint32_t y = __shfl_up_sync(0xFFFFFFFFu, x, o); if (lane >= o) x += y; }
        if (lane == 31) wsum[warp] = x;
        __syncthreads();
        uint32_t before = 0;
        for (uint32_t w = 0; w < warp; w++) before += wsum[w];
        base[tid] = before + x - tot + part;
    }
    const uint32_t t0 = blockIdx.x * kTile;
    for (uint32_t r = 0; r < kTile / 256; r++) {
#pragma unroll
        for (uint32_t w = 0; w < 8; w++) wc[w][tid] = 0;
        __syncthreads();
        const uint32_t i = t0 + r * 256 + tid;
        const bool valid = i < n;
        const uint32_t key = valid ? kin[i] : 0u;
        const uint32_t d = valid ? ((key >> shift) & 255u) : (256u + lane);      // idle lanes match nobody
        const uint32_t peers = __match_any_sync(0xFFFFFFFFu, d);
        const uint32_t below = __popc(peers & ((1u << lane) - 1u));
        if (valid && below == 0) wc[warp][d] = __popc(peers);
        __syncthreads();
        uint32_t acc = base[tid];                               // digit `tid`: this round's warps in order
#pragma unroll
        for (uint32_t w = 0; w < 8; w++) { const uint32_t c = wc[w][tid]; wc[w][tid] = acc; acc += c; }
        base[tid] = acc;
        __syncthreads();
        if (valid) {
            const uint32_t p = wc[warp][d] + below;
            const uint32_t id = iin[i];
            kout[p] = key;
            iout[p] = id;
            // last pass: a key is the arrival index of its flow's first packet, so the item whose index equals its key opens
            // the flow's run in the sorted order
            if (run_start_of && id == key) run_start_of[key] = p;
            if (next_hist) atomicAdd(&nh[((key >> (shift + 8)) & 255u) * (kMaxTiles / 2) + (p >> 11)], 1u << (16u * ((p >> 10) & 1u)));
        }
        __syncthreads();
    }
    if (next_hist) {
        for (uint32_t i = tid; i < 256 * (kMaxTiles / 2); i += 256) {
            const uint32_t v = nh[i];
            if (v) {
                const uint32_t dg = i / (kMaxTiles / 2), tp = (i % (kMaxTiles / 2)) * 2u;
                if (v & 0xFFFFu) atomicAdd(&next_hist[tp * 256u + dg], v & 0xFFFFu);
                if (v >> 16) atomicAdd(&next_hist[(tp + 1u) * 256u + dg], v >> 16);
            }
        }
    }
}

__device__ __forceinline__ void store_packet(uint16_t* sz, uint32_t* ia, uint32_t* dirw, uint8_t* hd, uint32_t row,
                                             uint32_t pitch, uint32_t words, uint32_t pos, const sf_pkt_batch& b, uint32_t i)
{
    sz[(size_t)row * pitch + pos] = b.size[i];
    ia[(size_t)row * pitch + pos] = b.iat_us[i];
    if (b.dir[i] & 1u) atomicOr(&dirw[(size_t)row * words + (pos >> 5)], 1u << (pos & 31));
    uint8_t* o = hd + ((size_t)row * pitch + pos) * kHdr;
    const uint8_t* s = b.hdr + (size_t)i * kHdr;
#pragma unroll
    for (int k = 0; k < (int)kHdr; k++) o[k] = s[k];
}

// Returns a slab to the free stack with its direction words cleared (they are filled by atomicOr).
__device__ __forceinline__ void release_slab(const TableDev& t, uint32_t s) {
    const uint32_t words = (t.slow_pkts + 31) / 32;
    for (uint32_t w = 0; w < words; w++) t.s_dir[(size_t)s * words + w] = 0;
    t.slab_free[atomicAdd(t.slab_free_n, 1)] = s;
}

__global__ void apply1_kernel(TableDev t, sf_pkt_batch b, const uint32_t* __restrict__ s_key, const uint32_t* __restrict__ s_idx,
                              const uint32_t* __restrict__ run_start_of,
                              const uint32_t* __restrict__ pkt_slot, uint32_t* __restrict__ rank, uint32_t* __restrict__ pos_out,
                              uint32_t* __restrict__ fire1_slot, uint32_t* __restrict__ counts)
{
    sf_chain_enter();
    const uint32_t j = blockIdx.x * blockDim.x + threadIdx.x;
    if (j >= b.n) return;
    const uint32_t slot = pkt_slot[s_idx[j]];
    if (slot >= t.n_slots) { pos_out[j] = kMiss; rank[j] = 0; return; }
    const uint32_t rk = j - run_start_of[s_key[j]];              // arrival rank among the flow's packets of this batch
    rank[j] = rk;
    const uint32_t pos = t.cnt[slot] + rk;
    pos_out[j] = pos;
    if (pos < t.fast_pkts) {
        store_packet(t.f_size, t.f_iat, t.f_dir, t.f_hdr, slot, t.fast_pkts, 1, pos, b, s_idx[j]);
        if (pos == t.fast_pkts - 1) fire1_slot[atomicAdd(&counts[0], 1u)] = slot;
    }
}

// Finishes the fast model for the flows that fired in this batch and applies the assignment, one kernel instead of
// three (leaf sums, score, application): 16 lanes per flow, lane c < C adds class c's leaf values in tree order
// t = 0..T-1 and divides by T (the random forest's soft vote, same operations and order as the batch kernels), the group
// finds the largest probability (lowest class on ties), and its first lane takes the least-confidence decision
// u = 1 - max > tau[label] and updates the table.
__global__ void __launch_bounds__(256)
fast_finish_kernel(TableDev t, const uint32_t* __restrict__ fire1_slot, const uint32_t* __restrict__ counts,
                   const uint16_t* __restrict__ leaf_idx, const float* __restrict__ leaf, uint32_t T, uint32_t n_leaf, uint32_t C,
                   const float* __restrict__ tau, sf_batch_result* res, sf_dev_state* st)
{
    sf_chain_enter();
    const uint32_t c = threadIdx.x & 15u;
    const uint32_t n_fired = counts[0];
    // a few hundred flows fire per batch, the batch could hold 65,536: a small grid walks over the fired flows
    for (uint32_t k0 = blockIdx.x * (blockDim.x >> 4); k0 < n_fired; k0 += gridDim.x * (blockDim.x >> 4)) {
    const uint32_t k = k0 + (threadIdx.x >> 4);
    const bool live = k < n_fired;
    float prob = -1.0f;                                  // below every probability: lanes past C never win
    if (live && c < C) {
        const uint16_t* idx = leaf_idx + (size_t)k * T;
        float acc = 0.0f;
        uint32_t tt = 0;
        for (; tt + 32 <= T; tt += 32) {                  // 32 loads in flight (the kernel lives on their latency), added in tree order
            float v[32];
#pragma unroll
            for (int q = 0; q < 32; q++) v[q] = __ldg(leaf + ((size_t)(tt + q) * n_leaf + idx[tt + q]) * C + c);
#pragma unroll
            for (int q = 0; q < 32; q++) acc = __fadd_rn(acc, v[q]);
        }
        for (; tt + 8 <= T; tt += 8) {
            float v[8];
#pragma unroll
            for (int q = 0; q < 8; q++) v[q] = __ldg(leaf + ((size_t)(tt + q) * n_leaf + idx[tt + q]) * C + c);
#pragma unroll
            for (int q = 0; q < 8; q++) acc = __fadd_rn(acc, v[q]);
        }
        for (; tt < T; tt++) acc = __fadd_rn(acc, __ldg(leaf + ((size_t)tt * n_leaf + idx[tt]) * C + c));
        prob = __fdiv_rn(acc, __uint2float_rn(T));
    }
    float best = prob; uint32_t arg = c;
#pragma unroll
    for (int o = 8; o >= 1; o >>= 1) {                    // stays inside the 16-lane group
        const float ob = __shfl_xor_sync(0xFFFFFFFFu, best, o);
        const uint32_t oa = __shfl_xor_sync(0xFFFFFFFFu, arg, o);
        if (ob > best || (ob == best && oa < arg)) { best = ob; arg = oa; }
    }
    // the group's first lane decides and books the flow; all 16 lanes then copy its fast context into the slab
    const bool lead = live && c == 0;
    uint32_t slot = 0, slab = kMiss;
    if (lead) {
        const float u = __fsub_rn(1.0f, best);
        bool assigned = u > __ldg(tau + arg);
        slot = fire1_slot[k];
        t.label_fast[slot] = (uint8_t)arg;
        t.score[slot] = u;
        atomicAdd(&res->n_fast_fired, 1u);
        if (assigned) {
            uint32_t sl;
            const int k_free = atomicSub(t.slab_free_n, 1);              // returned slabs first, then never-used ones
            if (k_free >= 1) sl = t.slab_free[k_free - 1];
            else { atomicAdd(t.slab_free_n, 1); sl = atomicAdd(t.slab_next, 1u); if (sl >= t.slow_slabs) atomicSub(t.slab_next, 1u); }
            if (sl < t.slow_slabs) {
                t.slab[slot] = sl;
                slab = sl;
            } else {
                // no slab left: the flow keeps its fast answer and is counted as missed by the slow path
                assigned = false;
                atomicAdd(&res->n_missed, 1u);
                atomicAdd((unsigned long long*)&st->counters.n_missed, 1ull);
                sf_dev_set_error(st, SF_ERR_TABLE_FULL);
            }
        }
        t.stage[slot] = assigned ? 2 : 1;
        if (assigned) { atomicAdd(&res->n_escalated, 1u); atomicAdd((unsigned long long*)&st->counters.n_escalated, 1ull); }
        else          { atomicAdd(&res->n_fast_done, 1u); atomicAdd((unsigned long long*)&st->counters.n_fast_done, 1ull); }
        atomicAdd((unsigned long long*)&st->counters.n_flows, 1ull);
    }
    const uint32_t lead_lane = (threadIdx.x & 31u) & 16u;
    slot = __shfl_sync(0xFFFFFFFFu, slot, lead_lane);
    slab = __shfl_sync(0xFFFFFFFFu, slab, lead_lane);
    if (slab != kMiss) {                                  // one element or byte per lane and step: the loads of a step are all in flight at once
        for (uint32_t p = c; p < t.fast_pkts; p += 16) {
            t.s_size[(size_t)slab * t.slow_pkts + p] = t.f_size[(size_t)slot * t.fast_pkts + p];
            t.s_iat[(size_t)slab * t.slow_pkts + p] = t.f_iat[(size_t)slot * t.fast_pkts + p];
        }
        const uint8_t* src = t.f_hdr + (size_t)slot * t.fast_pkts * kHdr;
        uint8_t* dst = t.s_hdr + (size_t)slab * t.slow_pkts * kHdr;
        for (uint32_t i = c; i < t.fast_pkts * kHdr; i += 16) dst[i] = src[i];
        if (c == 0) atomicOr(&t.s_dir[(size_t)slab * ((t.slow_pkts + 31) / 32)], t.f_dir[slot]);
    }
    }
}

__global__ void apply2_kernel(TableDev t, sf_pkt_batch b, const uint32_t* __restrict__ s_key, const uint32_t* __restrict__ s_idx,
                              const uint32_t* __restrict__ pkt_slot, const uint32_t* __restrict__ rank, const uint32_t* __restrict__ pos_in,
                              uint32_t* __restrict__ fire2_slab, uint32_t* __restrict__ fire2_slot,
                              uint32_t* __restrict__ counts, sf_batch_result* res, sf_dev_state* st)
{
    sf_chain_enter();
    const uint32_t j = blockIdx.x * blockDim.x + threadIdx.x;
    const uint32_t slot = (j < b.n) ? pkt_slot[s_idx[j]] : t.n_slots;
    const bool live = slot < t.n_slots;              // every lane stays to the end: the counter is added up per warp
    bool dropped = false;
    const uint32_t pos = live ? pos_in[j] : 0u;
    if (live && pos >= t.fast_pkts) {
        const uint32_t stg = t.stage[slot];
        if (stg == 2 && pos < t.slow_pkts) {
            const uint32_t s = t.slab[slot];
            store_packet(t.s_size, t.s_iat, t.s_dir, t.s_hdr, s, t.slow_pkts, (t.slow_pkts + 31) / 32, pos, b, s_idx[j]);
            if (pos == t.slow_pkts - 1) {
                const uint32_t k = atomicAdd(&counts[1], 1u);
                fire2_slab[k] = s; fire2_slot[k] = slot;
            }
        } else {
            dropped = true;
        }
    }
    const uint32_t m_drop = __ballot_sync(0xFFFFFFFFu, dropped);
    if ((threadIdx.x & 31u) == 0 && m_drop) {
        atomicAdd(&res->n_dropped_after_decision, (uint32_t)__popc(m_drop));
        atomicAdd((unsigned long long*)&st->counters.n_dropped_after_decision, (unsigned long long)__popc(m_drop));
    }
    if (!live) return;
    // the last packet of the flow's run in this batch advances the flow's packet counter
    if (j + 1 == b.n || s_key[j + 1] != s_key[j]) { t.cnt[slot] += rank[j] + 1; t.first[slot] = 0xFFFFFFFFu; t.last_seen[slot] = t.now; }
}

__global__ void apply_slow_kernel(TableDev t, const uint32_t* __restrict__ fire2_slot, const uint32_t* __restrict__ counts,
                                  const uint8_t* __restrict__ label_slow, sf_batch_result* res, sf_dev_state* st)
{
    sf_chain_enter();
    const uint32_t k = blockIdx.x * blockDim.x + threadIdx.x;
    if (k == 0) atomicAdd((unsigned long long*)&st->counters.n_slow_done, (unsigned long long)counts[1]);
    if (k >= counts[1]) return;
    const uint32_t slot = fire2_slot[k];
    t.label_slow[slot] = label_slow[k];
    t.stage[slot] = 3;
    atomicAdd(&res->n_slow_fired, 1u);
    release_slab(t, t.slab[slot]);                                   // the slow context has been used
}

__global__ void sweep_kernel(TableDev t, uint32_t now, uint32_t timeout, int rearm, sf_sweep_result* res)
{
    const uint32_t slot = blockIdx.x * blockDim.x + threadIdx.x;
    uint32_t what = 0;                     // 1 pending, 2 assigned, 3 done expired; 4 re-armed; 5 live
    if (slot < t.n_slots) {
        const ulonglong2 key = t.keys[slot];
        if (!(key.x == 0 && key.y == 0) && !(key.x == kTomb && key.y == kTomb)) {
            const uint32_t stg = t.stage[slot];
            if (now - t.last_seen[slot] > timeout) {
                what = stg == 0 ? 1 : (stg == 2 ? 2 : 3);
                if (stg == 2) release_slab(t, t.slab[slot]);
                t.cnt[slot] = 0; t.stage[slot] = 0; t.label_fast[slot] = 0; t.label_slow[slot] = 0; t.score[slot] = 0.0f;
                t.f_dir[slot] = 0;
                t.keys[slot] = make_ulonglong2(kTomb, kTomb);
            } else if (rearm && (stg == 1 || stg == 3)) {
                t.cnt[slot] = 0; t.stage[slot] = 0; t.f_dir[slot] = 0;
                what = 4;
            } else what = 5;
        }
    }
    // block-level counts, one atomic per counter and block
    __shared__ uint32_t c[6];
    if (threadIdx.x < 6) c[threadIdx.x] = 0;
    __syncthreads();
    if (what) atomicAdd(&c[what], 1u);
    __syncthreads();
    if (threadIdx.x == 0) {
        if (c[1]) atomicAdd(&res->n_expired_pending, c[1]);
        if (c[2]) atomicAdd(&res->n_expired_assigned, c[2]);
        if (c[3]) atomicAdd(&res->n_expired_done, c[3]);
        if (c[4]) atomicAdd(&res->n_rearmed, c[4]);
        if (c[4] + c[5]) atomicAdd(&res->n_live, c[4] + c[5]);
    }
}

__global__ void lookup_kernel(TableDev t, const sf_key* __restrict__ keys, uint32_t n, sf_flow_result* __restrict__ out)
{
    const uint32_t i = blockIdx.x * blockDim.x + threadIdx.x;
    if (i >= n) return;
    uint64_t lo, hi;
    make_key(keys[i].src, keys[i].dst, keys[i].sport, keys[i].dport, keys[i].proto, lo, hi);
    uint32_t h = hash_key(lo, hi, t.mask);
    sf_flow_result r;
    r.found = 0; r.stage = 0; r.label_fast = 0; r.label_slow = 0; r.n_pkts = 0; r.score = 0.0f;
    for (uint32_t p = 0; p < kProbeLimit; p++) {
        const ulonglong2 cur = t.keys[h];
        if (cur.x == lo && cur.y == hi) {
            r.found = 1; r.stage = t.stage[h]; r.label_fast = t.label_fast[h]; r.label_slow = t.label_slow[h];
            r.n_pkts = t.cnt[h]; r.score = t.score[h];
            break;
        }
        if (cur.x == 0 && cur.y == 0) break;
        h = (h + 1) & t.mask;
    }
    out[i] = r;
}

template <typename T>
T* carve(char*& p, size_t count) {
    T* r = reinterpret_cast<T*>(p);
    p += sf_align256(count * sizeof(T));
    return r;
}

}  // namespace

extern "C" int sf_table_create(sf_ctx* ctx, uint32_t log2_slots, uint32_t fast_pkts, uint32_t slow_pkts,
                               uint32_t slow_slabs, sf_table** out)
{
    if (!ctx || !out) return SF_ERR_ARG;
    if (log2_slots < 4 || log2_slots > 28) return SF_ERR_ARG;
    if (fast_pkts < 1 || fast_pkts > 32 || slow_pkts <= fast_pkts || slow_pkts > 128 || slow_slabs < 1) return SF_ERR_ARG;
    SF_CUDA(cudaSetDevice(ctx->device));
    sf_table* t = new (std::nothrow) sf_table();
    if (!t) return SF_ERR_ALLOC;
    memset(t, 0, sizeof(*t));
    t->ctx = ctx; t->log2_slots = log2_slots;
    const size_t S = (size_t)1 << log2_slots, B = slow_slabs, W = (slow_pkts + 31) / 32;
    size_t total = 0;
    auto need = [&](size_t bytes) { total += sf_align256(bytes); };
    need(S * 16); need(S * 4); need(S); need(S); need(S); need(S * 4); need(S * 4);
    need(S * fast_pkts * 2); need(S * fast_pkts * 4); need(S * 4); need(S * fast_pkts * kHdr);
    need(B * slow_pkts * 2); need(B * slow_pkts * 4); need(B * W * 4); need(B * slow_pkts * kHdr); need(4);
    need(B * 4); need(4); need(S * 4);
    for (int k = 0; k < 10; k++) need((size_t)kMaxBatch * 4);
    need((16 + 2 * kHistWords) * 4); need((size_t)kMaxBatch * 4); need(S * 4);     // counters + digit counts, pkt_slot, first
    cudaError_t e = cudaMalloc(&t->all, total);
    if (e != cudaSuccess) { delete t; sf_set_cuda_error(e, "cudaMalloc(table)"); return SF_ERR_ALLOC; }
    e = cudaMemset(t->all, 0, total);
    if (e != cudaSuccess) { cudaFree(t->all); delete t; return sf_set_cuda_error(e, "cudaMemset(table)"); }
    char* p = reinterpret_cast<char*>(t->all);
    TableDev& d = t->d;
    d.keys = carve<ulonglong2>(p, S); d.cnt = carve<uint32_t>(p, S); d.stage = carve<uint8_t>(p, S);
    d.label_fast = carve<uint8_t>(p, S); d.label_slow = carve<uint8_t>(p, S); d.score = carve<float>(p, S);
    d.slab = carve<uint32_t>(p, S);
    d.f_size = carve<uint16_t>(p, S * fast_pkts); d.f_iat = carve<uint32_t>(p, S * fast_pkts);
    d.f_dir = carve<uint32_t>(p, S); d.f_hdr = carve<uint8_t>(p, S * fast_pkts * kHdr);
    d.s_size = carve<uint16_t>(p, B * slow_pkts); d.s_iat = carve<uint32_t>(p, B * slow_pkts);
    d.s_dir = carve<uint32_t>(p, B * W); d.s_hdr = carve<uint8_t>(p, B * slow_pkts * kHdr);
    d.slab_next = carve<uint32_t>(p, 1);
    d.slab_free = carve<uint32_t>(p, B); d.slab_free_n = carve<int>(p, 1); d.last_seen = carve<uint32_t>(p, S);
    d.now = 0;
    d.mask = (uint32_t)(S - 1); d.n_slots = (uint32_t)S; d.fast_pkts = fast_pkts; d.slow_pkts = slow_pkts; d.slow_slabs = slow_slabs;
    t->key_a = carve<uint32_t>(p, kMaxBatch); t->key_b = carve<uint32_t>(p, kMaxBatch);
    t->idx_a = carve<uint32_t>(p, kMaxBatch); t->idx_b = carve<uint32_t>(p, kMaxBatch);
    t->rank = carve<uint32_t>(p, kMaxBatch); t->pos = carve<uint32_t>(p, kMaxBatch);
    t->fire1_slot = carve<uint32_t>(p, kMaxBatch); t->fire2_slab = carve<uint32_t>(p, kMaxBatch);
    t->fire2_slot = carve<uint32_t>(p, kMaxBatch);
    t->run0 = carve<uint32_t>(p, kMaxBatch);
    t->counts = carve<uint32_t>(p, 16 + 2 * kHistWords);     // counters, then the two passes' digit counts (cleared together)
    t->hist = t->counts + 16;
    t->pkt_slot = carve<uint32_t>(p, kMaxBatch);
    d.first = carve<uint32_t>(p, S);
    if ((size_t)(p - reinterpret_cast<char*>(t->all)) > total) {          // the size list above and the carving must agree
        cudaFree(t->all); delete t; return SF_ERR_ALLOC;
    }
    e = cudaMemset(d.first, 0xFF, S * 4);
    if (e != cudaSuccess) { cudaFree(t->all); delete t; return sf_set_cuda_error(e, "cudaMemset(table)"); }
    t->set[0] = sf_table::SortSet{t->key_a, t->key_b, t->idx_a, t->idx_b, t->run0, t->pkt_slot, t->hist, d.first};
    *out = t;
    return SF_OK;
}

// Makes `stream` wait for the model-phase work of every batch ingested so far (pipelined mode; nothing to do otherwise).
extern "C" int sf_table_flush(sf_ctx* ctx, sf_table* t, void* stream)
{
    if (!ctx || !t) return SF_ERR_ARG;
    if (!t->pipelined || !t->outstanding) return SF_OK;
    SF_CUDA(cudaSetDevice(ctx->device));
    // the model stream runs the batches in order: the last recorded "done" event covers all of them
    const uint32_t last = (uint32_t)((t->n_batches - 1) & 1u);
    SF_CUDA(cudaStreamWaitEvent((cudaStream_t)stream, t->ev_done[last], 0));
    return SF_OK;
}

extern "C" int sf_table_set_pipelined(sf_ctx* ctx, sf_table* t, int on)
{
    if (!ctx || !t) return SF_ERR_ARG;
    SF_CUDA(cudaSetDevice(ctx->device));
    if (!on) {
        if (t->pipelined) { SF_CUDA(cudaStreamSynchronize(t->model_stream)); t->outstanding = false; }
        t->pipelined = 0;
        return SF_OK;
    }
    if (t->pipelined) return SF_OK;
    if (!t->all2) {
        const size_t S = t->d.n_slots;
        size_t total = 0;
        for (int k = 0; k < 6; k++) total += sf_align256((size_t)kMaxBatch * 4);
        total += sf_align256((size_t)2 * kHistWords * 4) + sf_align256(S * 4);
        cudaError_t e = cudaMalloc(&t->all2, total);
        if (e != cudaSuccess) { sf_set_cuda_error(e, "cudaMalloc(table, second sort set)"); return SF_ERR_ALLOC; }
        char* p = reinterpret_cast<char*>(t->all2);
        sf_table::SortSet& s1 = t->set[1];
        s1.key_a = carve<uint32_t>(p, kMaxBatch); s1.key_b = carve<uint32_t>(p, kMaxBatch);
        s1.idx_a = carve<uint32_t>(p, kMaxBatch); s1.idx_b = carve<uint32_t>(p, kMaxBatch);
        s1.run0 = carve<uint32_t>(p, kMaxBatch); s1.pkt_slot = carve<uint32_t>(p, kMaxBatch);
        s1.hist = carve<uint32_t>(p, 2 * kHistWords);
        s1.first = carve<uint32_t>(p, S);
        SF_CUDA(cudaMemset(t->all2, 0, total));
        SF_CUDA(cudaMemset(s1.first, 0xFF, S * 4));
        SF_CUDA(cudaStreamCreateWithFlags(&t->model_stream, cudaStreamNonBlocking));
        for (int k = 0; k < 2; k++) {
            SF_CUDA(cudaEventCreateWithFlags(&t->ev_sorted[k], cudaEventDisableTiming));
            SF_CUDA(cudaEventCreateWithFlags(&t->ev_done[k], cudaEventDisableTiming));
        }
    }
    SF_CUDA(cudaDeviceSynchronize());                     // whatever ran the plain way so far is done
    t->pipelined = 1;
    t->n_batches = 0;
    t->outstanding = false;
    return SF_OK;
}

extern "C" void sf_table_destroy(sf_table* t) {
    if (!t) return;
    if (t->all2) {
        cudaStreamSynchronize(t->model_stream);
        for (int k = 0; k < 2; k++) { cudaEventDestroy(t->ev_sorted[k]); cudaEventDestroy(t->ev_done[k]); }
        cudaStreamDestroy(t->model_stream);
        cudaFree(t->all2);
    }
    if (t->all) cudaFree(t->all);
    delete t;
}

namespace {
int ingest_chunk(sf_ctx* ctx, sf_table* t, const sf_pkt_batch* batch, const sf_forest* fo, uint32_t F,
                 const sf_slow* slow, const sf_route_cfg* cfg, sf_batch_result* result_dev, void* stream, bool zero_result);
}

// A batch of more than 65,536 packets (the sort keys are 16-bit arrival indices) is ingested as consecutive pieces of at most
// 65,536 packets on the same stream: the table sees the packets in the same order as if they had come in separate calls,
// and the pieces' counts add up in *result_dev.
extern "C" int sf_table_ingest(sf_ctx* ctx, sf_table* t, const sf_pkt_batch* batch, const sf_forest* fo, uint32_t F,
                               const sf_slow* slow, const sf_route_cfg* cfg, sf_batch_result* result_dev, void* stream)
{
    if (!ctx || !t || !batch || !fo || !slow || !cfg || !result_dev || !cfg->tau) return SF_ERR_ARG;
    if (batch->n <= kMaxBatch) return ingest_chunk(ctx, t, batch, fo, F, slow, cfg, result_dev, stream, true);
    for (uint32_t o = 0; o < batch->n; o += kMaxBatch) {
        sf_pkt_batch part = *batch;
        part.src += o; part.dst += o; part.sport += o; part.dport += o; part.proto += o; part.dir += o; part.size += o;
        part.iat_us += o; part.hdr += (size_t)o * kHdr;
        part.n = std::min<uint32_t>(kMaxBatch, batch->n - o);
        const int rc = ingest_chunk(ctx, t, &part, fo, F, slow, cfg, result_dev, stream, o == 0);
        if (rc != SF_OK) return rc;
    }
    return SF_OK;
}

namespace {
int ingest_chunk(sf_ctx* ctx, sf_table* t, const sf_pkt_batch* batch, const sf_forest* fo, uint32_t F,
                 const sf_slow* slow, const sf_route_cfg* cfg, sf_batch_result* result_dev, void* stream, bool zero_result)
{
    if (batch->n > kMaxBatch) return SF_ERR_ARG;
    if (!batch->src || !batch->dst || !batch->sport || !batch->dport || !batch->proto || !batch->dir || !batch->size ||
        !batch->iat_us || !batch->hdr) return SF_ERR_ARG;
    if (F != fo->F || fo->kind != SF_RF || cfg->rule != SF_LC_GT) return SF_ERR_UNSUPPORTED;
    if (slow->arch != SF_SLOW_MLP || cfg->wide_layout != SF_MLP16 || cfg->row_dtype != slow->dtype) return SF_ERR_UNSUPPORTED;
    if (cfg->P * 16 != slow->dims[0] || cfg->P < t->d.slow_pkts) return SF_ERR_ARG;
    SF_CUDA(cudaSetDevice(ctx->device));
    cudaStream_t ss = (cudaStream_t)stream;                   // look-up and sort: the caller's stream
    const uint32_t n = batch->n;
    if (zero_result) SF_CUDA(cudaMemsetAsync(result_dev, 0, sizeof(sf_batch_result), ss));
    if (n == 0) return SF_OK;
    // Pipelined: this batch uses sort set b & 1 and hands over to the table's stream for everything from apply1 on; the set (and
    // its `first` array) is free again when the model phase of batch b - 2 has ended.
    const bool pipe = t->pipelined != 0;
    const uint32_t si = pipe ? (uint32_t)(t->n_batches & 1u) : 0u;
    const sf_table::SortSet& S = t->set[si];
    cudaStream_t st = pipe ? t->model_stream : ss;            // the model phase
    if (pipe && t->n_batches >= 2) SF_CUDA(cudaStreamWaitEvent(ss, t->ev_done[si], 0));
    TableDev d = t->d;
    d.first = S.first;
    // workspace: features, probabilities, decisions, wide rows and slow-model scratch for at most n flows
    const size_t esz = slow->dtype == SF_BF16 ? 2 : 4;
    const uint32_t Cs = slow->dims[slow->n_layers];
    size_t off = 0;
    auto take = [&](size_t bytes) { size_t o = off; off += sf_align256(bytes); return o; };
    const size_t o_feat = take((size_t)n * F * 4), o_lidx = take((size_t)n * fo->T * 2),
                 o_rows = take((size_t)n * slow->dims[0] * esz), o_logits = take((size_t)n * Cs * 4), o_slab_lab = take(n),
                 o_slow = take(sf_slow_scratch_bytes(slow, n));
    int rc = sf_ws_reserve(ctx, off);
    if (rc != SF_OK) return rc;
    sf_ws_reset(ctx);
    char* w = reinterpret_cast<char*>(sf_ws_alloc(ctx, off));
    if (!w) return SF_ERR_ALLOC;
    sf_time_new_record(ctx);
    sf_time_begin(ctx, SF_T_TABLE, ss);
    if (!pipe) {
        SF_CUDA(cudaMemsetAsync(t->counts, 0, (16 + 2 * kHistWords) * sizeof(uint32_t), ss));     // fire counts and digit counts lie together
    } else {
        SF_CUDA(cudaMemsetAsync(S.hist, 0, 2 * kHistWords * sizeof(uint32_t), ss));
    }
    const uint32_t blocks = (n + 255) / 256;
    probe_kernel<<<blocks, 256, 0, ss>>>(d, *batch, S.pkt_slot, result_dev, ctx->d_state);
    SF_LAUNCH_CHECK("probe_kernel");
    const uint32_t nblk = (n + kTile - 1) / kTile;
    // from here on every kernel of the batch is a chained launch (set up while its predecessor drains)
    SF_CUDA(sf_launch_chained(key_kernel, blocks, 256, 0, ss, d, S.pkt_slot, n, S.key_a, S.idx_a, S.hist));
    {
        // 16-bit keys: two 8-bit passes, ping-ponging between the two buffers, end in (key_a, idx_a)
        SF_CUDA(sf_launch_chained(radix8_scatter_kernel, nblk, 256, 0, ss, S.key_a, S.idx_a, S.key_b, S.idx_b, n, 0u, S.hist, nblk,
                                  S.hist + kHistWords, (uint32_t*)nullptr));
        SF_CUDA(sf_launch_chained(radix8_scatter_kernel, nblk, 256, 0, ss, S.key_b, S.idx_b, S.key_a, S.idx_a, n, 8u, S.hist + kHistWords, nblk,
                                  (uint32_t*)nullptr, S.run0));
    }
    if (pipe) {
        SF_CUDA(cudaEventRecord(t->ev_sorted[si], ss));
        SF_CUDA(cudaStreamWaitEvent(st, t->ev_sorted[si], 0));
        SF_CUDA(cudaMemsetAsync(t->counts, 0, 16 * sizeof(uint32_t), st));                       // this batch's fire counts
        t->n_batches++;
        t->outstanding = true;
    }
    SF_CUDA(sf_launch_chained(apply1_kernel, blocks, 256, 0, st, d, *batch, S.key_a, S.idx_a, S.run0, S.pkt_slot, t->rank, t->pos, t->fire1_slot, t->counts));
    sf_time_end(ctx, SF_T_TABLE, st);
    // S1..S3 on the flows that just completed their fast context (count stays on the device); the feature kernel reads
    // their packets in place, through the list of their slots
    sf_packets fpk;
    fpk.size = d.f_size; fpk.iat_us = d.f_iat; fpk.dir_bits = d.f_dir; fpk.hdr = nullptr; fpk.n_valid = nullptr;
    fpk.n_flows = n; fpk.pitch_pkts = d.fast_pkts; fpk.hdr_bytes = 0;
    float* feat = reinterpret_cast<float*>(w + o_feat);
    sf_time_begin(ctx, SF_T_FOREST, st);
    // a few hundred flows fire per batch: trees spread over the grid, one leaf index per flow and tree; the kernel computes
    // the fired flows' features itself, in its shared-memory tile, straight from the table's fast contexts ...
    rc = sf_launch_forest_leaf_index_packets(fo, &fpk, d.fast_pkts, t->fire1_slot, n, reinterpret_cast<uint16_t*>(w + o_lidx), st, &t->counts[0]);
    if (rc == SF_ERR_UNSUPPORTED) {                        // (planes not laid out for that: features first, then the trees)
        rc = sf_launch_extract(&fpk, d.fast_pkts, F, feat, st, &t->counts[0], t->fire1_slot);
        if (rc == SF_OK) rc = sf_launch_forest_leaf_index(fo, feat, n, reinterpret_cast<uint16_t*>(w + o_lidx), st, &t->counts[0]);
    }
    sf_time_end(ctx, SF_T_FOREST, st);
    if (rc != SF_OK) return rc;
    sf_time_begin(ctx, SF_T_SCORE, st);
    // ... then leaf sums, score, decision and the table update in one kernel (16 lanes per flow)
    SF_CUDA(sf_launch_chained(fast_finish_kernel, std::min<uint32_t>((n * 16u + 255) / 256, (uint32_t)ctx->num_sms * 2u), 256, 0, st, d, t->fire1_slot,
                              t->counts, reinterpret_cast<const uint16_t*>(w + o_lidx), fo->d_leaf, fo->T, 1u << fo->depth, fo->C, cfg->tau,
                              result_dev, ctx->d_state));
    SF_CUDA(sf_launch_chained(apply2_kernel, blocks, 256, 0, st, d, *batch, S.key_a, S.idx_a, S.pkt_slot, t->rank, t->pos, t->fire2_slab,
                              t->fire2_slot, t->counts, result_dev, ctx->d_state));
    sf_time_end(ctx, SF_T_SCORE, st);
    // S4 on the flows that just completed their slow context
    sf_packets spk;
    spk.size = d.s_size; spk.iat_us = d.s_iat; spk.dir_bits = d.s_dir; spk.hdr = d.s_hdr; spk.n_valid = nullptr;
    spk.n_flows = d.slow_slabs; spk.pitch_pkts = d.slow_pkts; spk.hdr_bytes = kHdr;
    sf_route_cfg gcfg = *cfg;
    gcfg.P_real = d.slow_pkts;
    sf_time_begin(ctx, SF_T_GATHER, st);
    rc = sf_launch_gather(ctx, &gcfg, &spk, t->fire2_slab, &t->counts[1], n, w + o_rows, st);
    sf_time_end(ctx, SF_T_GATHER, st);
    if (rc != SF_OK) return rc;
    rc = sf_launch_slow(ctx, slow, w + o_rows, &t->counts[1], n, reinterpret_cast<float*>(w + o_logits),
                        reinterpret_cast<uint8_t*>(w + o_slab_lab), w + o_slow, st, false);
    if (rc != SF_OK) return rc;
    SF_CUDA(sf_launch_chained(apply_slow_kernel, blocks, 256, 0, st, d, t->fire2_slot, t->counts, reinterpret_cast<const uint8_t*>(w + o_slab_lab),
                              result_dev, ctx->d_state));
    if (pipe) SF_CUDA(cudaEventRecord(t->ev_done[si], st));
    return SF_OK;
}
}  // namespace

// The same with a batch that lives in HOST memory: the nine planes are copied to the context's device
// staging buffer on the stream (one copy per plane), the batch is ingested, the counts come back.
extern "C" int sf_table_ingest_host(sf_ctx* ctx, sf_table* t, const sf_pkt_batch* bh, const sf_forest* fo, uint32_t F,
                                    const sf_slow* slow, const sf_route_cfg* cfg, sf_batch_result* result_host_out, void* stream)
{
    if (!ctx || !t || !bh || !result_host_out) return SF_ERR_ARG;
    if (bh->n && (!bh->src || !bh->dst || !bh->sport || !bh->dport || !bh->proto || !bh->dir || !bh->size || !bh->iat_us || !bh->hdr))
        return SF_ERR_ARG;
    SF_CUDA(cudaSetDevice(ctx->device));
    cudaStream_t st = (cudaStream_t)stream;
    const size_t n = bh->n;
    const void* src[9] = {bh->src, bh->dst, bh->sport, bh->dport, bh->proto, bh->dir, bh->size, bh->iat_us, bh->hdr};
    const size_t bytes[9] = {n * 4, n * 4, n * 2, n * 2, n, n, n * 2, n * 4, n * kHdr};
    size_t off[10], total = 0;
    for (int i = 0; i < 9; i++) { off[i] = total; total += sf_align256(bytes[i]); }
    off[9] = total; total += 256;                                        // the counts
    if (total > ctx->stage_bytes) {
        SF_CUDA(cudaDeviceSynchronize());
        if (ctx->stage) { cudaFree(ctx->stage); ctx->stage = nullptr; ctx->stage_bytes = 0; }
        const size_t want = std::max(total, (size_t)kMaxBatch * 40 + 4096);     // once: room for the largest batch
        cudaError_t e = cudaMalloc(&ctx->stage, want);
        if (e != cudaSuccess) { sf_set_cuda_error(e, "cudaMalloc(staging)"); return SF_ERR_ALLOC; }
        ctx->stage_bytes = want;
    }
    char* sb = ctx->stage;
    for (int i = 0; i < 9; i++)
        if (bytes[i]) SF_CUDA(cudaMemcpyAsync(sb + off[i], src[i], bytes[i], cudaMemcpyHostToDevice, st));
    sf_pkt_batch bd;
    bd.src = (const uint32_t*)(sb + off[0]); bd.dst = (const uint32_t*)(sb + off[1]);
    bd.sport = (const uint16_t*)(sb + off[2]); bd.dport = (const uint16_t*)(sb + off[3]);
    bd.proto = (const uint8_t*)(sb + off[4]); bd.dir = (const uint8_t*)(sb + off[5]);
    bd.size = (const uint16_t*)(sb + off[6]); bd.iat_us = (const uint32_t*)(sb + off[7]);
    bd.hdr = (const uint8_t*)(sb + off[8]); bd.n = bh->n;
    sf_batch_result* res_dev = reinterpret_cast<sf_batch_result*>(sb + off[9]);
    int rc = sf_table_ingest(ctx, t, &bd, fo, F, slow, cfg, res_dev, stream);
    if (rc != SF_OK) return rc;
    rc = sf_table_flush(ctx, t, stream);                                 // pipelined mode: the counts are complete after the model phase
    if (rc != SF_OK) return rc;
    SF_CUDA(cudaMemcpyAsync(result_host_out, res_dev, sizeof(sf_batch_result), cudaMemcpyDeviceToHost, st));
    SF_CUDA(cudaStreamSynchronize(st));
    return SF_OK;
}

extern "C" int sf_table_set_time(sf_table* t, uint32_t now)
{
    if (!t) return SF_ERR_ARG;
    t->d.now = now;
    return SF_OK;
}

extern "C" int sf_table_sweep(sf_ctx* ctx, sf_table* t, uint32_t now, uint32_t idle_timeout, int rearm,
                              sf_sweep_result* result_dev, void* stream)
{
    if (!ctx || !t || !result_dev) return SF_ERR_ARG;
    SF_CUDA(cudaSetDevice(ctx->device));
    cudaStream_t st = (cudaStream_t)stream;
    { const int rcf = sf_table_flush(ctx, t, stream); if (rcf != SF_OK) return rcf; }
    SF_CUDA(cudaMemsetAsync(result_dev, 0, sizeof(sf_sweep_result), st));
    sweep_kernel<<<(t->d.n_slots + 255) / 256, 256, 0, st>>>(t->d, now, idle_timeout, rearm, result_dev);
    SF_LAUNCH_CHECK("sweep_kernel");
    return SF_OK;
}

extern "C" int sf_table_lookup(sf_ctx* ctx, const sf_table* t, const sf_key* keys_dev, uint32_t n,
                               sf_flow_result* out_dev, void* stream)
{
    if (!ctx || !t || (n && (!keys_dev || !out_dev))) return SF_ERR_ARG;
    SF_CUDA(cudaSetDevice(ctx->device));
    if (n == 0) return SF_OK;
    { const int rcf = sf_table_flush(ctx, const_cast<sf_table*>(t), stream); if (rcf != SF_OK) return rcf; }
    lookup_kernel<<<(n + 255) / 256, 256, 0, (cudaStream_t)stream>>>(t->d, keys_dev, n, out_dev);
    SF_LAUNCH_CHECK("lookup_kernel");
    return SF_OK;
}

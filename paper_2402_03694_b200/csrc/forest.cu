// S2: tree-ensemble inference (the cascade's fast model).
//
// One thread per flow, 512 flows per block.  The block's feature rows sit in shared
// memory transposed ([feature][flow], so a lane's read of x[fid] hits bank = lane
// whatever fid is).  The ensemble streams through shared memory in chunks of whole
// trees: a producer warp (one extra warp per block) issues a bulk copy (cp.async.bulk, completion on a
// "full" mbarrier) of a chunk as soon as every walking warp has released that buffer (an "empty" mbarrier
// with one arrival per warp), so the copy costs no load/store instructions and no warp ever waits at a
// block-wide barrier for the slowest one: a warp that is done with a chunk goes straight on to the next.  A node is 8 bytes {threshold bits, byte offset of its feature's
// row in the tile}; trees are 1-based heaps.  A walk keeps the node's shared-memory
// ADDRESS as its state (addr' = 2*addr + (go right ? 8 : 0) - base), so a level costs
// six instructions: node load, feature address, feature load, compare, select, shift-add.
// Each thread walks NCH trees of the chunk at once (independent dependency chains
// hide the shared-memory latency), then adds their leaf payloads in tree order
// t = 0..T-1, which fixes the fp32 summation order.  Random-forest leaf vectors are
// gathered from L2 one group ahead of their use; boosted-tree leaf scalars travel
// with their tree's nodes in the shared-memory image.
// The walk keeps the SM's load/store pipe busy (shared-memory wavefronts), and a gather of one
// 32-byte sector per lane through the same pipe costs as much as nine levels of the walk.  So,
// where the class count is a multiple of four, the leaf vectors are fetched through the texture
// path instead (a linear texture of 16-byte integer texels over the same table: raw bits, no
// filtering): it has its own queue into the L1, and the gather then overlaps the walk (115 -> 88
// cycles per warp and tree in a microbenchmark of exactly this mix).
// The streaming path, where a launch carries a few hundred flows, has kernels of its own further down
// (trees spread over the grid as well as flows).
#include "tc_common.cuh"
#include "extract_device.cuh"
#include <algorithm>
#include <new>
#include <stdlib.h>
#include <string.h>

namespace {

constexpr uint32_t kB = 512;                       // flows (= threads) per block
constexpr uint32_t kBSmall = 128;                  // ... of a tile of the small-batch kernels (streaming: a few hundred flows per launch)
constexpr uint32_t kMaxSmem = 232448;              // 227 KB

__device__ __forceinline__ uint32_t smem_u32(const void* p) { return (uint32_t)__cvta_generic_to_shared(p); }
__device__ __forceinline__ uint2 lds64(uint32_t a) {
    uint2 v;
    asm volatile("ld.shared.v2.u32 {%0, %1}, [%2];\n" : "=r"(v.x), "=r"(v.y) : "r"(a));
    return v;
}
__device__ __forceinline__ float lds32f(uint32_t a) {
    float v;
    asm volatile("ld.shared.f32 %0, [%1];\n" : "=f"(v) : "r"(a));
    return v;
}

// The two top levels of every tree (nodes 1, 2, 3 of the 1-based heap) as a kernel argument: kernel arguments live in
// the constant bank, a tree index is the same in every lane, so these loads never touch the load/store pipe that the
// rest of the walk saturates (two 64-bit shared-memory loads = four wavefronts less per warp and tree).  Measured on
// 500 boosted trees of depth 6: 4.56 -> 4.20 ms; a third level this way (four more loads, six selects) cost more than it
// saved (5.07 ms), and random forests of depth 10 to 12 gained nothing, so only binary boosted trees take this path.
constexpr uint32_t kTopMaxTrees = SF_FOREST_TOP_TREES;
typedef sf_forest_top ForestTop;

// Walk NCH consecutive trees (shared-memory images at base, base+stride, ...) for the
// flow whose feature column starts at xbase; returns leaf indices.
// TOPC: levels 0 and 1 come from `top` (trees t_first, t_first + 1, ...; depth >= 2), the walk through shared memory
// starts at level 2.
template <int NCH, bool TOPC = false>
__device__ __forceinline__ void walk(uint32_t base, uint32_t stride, uint32_t xbase, uint32_t depth, uint32_t (&leaf)[NCH],
                                     const ForestTop* top = nullptr, uint32_t t_first = 0) {
    uint32_t a[NCH], left[NCH], right[NCH];
#pragma unroll
    for (int c = 0; c < NCH; c++) {
        const uint32_t b = base + c * stride;
        a[c] = b + 8u;                 // node 1
        left[c] = 0u - b;              // addr' = 2*addr - base      (child 2i)
        right[c] = 8u - b;             // addr' = 2*addr - base + 8  (child 2i+1)
    }
    if (TOPC) {
        float x0[NCH], x1[NCH];
        uint2 n1[NCH], n2[NCH];
#pragma unroll
        for (int c = 0; c < NCH; c++) { n1[c] = top->n[t_first + c][0]; x0[c] = lds32f(xbase + n1[c].y); }
#pragma unroll
        for (int c = 0; c < NCH; c++) {
            const bool r0 = !(x0[c] <= __uint_as_float(n1[c].x));
            const uint2 nl = top->n[t_first + c][1], nr = top->n[t_first + c][2];
            n2[c].x = r0 ? nr.x : nl.x; n2[c].y = r0 ? nr.y : nl.y;
            a[c] = r0 ? 48u : 32u;                                   // byte offset of node 6 or 4: 8 * (4 + 2 * r0)
        }
#pragma unroll
        for (int c = 0; c < NCH; c++) x1[c] = lds32f(xbase + n2[c].y);
#pragma unroll
        for (int c = 0; c < NCH; c++) a[c] = base + c * stride + a[c] + ((x1[c] <= __uint_as_float(n2[c].x)) ? 0u : 8u);
    }
    for (uint32_t l = TOPC ? 2u : 0u; l < depth; l++) {
        uint2 nd[NCH];
        float x[NCH];
#pragma unroll
        for (int c = 0; c < NCH; c++) nd[c] = lds64(a[c]);
#pragma unroll
        for (int c = 0; c < NCH; c++) x[c] = lds32f(xbase + nd[c].y);
#pragma unroll
        for (int c = 0; c < NCH; c++) a[c] = 2u * a[c] + ((x[c] <= __uint_as_float(nd[c].x)) ? left[c] : right[c]);
    }
#pragma unroll
    for (int c = 0; c < NCH; c++) leaf[c] = ((a[c] - (base + c * stride)) >> 3) - (1u << depth);
}

template <int C>
__device__ __forceinline__ void load_leaf_vec(const float* __restrict__ lv, float (&p)[C]) {
    if ((C & 7) == 0) {
        // 32-byte vectors: one 256-bit load touches one sector per lane
#pragma unroll
        for (int c = 0; c < C; c += 8)
            asm volatile("ld.global.nc.v8.f32 {%0, %1, %2, %3, %4, %5, %6, %7}, [%8];\n"
                         : "=f"(p[c]), "=f"(p[c + 1]), "=f"(p[c + 2]), "=f"(p[c + 3]),
                           "=f"(p[c + 4]), "=f"(p[c + 5]), "=f"(p[c + 6]), "=f"(p[c + 7])
                         : "l"(lv + c));
    } else if ((C & 3) == 0) {
#pragma unroll
        for (int c = 0; c < C; c += 4) {
            float4 v = __ldg(reinterpret_cast<const float4*>(lv + c));
            p[c] = v.x; p[c + 1] = v.y; p[c + 2] = v.z; p[c + 3] = v.w;
        }
    } else {
#pragma unroll
        for (int c = 0; c < C; c++) p[c] = __ldg(lv + c);
    }
}

// the same vector through the texture path: C / 4 texels of 16 bytes, starting at texel index `texel`.
// A vector of 16 classes (four texels per lane) would make the texture queue the bottleneck in its turn, so from
// C = 16 on the second half of the vector comes through the load/store pipe (one 256-bit load): both paths share the work.
template <int C>
__device__ __forceinline__ void load_leaf_vec_tex(cudaTextureObject_t tex, uint32_t texel, const float* __restrict__ lv, float (&p)[C]) {
    constexpr int CT = (C >= 16 && (C % 16) == 0) ? C / 2 : C;       // classes fetched as texels
#pragma unroll
    for (int c = 0; c < CT; c += 4) {
        const uint4 v = tex1Dfetch<uint4>(tex, (int)(texel + c / 4));
        p[c] = __uint_as_float(v.x); p[c + 1] = __uint_as_float(v.y); p[c + 2] = __uint_as_float(v.z); p[c + 3] = __uint_as_float(v.w);
    }
#pragma unroll
    for (int c = CT; c < C; c += 8)
        asm volatile("ld.global.nc.v8.f32 {%0, %1, %2, %3, %4, %5, %6, %7}, [%8];\n"
                     : "=f"(p[c]), "=f"(p[c + 1]), "=f"(p[c + 2]), "=f"(p[c + 3]), "=f"(p[c + 4]), "=f"(p[c + 5]), "=f"(p[c + 6]), "=f"(p[c + 7])
                     : "l"(lv + c));
}

// KIND: SF_RF (leaf = C-vector of class probabilities in global memory), SF_GBDT (leaf =
// scalar stored behind the tree's nodes in the image, C = 1) or SF_GBDT_MC (scalar leaves, tree t
// adds to class t mod C; a chunk holds whole boosting rounds, so the class of every tree in the
// unrolled round loop is a compile-time register index).  NCH: trees walked at once.
// TEX: leaf vectors come through the texture object (random forests whose C is a multiple of 4).
template <int KIND, int C, int NCH, uint32_t KB, bool TEX, bool TOPC>
__global__ void __launch_bounds__(KB + 32, 1)
forest_kernel(const __grid_constant__ ForestTop top, const float* __restrict__ feat, uint32_t n, uint32_t F,
              const unsigned char* __restrict__ image, const float* __restrict__ leaf, cudaTextureObject_t leaf_tex,
              uint32_t T, uint32_t depth, uint32_t tree_stride, uint32_t trees_per_chunk, uint32_t chunk_bytes,
              float* __restrict__ out, uint16_t* __restrict__ leaf_idx, sf_dev_state* st, const uint32_t* __restrict__ n_dev,
              const sf_fused_route fr)
{
    extern __shared__ __align__(16) unsigned char smem_raw[];
    // a chained launch: barrier set-up and the first tree chunks (model data) overlap the previous kernel's tail; every thread waits
    // for that kernel before it reads a count or a feature, or writes anything
    sf_chain_release();
    if (n_dev) { sf_chain_wait(); n = min(n, *n_dev); }     // optional device-side flow count (streaming path)
    if (blockIdx.x * KB >= n) {
        sf_chain_wait();
        if (fr.tau && threadIdx.x == 0) fr.block_counts[blockIdx.x] = 0;
        return;
    }
    const uint32_t sbuf0 = smem_u32(smem_raw);
    float* xs = reinterpret_cast<float*>(smem_raw + 2 * (size_t)chunk_bytes);       // [F][KB]
    uint64_t* bars = reinterpret_cast<uint64_t*>(smem_raw + 2 * (size_t)chunk_bytes + (size_t)F * KB * 4);   // full[2], empty[2], flag
    uint64_t* empty = bars + 2;
    volatile uint32_t* abort_flag = reinterpret_cast<volatile uint32_t*>(bars + 4);
    const uint32_t xbase = smem_u32(xs) + threadIdx.x * 4u;
    const uint32_t f = blockIdx.x * KB + threadIdx.x;
    const bool producer = threadIdx.x >= KB;                 // the extra warp
    const bool live = !producer && f < n;
    const uint32_t n_leaf = 1u << depth;
    const uint32_t n_chunks = (T + trees_per_chunk - 1) / trees_per_chunk;

    if (threadIdx.x == 0) {
        sftc::mbar_init(&bars[0], 1);
        sftc::mbar_init(&bars[1], 1);
        sftc::mbar_init(&empty[0], KB / 32);
        sftc::mbar_init(&empty[1], KB / 32);
        *abort_flag = 0;
        sftc::fence_barrier_init();
    }
    __syncthreads();                              // barriers initialised: the producer starts streaming trees right away

    if (producer) {
        if (threadIdx.x == KB) {
            for (uint32_t ck = 0; ck < n_chunks; ck++) {
                // the buffer's previous chunk (ck - 2) has been released by every walking warp
                if (ck >= 2 && !sftc::mbar_wait_relaxed(&empty[ck & 1u], ((ck >> 1) - 1u) & 1u, abort_flag)) break;
                const uint32_t t0 = ck * trees_per_chunk;
                const uint32_t nt = min(trees_per_chunk, T - t0);
                const uint32_t bytes = nt * tree_stride;                         // a multiple of 16
                sftc::mbar_expect_tx(&bars[ck & 1u], bytes);
                sftc::bulk_load(smem_raw + (size_t)(ck & 1u) * chunk_bytes, image + (size_t)t0 * tree_stride, bytes, &bars[ck & 1u]);
            }
        }
        return;
    }

    sf_chain_wait();
    if (live) {
        const float* row = feat + (size_t)f * F;
        if ((F & 3) == 0) {
            for (uint32_t j = 0; j < F; j += 4) {
                float4 v = __ldg(reinterpret_cast<const float4*>(row + j));
                xs[(j + 0) * KB + threadIdx.x] = v.x; xs[(j + 1) * KB + threadIdx.x] = v.y;
                xs[(j + 2) * KB + threadIdx.x] = v.z; xs[(j + 3) * KB + threadIdx.x] = v.w;
            }
        } else {
            for (uint32_t j = 0; j < F; j++) xs[j * KB + threadIdx.x] = row[j];
        }
    } else {
        for (uint32_t j = 0; j < F; j++) xs[j * KB + threadIdx.x] = 0.0f;
    }
    // the feature tile is read by its own thread only (column threadIdx.x of every row): no barrier needed

    float acc[C];
    float pend[NCH][C];
#pragma unroll
    for (int c = 0; c < C; c++) acc[c] = 0.0f;
    int n_pend = 0;                                   // leaf vectors in flight (RF)

    auto flush_pending = [&]() {
#pragma unroll
        for (int k = 0; k < NCH; k++)
            if (k < n_pend) {
#pragma unroll
                for (int c = 0; c < C; c++) acc[c] = __fadd_rn(acc[c], pend[k][c]);
            }
        n_pend = 0;
    };

    for (uint32_t ck = 0; ck < n_chunks; ck++) {
        // every thread waits for this chunk's bytes (bounded: all give up together if they never land)
        if (!sftc::mbar_wait(&bars[ck & 1u], (ck >> 1) & 1u, abort_flag)) break;
        const uint32_t cur = sbuf0 + (ck & 1u) * chunk_bytes;
        const uint32_t t0 = ck * trees_per_chunk;
        const uint32_t nt = min(trees_per_chunk, T - t0);
        uint32_t tt = 0;
        if (KIND == SF_GBDT_MC) {
            for (uint32_t r0 = 0; r0 < nt; r0 += C) {             // one boosting round: classes 0..C-1 in order
#pragma unroll
                for (int c0 = 0; c0 + NCH <= C; c0 += NCH) {
                    uint32_t l[NCH];
                    float v[NCH];
                    walk<NCH>(cur + (r0 + c0) * tree_stride, tree_stride, xbase, depth, l);
                    if (leaf_idx && live) {
#pragma unroll
                        for (int k = 0; k < NCH; k++) leaf_idx[(size_t)f * T + t0 + r0 + c0 + k] = (uint16_t)l[k];
                    }
#pragma unroll
                    for (int k = 0; k < NCH; k++) v[k] = lds32f(cur + (r0 + c0 + k) * tree_stride + n_leaf * 8u + l[k] * 4u);
#pragma unroll
                    for (int k = 0; k < NCH; k++) acc[c0 + k] = __fadd_rn(acc[c0 + k], v[k]);
                }
#pragma unroll
                for (int c1 = (C / NCH) * NCH; c1 < C; c1++) {
                    uint32_t l[1];
                    walk<1>(cur + (r0 + c1) * tree_stride, tree_stride, xbase, depth, l);
                    if (leaf_idx && live) leaf_idx[(size_t)f * T + t0 + r0 + c1] = (uint16_t)l[0];
                    acc[c1] = __fadd_rn(acc[c1], lds32f(cur + (r0 + c1) * tree_stride + n_leaf * 8u + l[0] * 4u));
                }
            }
            tt = nt;
        }
        for (; tt + NCH <= nt; tt += NCH) {
            uint32_t l[NCH];
            walk<NCH, TOPC>(cur + tt * tree_stride, tree_stride, xbase, depth, l, &top, t0 + tt);
            if (leaf_idx && live) {
#pragma unroll
                for (int k = 0; k < NCH; k++) leaf_idx[(size_t)f * T + t0 + tt + k] = (uint16_t)l[k];
            }
            if (KIND == SF_GBDT) {
                float v[NCH];
#pragma unroll
                for (int k = 0; k < NCH; k++) v[k] = lds32f(cur + (tt + k) * tree_stride + n_leaf * 8u + l[k] * 4u);
#pragma unroll
                for (int k = 0; k < NCH; k++) acc[0] = __fadd_rn(acc[0], v[k]);
            } else {
                flush_pending();                      // the previous group's vectors have landed by now
#pragma unroll
                for (int k = 0; k < NCH; k++) {
                    if (TEX) load_leaf_vec_tex<C>(leaf_tex, ((t0 + tt + k) * n_leaf + l[k]) * (C / 4), leaf + ((size_t)(t0 + tt + k) * n_leaf + l[k]) * C, pend[k]);
                    else load_leaf_vec<C>(leaf + ((size_t)(t0 + tt + k) * n_leaf + l[k]) * C, pend[k]);
                }
                n_pend = NCH;
            }
        }
        for (; tt < nt; tt++) {                       // ragged end of the chunk: one tree at a time
            uint32_t l[1];
            walk<1, TOPC>(cur + tt * tree_stride, tree_stride, xbase, depth, l, &top, t0 + tt);
            if (leaf_idx && live) leaf_idx[(size_t)f * T + t0 + tt] = (uint16_t)l[0];
            if (KIND == SF_GBDT) {
                acc[0] = __fadd_rn(acc[0], lds32f(cur + tt * tree_stride + n_leaf * 8u + l[0] * 4u));
            } else {
                flush_pending();
                if (TEX) load_leaf_vec_tex<C>(leaf_tex, ((t0 + tt) * n_leaf + l[0]) * (C / 4), leaf + ((size_t)(t0 + tt) * n_leaf + l[0]) * C, pend[0]);
                else load_leaf_vec<C>(leaf + ((size_t)(t0 + tt) * n_leaf + l[0]) * C, pend[0]);
                n_pend = 1;
            }
        }
        __syncwarp();             // this warp is done with the buffer: one arrival per warp lets the producer refill it
        if ((threadIdx.x & 31u) == 0) sftc::mbar_arrive(&empty[ck & 1u]);
    }
    if (KIND == SF_RF) flush_pending();
    const bool aborted = *abort_flag != 0;
    if (aborted && threadIdx.x == 0) sf_dev_set_error(st, SF_ERR_DEVICE_TIMEOUT);
    bool assigned = false;
    if (live && !aborted) {
        if (KIND == SF_GBDT) {
            out[f] = acc[0];
            if (fr.tau) {                             // |margin| < tau (the binary rule taken in margin space), label = margin > 0
                const float m = acc[0];
                assigned = fabsf(m) < __ldg(fr.tau);
                const uint8_t a = (m > 0.0f) ? 1 : 0;
                fr.decision[f] = assigned ? 1 : 0; fr.label_fast[f] = a;
                if (fr.label_out) fr.label_out[f] = a;
                if (fr.stage_out) fr.stage_out[f] = 1;
            }
        } else if (KIND == SF_GBDT_MC) {
#pragma unroll
            for (int c = 0; c < C; c++) out[(size_t)f * C + c] = acc[c];
        } else {
            const float fT = __uint2float_rn(T);
            float mx = 0.0f; uint32_t a = 0;
#pragma unroll
            for (int c = 0; c < C; c++) {
                const float p = __fdiv_rn(acc[c], fT);
                out[(size_t)f * C + c] = p;
                if (c == 0 || p > mx) { mx = p; a = c; }      // lowest index on ties
            }
            if (fr.tau) {                             // least confidence 1 - max > tau[label], strict
                assigned = __fsub_rn(1.0f, mx) > __ldg(fr.tau + a);
                fr.decision[f] = assigned ? 1 : 0; fr.label_fast[f] = (uint8_t)a;
                if (fr.label_out) fr.label_out[f] = (uint8_t)a;
                if (fr.stage_out) fr.stage_out[f] = 1;
            }
        }
    }
    if (fr.tau) {
        // assigned flows of this block: one count per warp in the warp's own first column of the feature tile (nobody
        // reads that column any more), then a barrier of the walking warps only (the producer warp has left)
        const uint32_t b = __ballot_sync(0xFFFFFFFFu, assigned);
        uint32_t* cnt = reinterpret_cast<uint32_t*>(xs);
        if ((threadIdx.x & 31u) == 0) cnt[threadIdx.x] = __popc(b);
        asm volatile("bar.sync 1, %0;" ::"r"(KB) : "memory");
        if (threadIdx.x == 0) {
            uint32_t tot = 0;
            for (uint32_t w = 0; w < KB / 32; w++) tot += cnt[w * 32];
            fr.block_counts[blockIdx.x] = tot;
        }
    }
}

// ---- small batches (the streaming path: a few hundred flows fire per batch) ----------------------------------
// With so few flows a block of the kernel above walks the whole forest on its own, chunk after chunk, with four
// warps and nothing to hide the latency behind.  Here the trees are spread over the grid as well: a work item is
// (tile of 128 flows, slice of trees that fits one buffer); persistent blocks take items in turn, walk the slice
// and write each tree's leaf index.  A second kernel then adds every flow's leaf vectors in tree order
// t = 0..T-1 (the same fp32 sums, bit for bit, as the fused kernel) and divides by T.
// G > 0: the features are not read from `feat` but computed here, straight into the tile, from the flows' packets
// (8 * G statistics of the first N packets of row row_ids[f] of the planes pk; rows 16-byte aligned, no n_valid):
// one launch less on a path whose cost is launch latency.
struct LeafIndexPackets { const uint16_t* size; const uint32_t* iat; const uint32_t* dir_bits; const uint32_t* row_ids; uint32_t pitch, N; };

template <int NCH, int G>
__global__ void __launch_bounds__(kBSmall, 2)
forest_leaf_index_kernel(const float* __restrict__ feat, uint32_t n, uint32_t F, const unsigned char* __restrict__ image,
                         uint32_t T, uint32_t depth, uint32_t tree_stride, uint32_t trees_per_item, uint32_t buf_bytes,
                         uint16_t* __restrict__ leaf_idx, sf_dev_state* st, const uint32_t* __restrict__ n_dev, LeafIndexPackets pk)
{
    extern __shared__ __align__(16) unsigned char smem_raw[];
    sf_chain_enter();
    if (n_dev) n = min(n, *n_dev);
    float* xs = reinterpret_cast<float*>(smem_raw + buf_bytes);                                  // [F][128]
    uint64_t* bar = reinterpret_cast<uint64_t*>(smem_raw + buf_bytes + (size_t)F * kBSmall * 4);
    volatile uint32_t* abort_flag = reinterpret_cast<volatile uint32_t*>(bar + 1);
    const uint32_t n_tiles = (n + kBSmall - 1) / kBSmall, n_slices = (T + trees_per_item - 1) / trees_per_item;
    const uint32_t n_items = n_tiles * n_slices;
    if (blockIdx.x >= n_items) return;
    const uint32_t cur = smem_u32(smem_raw);
    const uint32_t xbase = smem_u32(xs) + threadIdx.x * 4u;
    if (threadIdx.x == 0) { sftc::mbar_init(bar, 1); *abort_flag = 0; sftc::fence_barrier_init(); }
    __syncthreads();
    uint32_t it = 0, tile_loaded = 0xFFFFFFFFu;
    for (uint32_t w = blockIdx.x; w < n_items; w += gridDim.x, it++) {
        const uint32_t tile = w / n_slices, slice = w - tile * n_slices;
        const uint32_t t0 = slice * trees_per_item, nt = min(trees_per_item, T - t0);
        if (threadIdx.x == 0) {
            sftc::mbar_expect_tx(bar, nt * tree_stride);
            sftc::bulk_load(smem_raw, image + (size_t)t0 * tree_stride, nt * tree_stride, bar);
        }
        const uint32_t f = tile * kBSmall + threadIdx.x;
        const bool live = f < n;
        if (tile != tile_loaded) {                          // every thread reads its own column only
            if (live) {
                if (G > 0) {
                    const size_t fr = pk.row_ids ? pk.row_ids[f] : f;
                    sfx::extract_flow<(G > 0 ? G : 1), true>(pk.size, pk.iat, fr, pk.pitch, pk.N, pk.dir_bits[fr * ((pk.pitch + 31) >> 5)],
                                                             sfx::ColOut{xs + threadIdx.x, kBSmall});
                } else {
                    for (uint32_t j = 0; j < F; j++) xs[j * kBSmall + threadIdx.x] = __ldg(feat + (size_t)f * F + j);
                }
            } else {
                for (uint32_t j = 0; j < F; j++) xs[j * kBSmall + threadIdx.x] = 0.0f;
            }
            tile_loaded = tile;
        }
        if (!sftc::mbar_wait(bar, it & 1u, abort_flag)) break;
        uint32_t tt = 0;
        for (; tt + NCH <= nt; tt += NCH) {
            uint32_t l[NCH];
            walk<NCH>(cur + tt * tree_stride, tree_stride, xbase, depth, l);
            if (live) {
#pragma unroll
                for (int k = 0; k < NCH; k++) leaf_idx[(size_t)f * T + t0 + tt + k] = (uint16_t)l[k];
            }
        }
        for (; tt < nt; tt++) {
            uint32_t l[1];
            walk<1>(cur + tt * tree_stride, tree_stride, xbase, depth, l);
            if (live) leaf_idx[(size_t)f * T + t0 + tt] = (uint16_t)l[0];
        }
        __syncthreads();                                    // the buffer is refilled by the next item
    }
    if (*abort_flag && threadIdx.x == 0) sf_dev_set_error(st, SF_ERR_DEVICE_TIMEOUT);
}

// out[f][c] = (sum over t = 0..T-1, in that order, of leaf[t][idx[f][t]][c]) / T; one thread per (flow, class)
__global__ void __launch_bounds__(256)
forest_leaf_sum_kernel(const uint16_t* __restrict__ leaf_idx, const float* __restrict__ leaf, uint32_t n, uint32_t T, uint32_t n_leaf,
                       uint32_t C, float* __restrict__ out, const uint32_t* __restrict__ n_dev)
{
    if (n_dev) n = min(n, *n_dev);
    const uint32_t i = blockIdx.x * blockDim.x + threadIdx.x;
    const uint32_t f = i / C, c = i - f * C;
    if (f >= n) return;
    const uint16_t* idx = leaf_idx + (size_t)f * T;
    float acc = 0.0f;
    uint32_t t = 0;
    for (; t + 8 <= T; t += 8) {                            // eight loads in flight, added in tree order
        float v[8];
#pragma unroll
        for (int k = 0; k < 8; k++) v[k] = __ldg(leaf + ((size_t)(t + k) * n_leaf + idx[t + k]) * C + c);
#pragma unroll
        for (int k = 0; k < 8; k++) acc = __fadd_rn(acc, v[k]);
    }
    for (; t < T; t++) acc = __fadd_rn(acc, __ldg(leaf + ((size_t)t * n_leaf + idx[t]) * C + c));
    out[(size_t)f * C + c] = __fdiv_rn(acc, __uint2float_rn(T));
}

struct Plan { uint32_t chunk_bytes, tpc, nch; size_t smem; };

Plan make_plan(const sf_forest* fo, uint32_t kb = kB) {
    Plan p;
    const size_t feat_bytes = (size_t)fo->F * kb * sizeof(float);
    // two chunk buffers share what the feature tile leaves of the 227 KB: up to 64 KB each
    const uint32_t avail = (uint32_t)(((kMaxSmem - feat_bytes - 48) / 2) & ~(size_t)15);
    p.chunk_bytes = avail < 65536u ? avail : 65536u;
    p.tpc = p.chunk_bytes / fo->tree_stride;          // 0 if one tree does not fit (checked by the callers)
    if (p.tpc > fo->T) p.tpc = fo->T;
    if (fo->kind == SF_GBDT_MC) p.tpc -= p.tpc % fo->C;          // whole boosting rounds per chunk
    p.nch = (fo->kind == SF_GBDT_MC) ? (fo->C >= 4 ? 4u : (fo->C >= 2 ? 2u : 1u)) : (fo->kind == SF_GBDT) ? (p.tpc >= 4 ? 4u : (p.tpc >= 2 ? 2u : 1u)) : (p.tpc >= 2 ? 2u : 1u);
    p.smem = 2 * (size_t)p.chunk_bytes + feat_bytes + 48;       // + four mbarriers and the abort flag
    return p;
}

template <int KIND, int C, int NCH, uint32_t KB = kB, bool TEX = false, bool TOPC = false>
int launch3(const sf_forest* fo, const Plan& p, const float* feat, uint32_t n, float* out, uint16_t* leaf_idx, cudaStream_t st, const uint32_t* n_dev,
            const sf_fused_route& fr) {
    auto k = forest_kernel<KIND, C, NCH, KB, TEX, TOPC>;
    static size_t smem_set_dev[64] = {};               // per kernel instance and device: raise the opt-in limit only when it grows
    size_t& smem_set = smem_set_dev[fo->ctx->device & 63];
    if (p.smem > smem_set) {
        SF_CUDA(cudaFuncSetAttribute(k, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)p.smem));
        smem_set = p.smem;
    }
    const uint32_t grid = (n + KB - 1) / KB;
    SF_CUDA(sf_launch_chained(k, grid, KB + 32, p.smem, st, *fo->h_top, feat, n, fo->F, (const unsigned char*)(KB == kB ? fo->d_image : fo->d_image_small),
                              (const float*)fo->d_leaf, fo->leaf_tex, fo->T, fo->depth, fo->tree_stride, p.tpc, p.chunk_bytes, out, leaf_idx,
                              fo->ctx->d_state, n_dev, fr));
    return SF_OK;
}

template <int C>
int launch_rf(const sf_forest* fo, const float* feat, uint32_t n, float* out, uint16_t* leaf_idx, cudaStream_t st, const uint32_t* n_dev, const sf_fused_route& fr) {
    constexpr bool kTexOk = (C % 4) == 0;                 // whole 16-byte texels per leaf vector
    const bool tex = kTexOk && fo->leaf_tex != 0;
    const Plan p = make_plan(fo);
    if (p.tpc == 0) return SF_ERR_UNSUPPORTED;
    if (p.nch == 2) {
        if (tex) return launch3<SF_RF, C, 2, kB, kTexOk>(fo, p, feat, n, out, leaf_idx, st, n_dev, fr);
        return launch3<SF_RF, C, 2>(fo, p, feat, n, out, leaf_idx, st, n_dev, fr);
    }
    if (tex) return launch3<SF_RF, C, 1, kB, kTexOk>(fo, p, feat, n, out, leaf_idx, st, n_dev, fr);
    return launch3<SF_RF, C, 1>(fo, p, feat, n, out, leaf_idx, st, n_dev, fr);
}

int launch_gbdt(const sf_forest* fo, const float* feat, uint32_t n, float* out, uint16_t* leaf_idx, cudaStream_t st, const uint32_t* n_dev, const sf_fused_route& fr) {
    const Plan p = make_plan(fo);
    if (p.tpc == 0) return SF_ERR_UNSUPPORTED;
    if (fo->top_ok) {                                 // the two top levels of every tree travel as a kernel argument
        if (p.nch == 4) return launch3<SF_GBDT, 1, 4, kB, false, true>(fo, p, feat, n, out, leaf_idx, st, n_dev, fr);
        if (p.nch == 2) return launch3<SF_GBDT, 1, 2, kB, false, true>(fo, p, feat, n, out, leaf_idx, st, n_dev, fr);
        return launch3<SF_GBDT, 1, 1, kB, false, true>(fo, p, feat, n, out, leaf_idx, st, n_dev, fr);
    }
    if (p.nch == 4) return launch3<SF_GBDT, 1, 4>(fo, p, feat, n, out, leaf_idx, st, n_dev, fr);
    if (p.nch == 2) return launch3<SF_GBDT, 1, 2>(fo, p, feat, n, out, leaf_idx, st, n_dev, fr);
    return launch3<SF_GBDT, 1, 1>(fo, p, feat, n, out, leaf_idx, st, n_dev, fr);
}

template <int C>
int launch_mc(const sf_forest* fo, const float* feat, uint32_t n, float* out, uint16_t* leaf_idx, cudaStream_t st, const uint32_t* n_dev, const sf_fused_route& fr) {
    const Plan p = make_plan(fo);
    if (p.tpc == 0) return SF_ERR_UNSUPPORTED;           // one boosting round does not fit in a chunk
    return launch3<SF_GBDT_MC, C, (C >= 4 ? 4 : (C >= 2 ? 2 : 1))>(fo, p, feat, n, out, leaf_idx, st, n_dev, fr);
}

template <int G>
int launch_rf_leaf_index_g(const sf_forest* fo, const float* feat, uint32_t n, uint16_t* leaf_idx, cudaStream_t st, const uint32_t* n_dev,
                           const LeafIndexPackets& pk) {
    const size_t feat_bytes = (size_t)fo->F * kBSmall * sizeof(float);
    uint32_t buf = 65536u;
    uint32_t tpi = buf / fo->tree_stride;
    if (tpi == 0) return SF_ERR_UNSUPPORTED;
    if (tpi > 8) tpi = 8;                                  // more items rather than longer ones
    if (tpi > fo->T) tpi = fo->T;
    buf = tpi * fo->tree_stride;
    const size_t smem = buf + feat_bytes + 16;
    static size_t smem_set_dev[64] = {};
    size_t& smem_set = smem_set_dev[fo->ctx->device & 63];
    if (smem > smem_set) {
        SF_CUDA(cudaFuncSetAttribute(forest_leaf_index_kernel<2, G>, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)smem));
        smem_set = smem;
    }
    const uint32_t n_items = ((n + kBSmall - 1) / kBSmall) * ((fo->T + tpi - 1) / tpi);
    const uint32_t grid = std::min<uint32_t>(n_items, (uint32_t)fo->ctx->num_sms * 2u);
    SF_CUDA(sf_launch_chained(forest_leaf_index_kernel<2, G>, grid, kBSmall, smem, st, feat, n, fo->F, (const unsigned char*)fo->d_image_small, fo->T,
                              fo->depth, fo->tree_stride, tpi, buf, leaf_idx, fo->ctx->d_state, n_dev, pk));
    return SF_OK;
}

int launch_rf_leaf_index(const sf_forest* fo, const float* feat, uint32_t n, uint16_t* leaf_idx, cudaStream_t st, const uint32_t* n_dev) {
    return launch_rf_leaf_index_g<0>(fo, feat, n, leaf_idx, st, n_dev, LeafIndexPackets{});
}

// small batches of a random forest: leaf indices by (tile, tree slice) work items, then the ordered sums.
// leaf_idx doubles as the scratch between the two kernels.
int launch_rf_split(const sf_forest* fo, const float* feat, uint32_t n, float* out, uint16_t* leaf_idx, cudaStream_t st, const uint32_t* n_dev) {
    int rc = launch_rf_leaf_index(fo, feat, n, leaf_idx, st, n_dev);
    if (rc != SF_OK) return rc;
    const uint64_t threads = (uint64_t)n * fo->C;
    forest_leaf_sum_kernel<<<(uint32_t)((threads + 255) / 256), 256, 0, st>>>(leaf_idx, fo->d_leaf, n, fo->T, 1u << fo->depth, fo->C, out, n_dev);
    SF_LAUNCH_CHECK("forest_leaf_sum_kernel");
    return SF_OK;
}

}  // namespace

int sf_launch_forest_leaf_index(const sf_forest* fo, const float* feat, uint32_t n, uint16_t* leaf_idx, cudaStream_t st,
                                const uint32_t* n_dev) {
    if (n == 0) return SF_OK;
    if (fo->kind != SF_RF || !fo->d_image_small || !leaf_idx) return SF_ERR_UNSUPPORTED;
    return launch_rf_leaf_index(fo, feat, n, leaf_idx, st, n_dev);
}

// leaf indices of the flows whose packets are rows row_ids[0..n) of the planes pk, features computed inside the kernel
int sf_launch_forest_leaf_index_packets(const sf_forest* fo, const sf_packets* pk, uint32_t N, const uint32_t* row_ids, uint32_t n,
                                        uint16_t* leaf_idx, cudaStream_t st, const uint32_t* n_dev) {
    if (n == 0) return SF_OK;
    if (fo->kind != SF_RF || !fo->d_image_small || !leaf_idx) return SF_ERR_UNSUPPORTED;
    if (pk->n_valid || pk->pitch_pkts % 8 != 0 || ((uintptr_t)pk->size & 15) != 0 || ((uintptr_t)pk->iat_us & 15) != 0) return SF_ERR_UNSUPPORTED;
    if (fo->F % 8 != 0 || N < 1 || N > 32 || N > pk->pitch_pkts) return SF_ERR_UNSUPPORTED;
    const LeafIndexPackets lp{pk->size, pk->iat_us, pk->dir_bits, row_ids, pk->pitch_pkts, N};
    switch (fo->F / 8) {
    case 1: return launch_rf_leaf_index_g<1>(fo, nullptr, n, leaf_idx, st, n_dev, lp);
    case 2: return launch_rf_leaf_index_g<2>(fo, nullptr, n, leaf_idx, st, n_dev, lp);
    case 3: return launch_rf_leaf_index_g<3>(fo, nullptr, n, leaf_idx, st, n_dev, lp);
    case 4: return launch_rf_leaf_index_g<4>(fo, nullptr, n, leaf_idx, st, n_dev, lp);
    case 5: return launch_rf_leaf_index_g<5>(fo, nullptr, n, leaf_idx, st, n_dev, lp);
    case 6: return launch_rf_leaf_index_g<6>(fo, nullptr, n, leaf_idx, st, n_dev, lp);
    case 7: return launch_rf_leaf_index_g<7>(fo, nullptr, n, leaf_idx, st, n_dev, lp);
    case 8: return launch_rf_leaf_index_g<8>(fo, nullptr, n, leaf_idx, st, n_dev, lp);
    }
    return SF_ERR_UNSUPPORTED;
}

int sf_launch_forest(const sf_forest* fo, const float* feat, uint32_t n, float* out, uint16_t* leaf_idx, cudaStream_t st, const uint32_t* n_dev,
                     bool small_tiles, const sf_fused_route* fused) {
    if (n == 0) return SF_OK;
    sf_fused_route fr;
    memset(&fr, 0, sizeof(fr));
    if (fused) {
        if (fo->kind == SF_GBDT_MC || small_tiles || kB != SF_FOREST_BLOCK) return SF_ERR_UNSUPPORTED;
        fr = *fused;
    }
    if (small_tiles && leaf_idx && fo->kind == SF_RF && fo->d_image_small) return launch_rf_split(fo, feat, n, out, leaf_idx, st, n_dev);
    if (fo->kind == SF_GBDT) return launch_gbdt(fo, feat, n, out, leaf_idx, st, n_dev, fr);
    if (fo->kind == SF_GBDT_MC) {
        switch (fo->C) {
        case 1:  return launch_mc<1>(fo, feat, n, out, leaf_idx, st, n_dev, fr);
        case 2:  return launch_mc<2>(fo, feat, n, out, leaf_idx, st, n_dev, fr);
        case 3:  return launch_mc<3>(fo, feat, n, out, leaf_idx, st, n_dev, fr);
        case 4:  return launch_mc<4>(fo, feat, n, out, leaf_idx, st, n_dev, fr);
        case 5:  return launch_mc<5>(fo, feat, n, out, leaf_idx, st, n_dev, fr);
        case 6:  return launch_mc<6>(fo, feat, n, out, leaf_idx, st, n_dev, fr);
        case 7:  return launch_mc<7>(fo, feat, n, out, leaf_idx, st, n_dev, fr);
        case 8:  return launch_mc<8>(fo, feat, n, out, leaf_idx, st, n_dev, fr);
        case 9:  return launch_mc<9>(fo, feat, n, out, leaf_idx, st, n_dev, fr);
        case 10: return launch_mc<10>(fo, feat, n, out, leaf_idx, st, n_dev, fr);
        case 11: return launch_mc<11>(fo, feat, n, out, leaf_idx, st, n_dev, fr);
        case 12: return launch_mc<12>(fo, feat, n, out, leaf_idx, st, n_dev, fr);
        case 13: return launch_mc<13>(fo, feat, n, out, leaf_idx, st, n_dev, fr);
        case 14: return launch_mc<14>(fo, feat, n, out, leaf_idx, st, n_dev, fr);
        case 15: return launch_mc<15>(fo, feat, n, out, leaf_idx, st, n_dev, fr);
        case 16: return launch_mc<16>(fo, feat, n, out, leaf_idx, st, n_dev, fr);
        }
        return SF_ERR_UNSUPPORTED;
    }
    switch (fo->C) {
    case 1:  return launch_rf<1>(fo, feat, n, out, leaf_idx, st, n_dev, fr);
    case 2:  return launch_rf<2>(fo, feat, n, out, leaf_idx, st, n_dev, fr);
    case 3:  return launch_rf<3>(fo, feat, n, out, leaf_idx, st, n_dev, fr);
    case 4:  return launch_rf<4>(fo, feat, n, out, leaf_idx, st, n_dev, fr);
    case 5:  return launch_rf<5>(fo, feat, n, out, leaf_idx, st, n_dev, fr);
    case 6:  return launch_rf<6>(fo, feat, n, out, leaf_idx, st, n_dev, fr);
    case 7:  return launch_rf<7>(fo, feat, n, out, leaf_idx, st, n_dev, fr);
    case 8:  return launch_rf<8>(fo, feat, n, out, leaf_idx, st, n_dev, fr);
    case 9:  return launch_rf<9>(fo, feat, n, out, leaf_idx, st, n_dev, fr);
    case 10: return launch_rf<10>(fo, feat, n, out, leaf_idx, st, n_dev, fr);
    case 11: return launch_rf<11>(fo, feat, n, out, leaf_idx, st, n_dev, fr);
    case 12: return launch_rf<12>(fo, feat, n, out, leaf_idx, st, n_dev, fr);
    case 13: return launch_rf<13>(fo, feat, n, out, leaf_idx, st, n_dev, fr);
    case 14: return launch_rf<14>(fo, feat, n, out, leaf_idx, st, n_dev, fr);
    case 15: return launch_rf<15>(fo, feat, n, out, leaf_idx, st, n_dev, fr);
    case 16: return launch_rf<16>(fo, feat, n, out, leaf_idx, st, n_dev, fr);
    }
    return SF_ERR_UNSUPPORTED;
}

extern "C" int sf_forest_create(sf_ctx* ctx, int kind, uint32_t T, uint32_t depth, uint32_t F, uint32_t C,
                                const uint16_t* fid, const float* thr, const float* leaf, sf_forest** out)
{
    if (!ctx || !fid || !thr || !leaf || !out) return SF_ERR_ARG;
    if (kind != SF_RF && kind != SF_GBDT && kind != SF_GBDT_MC) return SF_ERR_ARG;
    if (T < 1 || depth < 1 || depth > 12 || F < 1 || F > 64) return SF_ERR_ARG;
    if (kind != SF_GBDT && (C < 1 || C > 16)) return SF_ERR_ARG;
    if (kind == SF_GBDT_MC && T % C != 0) return SF_ERR_ARG;
    SF_CUDA(cudaSetDevice(ctx->device));
    const uint32_t n_int = (1u << depth) - 1u, n_ent = 1u << depth;
    for (size_t i = 0; i < (size_t)T * n_int; i++) if (fid[i] >= F) return SF_ERR_ARG;
    sf_forest* fo = new (std::nothrow) sf_forest();
    if (!fo) return SF_ERR_ALLOC;
    fo->ctx = ctx; fo->kind = kind; fo->T = T; fo->depth = depth; fo->F = F; fo->C = (kind == SF_GBDT) ? 1 : C;
    fo->d_image = nullptr; fo->d_leaf = nullptr; fo->d_image_small = nullptr; fo->leaf_tex = 0;
    fo->h_top = new (std::nothrow) ForestTop();
    if (!fo->h_top) { delete fo; return SF_ERR_ALLOC; }
    memset(fo->h_top, 0, sizeof(ForestTop));
    fo->top_ok = kind == SF_GBDT && depth >= 2 && T <= kTopMaxTrees;      // (random forests: measured, no gain at depth 10 to 12)
    // Image of one tree: 2^d node entries of 8 bytes in a 1-based heap (host node i, children
    // 2i+1 / 2i+2, becomes entry i+1, children 2j / 2j+1; entry 0 unused), then for boosted
    // trees the 2^d leaf scalars; padded to a multiple of 16 bytes for the 16-byte copies.
    uint32_t stride = n_ent * 8u + (kind != SF_RF ? n_ent * 4u : 0u);
    stride = (stride + 15u) & ~15u;
    fo->tree_stride = stride;
    unsigned char* h = (unsigned char*)calloc((size_t)T, stride);
    if (!h) { sf_forest_destroy(fo); return SF_ERR_ALLOC; }
    for (uint32_t t = 0; t < T; t++) {
        uint32_t* ent = reinterpret_cast<uint32_t*>(h + (size_t)t * stride);
        for (uint32_t i = 0; i < n_int; i++) {
            uint32_t bits; float v = thr[(size_t)t * n_int + i];
            memcpy(&bits, &v, 4);
            ent[2 * (i + 1)] = bits;
            ent[2 * (i + 1) + 1] = (uint32_t)fid[(size_t)t * n_int + i] * kB * 4u;     // byte offset of the feature's row
        }
        if (kind != SF_RF) memcpy(h + (size_t)t * stride + n_ent * 8u, leaf + (size_t)t * n_ent, n_ent * 4u);
        if (fo->top_ok)
            for (uint32_t i = 0; i < 3; i++) fo->h_top->n[t][i] = make_uint2(ent[2 * (i + 1)], ent[2 * (i + 1) + 1]);
    }
    // the small-batch variant of the kernel has a narrower feature tile, so its feature offsets differ
    unsigned char* h_small = nullptr;
    if (kind == SF_RF) {
        h_small = (unsigned char*)malloc((size_t)T * stride);
        if (!h_small) { free(h); sf_forest_destroy(fo); return SF_ERR_ALLOC; }
        memcpy(h_small, h, (size_t)T * stride);
        for (uint32_t t = 0; t < T; t++) {
            uint32_t* ent = reinterpret_cast<uint32_t*>(h_small + (size_t)t * stride);
            for (uint32_t i = 0; i < n_int; i++) ent[2 * (i + 1) + 1] = (uint32_t)fid[(size_t)t * n_int + i] * kBSmall * 4u;
        }
    }
    const size_t leaf_count = (size_t)T * n_ent * (kind == SF_RF ? fo->C : 1u);
    cudaError_t e = cudaMalloc(&fo->d_image, (size_t)T * stride);
    if (e == cudaSuccess) e = cudaMalloc(&fo->d_leaf, sizeof(float) * leaf_count);
    if (e == cudaSuccess) e = cudaMemcpy(fo->d_image, h, (size_t)T * stride, cudaMemcpyHostToDevice);
    if (e == cudaSuccess && h_small) e = cudaMalloc(&fo->d_image_small, (size_t)T * stride);
    if (e == cudaSuccess && h_small) e = cudaMemcpy(fo->d_image_small, h_small, (size_t)T * stride, cudaMemcpyHostToDevice);
    if (e == cudaSuccess) e = cudaMemcpy(fo->d_leaf, leaf, sizeof(float) * leaf_count, cudaMemcpyHostToDevice);
    free(h); free(h_small);
    if (e != cudaSuccess) { sf_forest_destroy(fo); return sf_set_cuda_error(e, "sf_forest_create"); }
    if (kind == SF_RF && (fo->C % 4) == 0) {
        // texture view of the leaf table (16-byte integer texels); where it cannot be made (table beyond the
        // linear-texture limit, base not aligned for textures) the kernel gathers through plain loads
        cudaDeviceProp prop;
        if (cudaGetDeviceProperties(&prop, ctx->device) == cudaSuccess && leaf_count / 4 <= (size_t)prop.maxTexture1DLinear &&
            ((uintptr_t)fo->d_leaf % prop.textureAlignment) == 0) {
            cudaResourceDesc rd; memset(&rd, 0, sizeof(rd));
            rd.resType = cudaResourceTypeLinear;
            rd.res.linear.devPtr = fo->d_leaf;
            rd.res.linear.desc = cudaCreateChannelDesc<uint4>();
            rd.res.linear.sizeInBytes = sizeof(float) * leaf_count;
            cudaTextureDesc td; memset(&td, 0, sizeof(td));
            td.readMode = cudaReadModeElementType;
            cudaTextureObject_t tex = 0;
            if (cudaCreateTextureObject(&tex, &rd, &td, nullptr) == cudaSuccess) fo->leaf_tex = tex;
            else (void)cudaGetLastError();
        }
    }
    *out = fo;
    return SF_OK;
}

extern "C" void sf_forest_destroy(sf_forest* fo) {
    if (!fo) return;
    if (fo->leaf_tex) cudaDestroyTextureObject(fo->leaf_tex);
    if (fo->d_image) cudaFree(fo->d_image);
    if (fo->d_image_small) cudaFree(fo->d_image_small);
    if (fo->d_leaf) cudaFree(fo->d_leaf);
    delete fo->h_top;
    delete fo;
}

extern "C" int sf_fast_infer(sf_ctx* ctx, const sf_forest* fo, const float* feat, uint32_t n,
                             float* out, uint16_t* leaf_idx_out, void* stream)
{
    if (!ctx || !fo || !feat || !out) return SF_ERR_ARG;
    if (((uintptr_t)feat & 15) != 0) return SF_ERR_ARG;
    SF_CUDA(cudaSetDevice(ctx->device));
    sf_time_new_record(ctx);
    sf_time_begin(ctx, SF_T_FOREST, (cudaStream_t)stream);
    int rc = sf_launch_forest(fo, feat, n, out, leaf_idx_out, (cudaStream_t)stream);
    sf_time_end(ctx, SF_T_FOREST, (cudaStream_t)stream);
    return rc;
}

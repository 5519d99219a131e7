// S4 (bf16 MLP): hidden layers as tcgen05 GEMMs with TMEM accumulators fed by
// TMA.  The narrow last layer (<= 16 classes) is folded into the epilogue of the last hidden layer where the
// batch is large (a CTA then owns whole 128-row panels, its epilogue warps multiply the bf16-rounded activations
// of every tile with the head's weights on the CUDA cores and the activations are never written); otherwise it
// runs through the same kernel as a 128 x 16 tile of its own.
//
// Hidden layer: out[r][o] = bf16( ReLU( sum_k A[r][k] * W[o][k] + b[o] ) ), r < *n_rows.
// Persistent kernel, one CTA per SM, tile 128 x BN, K slices of 64 bf16 (one 128-byte
// swizzled row per matrix row).  Warp roles:
//   warp 0      TMA producer: loads the A and W slices of a ring of stages
//   warp 1      allocates TMEM; one lane issues tcgen05.mma (4 per stage, K = 16 each)
//   warps 2..9  epilogue: tcgen05.ld the fp32 accumulators (TMEM lane quarter = warp % 4,
//               column half = (warp - 2) / 4), add bias, ReLU, round to bf16, transpose each
//               32 x 32 block through shared memory so that global stores are whole 64-byte
//               row segments (8 rows per instruction)
// Two accumulator buffers in TMEM (2 x BN columns) let the MMAs of tile i+1 overlap
// the epilogue of tile i.  Large batches of 256-column layers run the same kernel on CTA pairs (clusters of two, one
// tcgen05.mma.cta_group::2 per K step for a 256 x 256 tile): a third less operand traffic per flop, which is what counts
// on a part whose tensor pipe is power-limited.  The row count lives in device memory, so routing and the
// slow model need no host round trip; tiles past the count are never scheduled and
// rows past it are never stored.  Every barrier wait is bounded: on a timeout the
// block records SF_ERR_DEVICE_TIMEOUT, lets its copies land, frees TMEM and returns.
#include "tc_common.cuh"

namespace sftc {

int encode_tmap_bf16_2d(CUtensorMap* out, const void* base, uint64_t rows, uint64_t cols,
                        uint32_t box_rows, uint32_t box_cols)
{
    typedef CUresult (*encode_fn)(CUtensorMap*, CUtensorMapDataType, cuuint32_t, void*, const cuuint64_t*,
                                  const cuuint64_t*, const cuuint32_t*, const cuuint32_t*, CUtensorMapInterleave,
                                  CUtensorMapSwizzle, CUtensorMapL2promotion, CUtensorMapFloatOOBfill);
    static encode_fn fn = nullptr;
    if (!fn) {
        void* p = nullptr;
        cudaDriverEntryPointQueryResult q;
        cudaError_t e = cudaGetDriverEntryPoint("cuTensorMapEncodeTiled", &p, cudaEnableDefault, &q);
        if (e != cudaSuccess || q != cudaDriverEntryPointSuccess || !p) return sf_set_cuda_error(e != cudaSuccess ? e : cudaErrorUnknown, "cudaGetDriverEntryPoint(cuTensorMapEncodeTiled)");
        fn = (encode_fn)p;
    }
    cuuint64_t gdim[2] = {cols, rows};
    cuuint64_t gstride[1] = {cols * 2};
    cuuint32_t box[2] = {box_cols, box_rows};
    cuuint32_t estr[2] = {1, 1};
    CUresult r = fn(out, CU_TENSOR_MAP_DATA_TYPE_BFLOAT16, 2, const_cast<void*>(base), gdim, gstride, box, estr,
                    CU_TENSOR_MAP_INTERLEAVE_NONE, CU_TENSOR_MAP_SWIZZLE_128B, CU_TENSOR_MAP_L2_PROMOTION_L2_256B,
                    CU_TENSOR_MAP_FLOAT_OOB_FILL_NONE);
    if (r != CUDA_SUCCESS) return sf_set_cuda_error(cudaErrorInvalidValue, "cuTensorMapEncodeTiled");
    return SF_OK;
}

}  // namespace sftc

namespace {
using namespace sftc;

constexpr uint32_t BM = 128;
constexpr uint32_t BK = 64;
constexpr uint32_t kEpiWarps = 8;
constexpr uint32_t kGemmThreads = 64 + kEpiWarps * 32;

// PAIR: two CTAs (a cluster of two, on the two SMs of one TPC) share every MMA: the tile is 256 rows x BN, each CTA loads its
// 128 rows of A and its BN / 2 rows of W per stage (a third less shared-memory and L2 traffic per flop, two more stages)
template <uint32_t BN, bool PAIR = false> struct GemmCfg {
    static constexpr uint32_t kStageBytesA = BM * BK * 2;
    static constexpr uint32_t kStageBytesB = (PAIR ? BN / 2 : BN) * BK * 2;
    static constexpr uint32_t kStageBytes = kStageBytesA + kStageBytesB;
    static constexpr uint32_t kStages = PAIR ? 6 : ((BN == 256) ? 4 : (BN == 128 ? 6 : (BN == 64 ? 8 : 10)));
    static constexpr uint32_t kTmemCols = 2 * BN;             // a power of two >= 32
    static constexpr uint32_t kSmemBytes = kStages * kStageBytes + 1024 /*alignment slack*/ + 256 /*barriers*/ +
                                           kEpiWarps * 2048 /*epilogue staging*/;
    // fused head: the head's weights (N <= 1024 columns x 32 bytes) take the staging space and 16 KB more
    static constexpr uint32_t kSmemBytesHead16 = kSmemBytes + 16384;
};

constexpr uint32_t kFusedHeadMaxN = 1024;
enum { MODE_HIDDEN = 0, MODE_HEAD = 1, MODE_HIDDEN_HEAD = 2 };

struct GemmBars {
    uint64_t full[10];
    uint64_t empty[10];
    uint64_t tmem_full[2];
    uint64_t tmem_empty[2];
    uint64_t head_bar;            // fused head: the four high-half epilogue warps have stored their partial logits
    uint32_t tmem_base;
    uint32_t abort_flag;
};

// ---- a handful of rows (the streaming path: about ten flows reach the slow model per batch) --------------------
// A 128-row tensor-core tile would be almost empty and its K loop (K/16 dependent MMAs on one SM) takes 8 us per layer
// whatever the row count.  Up to kSmallRows rows are served by the same kernel on CUDA cores instead (the row count is
// only known on the device, so the choice is made there, at the top of the kernel): a warp per output column, lanes
// over K (8 consecutive inputs each per step), the rows' activations staged in shared memory, fp32 accumulation, a
// fixed shuffle tree over the lanes (deterministic), then bias (+ ReLU + bf16, or the logits and the argmax).
constexpr uint32_t kSmallRows = 16;
constexpr uint32_t kSmallMaxK = 4096;                // 16 rows x K bf16 must fit in the kernel's tile ring (>= 180 KB)

__device__ __forceinline__ float warp_rows_reduce16(float (&v)[16], uint32_t lane) {
#pragma unroll
    for (int j = 0; j < 16; j++) v[j] += __shfl_xor_sync(0xFFFFFFFFu, v[j], 16);
#pragma unroll
    for (int off = 8; off >= 1; off >>= 1) {
        const bool up = (lane & off) != 0;
#pragma unroll
        for (int j = 0; j < off; j++) {
            const float keep = up ? v[j + off] : v[j];
            const float send = up ? v[j] : v[j + off];
            v[j] = keep + __shfl_xor_sync(0xFFFFFFFFu, send, off);
        }
    }
    return v[0];                                     // lanes l and l + 16: total of row l & 15
}

// HEAD = false: out[r][n] = bf16(ReLU(sum + bias[n])), columns spread over all warps of the grid.
// HEAD = true (one block: block 0, or whichever block calls it with ANY_BLOCK; W padded to 16 rows): logits[r][c] = sum + bias[c]
// for c < C, label[r] = argmax (lowest index on ties).
template <bool HEAD, bool ANY_BLOCK = false>
__device__ void small_rows_layer(const __nv_bfloat16* __restrict__ A, const __nv_bfloat16* __restrict__ W, const float* __restrict__ bias,
                                 uint32_t rows, uint32_t N, uint32_t K, __nv_bfloat16* __restrict__ out,
                                 float* __restrict__ logits, uint8_t* __restrict__ label, uint32_t C, uint8_t* smem)
{
    __shared__ float lg[kSmallRows][16];
    if (HEAD && !ANY_BLOCK && blockIdx.x != 0) return;
    uint4* As = reinterpret_cast<uint4*>(smem);                           // [16 rows][K] bf16, rows past the count zero
    const uint32_t k16 = K / 8;                                           // 16-byte chunks per row
    const uint32_t warp = threadIdx.x >> 5, lane = threadIdx.x & 31, wpb = blockDim.x >> 5;
    const uint32_t n_cols = HEAD ? 16u : N;
    const uint32_t w0 = HEAD ? warp : blockIdx.x * wpb + warp, wstep = HEAD ? wpb : gridDim.x * wpb;
    // A lane holds kPF 16-byte pieces of a weight row at a time (K up to 2048 in one go): the loads are all in flight before the
    // first is used, so a column costs one trip to L2 instead of one per piece.  The first column's pieces are asked for before
    // the activations are staged, and travel meanwhile.
    constexpr int kPF = 8;
    uint4 wv[kPF];
    auto fetch = [&](uint32_t n, uint32_t c0) {
        const uint4* wrow = reinterpret_cast<const uint4*>(W + (size_t)n * K);
#pragma unroll
        for (int j = 0; j < kPF; j++) {
            const uint32_t c = c0 + lane + 32u * j;
            wv[j] = (c < k16) ? __ldg(wrow + c) : make_uint4(0, 0, 0, 0);
        }
    };
    if (w0 < n_cols) fetch(w0, 0);
    for (uint32_t i = threadIdx.x; i < kSmallRows * k16; i += blockDim.x) {
        const uint32_t r = i / k16, c = i - r * k16;
        // (from L2: with the head in the same launch these activations were written by other blocks a moment ago)
        As[i] = (r < rows) ? __ldcg(reinterpret_cast<const uint4*>(A + (size_t)r * K) + c) : make_uint4(0, 0, 0, 0);
    }
    __syncthreads();
    for (uint32_t n = w0; n < n_cols; n += wstep) {
        float acc[kSmallRows];
#pragma unroll
        for (int r = 0; r < (int)kSmallRows; r++) acc[r] = 0.0f;
        for (uint32_t c0 = 0; c0 < k16; c0 += 32u * kPF) {
            if (n != w0 || c0 != 0) fetch(n, c0);
#pragma unroll
            for (int j = 0; j < kPF; j++) {
                const uint32_t c = c0 + lane + 32u * j;
                if (c < k16) {
                    const uint32_t wq[4] = {wv[j].x, wv[j].y, wv[j].z, wv[j].w};
#pragma unroll
                    for (int r = 0; r < (int)kSmallRows; r++) {
                        const uint4 av = As[r * k16 + c];
                        const uint32_t aq[4] = {av.x, av.y, av.z, av.w};
#pragma unroll
                        for (int e = 0; e < 4; e++) {
                            acc[r] = fmaf(__uint_as_float(aq[e] << 16), __uint_as_float(wq[e] << 16), acc[r]);
                            acc[r] = fmaf(__uint_as_float(aq[e] & 0xFFFF0000u), __uint_as_float(wq[e] & 0xFFFF0000u), acc[r]);
                        }
                    }
                }
            }
        }
        const float tot = warp_rows_reduce16(acc, lane);
        const uint32_t r = lane & 15u;
        if (!HEAD) {
            if (lane < 16 && r < rows) out[(size_t)r * N + n] = __float2bfloat16_rn(fmaxf(tot + bias[n], 0.0f));
        } else if (lane < 16) {
            lg[r][n] = (n < C) ? tot + bias[n] : -3.0e38f;
        }
    }
    if (HEAD) {
        __syncthreads();
        if (threadIdx.x < rows) {
            float best = lg[threadIdx.x][0]; uint32_t arg = 0;
            for (uint32_t c = 0; c < C; c++) {
                const float v = lg[threadIdx.x][c];
                logits[(size_t)threadIdx.x * C + c] = v;
                if (v > best) { best = v; arg = c; }
            }
            if (label) label[threadIdx.x] = (uint8_t)arg;
        }
    }
}

// (d0, d1) += a * (w0, w1): two IEEE fp32 fused multiply-adds in one instruction
__device__ __forceinline__ void fma_pair(float& d0, float& d1, float a, float w0, float w1) {
    uint64_t d, aa, ww;
    asm("mov.b64 %0, {%1, %2};" : "=l"(d) : "f"(d0), "f"(d1));
    asm("mov.b64 %0, {%1, %1};" : "=l"(aa) : "f"(a));
    asm("mov.b64 %0, {%1, %2};" : "=l"(ww) : "f"(w0), "f"(w1));
    asm("fma.rn.f32x2 %0, %1, %2, %0;" : "+l"(d) : "l"(aa), "l"(ww));
    asm("mov.b64 {%0, %1}, %2;" : "=f"(d0), "=f"(d1) : "l"(d));
}

// bf16x2( ReLU(v0 + b0), ReLU(v1 + b1) ), first value in the low half: the conversion clamps at zero itself
__device__ __forceinline__ uint32_t bias_relu_bf16x2(uint32_t v0, uint32_t v1, float b0, float b1) {
    const float x0 = __uint_as_float(v0) + b0, x1 = __uint_as_float(v1) + b1;
    uint32_t h;
    asm("cvt.rn.relu.bf16x2.f32 %0, %1, %2;" : "=r"(h) : "f"(x1), "f"(x0));
    return h;
}

// HEAD = false: hidden layer, out = bf16(ReLU(acc + bias)) [rows][N].
// HEAD = true (BN = 16): last layer, W zero-padded to 16 rows; logits[r][c] = acc + bias for
// c < C (fp32, no activation) and label[r] = argmax (lowest index on ties).
// MODE_HIDDEN_HEAD: the last hidden layer with the head folded in.  head_w = the head's weights bf16 [16][N] (rows past C
// zero), head_b its bias, CH = 2, 4, 8 or 16 = classes kept per row.  A CTA takes whole 128-row panels (all N / BN tiles of
// a panel in turn), so a row's logits are summed in one place and in one fixed order: column chunks in increasing
// order inside each of the two epilogue warps that share the row, then (low half + high half) + bias.
//
// PAIR (launched as clusters of two CTAs, BN = 256): CTA rank 0 of a pair is the leader.  Both producers wait on their own
// `empty` barriers and load into their own shared memory, the bytes of both counted on the LEADER's `full` barrier; one thread
// of the leader issues the pair MMAs and commits to `empty` and `tmem_full` in both CTAs; each CTA's epilogue warps read their
// own TMEM (rows rank * 128 ... of the 256-row tile) and release the accumulator on the leader's `tmem_empty`.  No CTA leaves
// while its partner may still touch its shared memory: the producers first see every stage released, then the pair meets
// at a cluster barrier that every thread reaches (all waits before it are bounded).
template <uint32_t BN, int MODE, uint32_t CH = 8, bool PAIR = false>
__global__ void __launch_bounds__(kGemmThreads, 1)
gemm_bias_relu_bf16_kernel(const __grid_constant__ CUtensorMap tmA, const __grid_constant__ CUtensorMap tmW,
                           const float* __restrict__ bias, const uint32_t* __restrict__ n_rows_dev,
                           uint32_t N, uint32_t K, __nv_bfloat16* __restrict__ out, sf_dev_state* st,
                           float* __restrict__ logits, uint8_t* __restrict__ label, uint32_t C, uint32_t small_max,
                           const __nv_bfloat16* __restrict__ A_raw, const __nv_bfloat16* __restrict__ W_raw, uint32_t capacity,
                           const __nv_bfloat16* __restrict__ head_w, const float* __restrict__ head_b)
{
    using Cfg = GemmCfg<BN, PAIR>;
    constexpr bool HEAD = MODE == MODE_HEAD;
    constexpr bool FUSED = MODE == MODE_HIDDEN_HEAD;
    static_assert(!PAIR || (BN == 256 && !HEAD), "pairs: 256-column tiles of a hidden layer");
    constexpr uint32_t BMT = PAIR ? 2 * BM : BM;       // rows of a tile
    extern __shared__ uint8_t smem_raw[];
    sf_chain_enter();
    // the count is the caller's device word: never trust it beyond the rows the buffers hold
    const uint32_t n_rows = sf_clamp_rows(*n_rows_dev, capacity, st);
    if (n_rows <= small_max) {                       // a handful of rows (small_max = 0: never): CUDA cores, same launch (pairs: both CTAs alike)
        if constexpr (FUSED) {
            // hidden layer into the caller's 16-row scratch (`out`), then the head by whichever block stores its columns last:
            // nobody waits for anybody (an arrival counter in device memory; the last block puts it back to zero)
            __shared__ uint32_t is_last;
            if (n_rows) {
                small_rows_layer<false>(A_raw, W_raw, bias, n_rows, N, K, out, nullptr, nullptr, 0, smem_raw);
                __syncthreads();
                if (threadIdx.x == 0) {
                    __threadfence();
                    is_last = (atomicAdd(&st->blocks_done, 1u) == gridDim.x - 1u) ? 1u : 0u;
                }
                __syncthreads();
                if (is_last) {
                    if (threadIdx.x == 0) st->blocks_done = 0;
                    __threadfence();
                    small_rows_layer<true, true>(out, head_w, head_b, n_rows, 16, N, nullptr, logits, label, C, smem_raw);
                }
            }
        } else {
            if (n_rows) small_rows_layer<HEAD>(A_raw, W_raw, bias, n_rows, N, K, out, logits, label, C, smem_raw);
        }
        return;
    }
    const uint32_t base_u32 = (smem_u32(smem_raw) + 1023u) & ~1023u;
    uint8_t* tiles = smem_raw + (base_u32 - smem_u32(smem_raw));
    GemmBars* bars = reinterpret_cast<GemmBars*>(tiles + Cfg::kStages * Cfg::kStageBytes);
    volatile uint32_t* abort_flag = &bars->abort_flag;

    const uint32_t warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
    const uint32_t tiles_m = (n_rows + BMT - 1) / BMT;
    const uint32_t tiles_n = N / BN;
    const uint32_t k_blocks = K / BK;
    const uint32_t rank = PAIR ? cluster_ctarank() : 0u;                   // 0 = the pair's leader
    const uint32_t unit = PAIR ? blockIdx.x >> 1 : blockIdx.x;             // this CTA's (pair's) place among ...
    const uint32_t n_units = PAIR ? gridDim.x >> 1 : gridDim.x;            // ... the CTAs (pairs) that share the tiles
    // tiles of this CTA, in order: every gridDim.x-th tile of the (row panel, column tile) sequence, or - with the head
    // folded in - every gridDim.x-th row panel with all its column tiles
    const uint32_t n_my = FUSED ? ((tiles_m > unit) ? ((tiles_m - unit + n_units - 1) / n_units) * tiles_n : 0u)
                                : ((tiles_m * tiles_n > unit) ? (tiles_m * tiles_n - unit + n_units - 1) / n_units : 0u);
    auto tile_of = [&](uint32_t it, uint32_t& tm, uint32_t& tn) {
        if (FUSED) { tm = unit + (it / tiles_n) * n_units; tn = it % tiles_n; }
        else { const uint32_t tile = unit + it * n_units; tm = tile / tiles_n; tn = tile - tm * tiles_n; }
    };

    if (threadIdx.x == 0) {
        for (uint32_t s = 0; s < Cfg::kStages; s++) { mbar_init(&bars->full[s], 1); mbar_init(&bars->empty[s], 1); }
        for (uint32_t b = 0; b < 2; b++) { mbar_init(&bars->tmem_full[b], 1); mbar_init(&bars->tmem_empty[b], PAIR ? 2 * kEpiWarps : kEpiWarps); }
        mbar_init(&bars->head_bar, kEpiWarps / 2);
        bars->abort_flag = 0;
        fence_barrier_init();
    }
    if (warp == 1) { if constexpr (PAIR) tmem_alloc_pair(&bars->tmem_base, Cfg::kTmemCols); else tmem_alloc(&bars->tmem_base, Cfg::kTmemCols); }
    // fused head: the head's weights, transposed to [column][CH] bf16, where the other modes stage their output
    uint8_t* const epi_smem = tiles + Cfg::kStages * Cfg::kStageBytes + 256;
    if constexpr (FUSED) {
        // CH = 2, 4 or 8 classes kept: fp32 [column][CH] (the bf16 values widened once here instead of once per row in the
        // epilogue, whose integer pipe is the busy one); 16: bf16 [column][16]; at most 32 KB
        for (uint32_t i = threadIdx.x; i < N * CH; i += kGemmThreads) {
            const uint32_t col = i / CH, c = i - col * CH;
            const __nv_bfloat16 w = head_w[(size_t)c * N + col];                // rows past C are zero in the padded head matrix
            if (CH <= 8) reinterpret_cast<float*>(epi_smem)[i] = __bfloat162float(w);
            else reinterpret_cast<__nv_bfloat16*>(epi_smem)[i] = w;
        }
    }
    tc_fence_before();
    __syncthreads();
    if constexpr (PAIR) cluster_sync_all();          // the partner's barriers are initialised before anything reaches them
    tc_fence_after();
    const uint32_t tmem_base = bars->tmem_base;

    if (warp == 0) {
        if (lane == 0) {
            tma_prefetch_desc(&tmA);
            tma_prefetch_desc(&tmW);
            uint32_t stage = 0, phase = 0;
            bool ok = true;
            for (uint32_t it = 0; it < n_my && ok; it++) {
                uint32_t tm, tn;
                tile_of(it, tm, tn);
                for (uint32_t kb = 0; kb < k_blocks; kb++) {
                    if (!mbar_wait(&bars->empty[stage], phase ^ 1u, abort_flag)) { ok = false; break; }
                    uint8_t* sA = tiles + stage * Cfg::kStageBytes;
                    uint8_t* sB = sA + Cfg::kStageBytesA;
                    if constexpr (PAIR) {
                        const uint32_t full_leader = map_to_cta(smem_u32(&bars->full[stage]), 0);
                        if (rank == 0) mbar_expect_tx(&bars->full[stage], 2 * Cfg::kStageBytes);
                        tma_load_2d_pair(sA, &tmA, (int32_t)(kb * BK), (int32_t)(tm * BMT + rank * BM), full_leader);
                        tma_load_2d_pair(sB, &tmW, (int32_t)(kb * BK), (int32_t)(tn * BN + rank * (BN / 2)), full_leader);
                    } else {
                        mbar_expect_tx(&bars->full[stage], Cfg::kStageBytes);
                        tma_load_2d(sA, &tmA, (int32_t)(kb * BK), (int32_t)(tm * BM), &bars->full[stage]);
                        tma_load_2d(sB, &tmW, (int32_t)(kb * BK), (int32_t)(tn * BN), &bars->full[stage]);
                    }
                    if (++stage == Cfg::kStages) { stage = 0; phase ^= 1u; }
                }
            }
            if constexpr (PAIR) {
                // every stage's last use released: no arrival from the leader is still on its way to this CTA's barriers
                for (uint32_t s = 0; s < Cfg::kStages && ok; s++) {
                    if (!mbar_wait(&bars->empty[stage], phase ^ 1u, abort_flag)) ok = false;
                    if (++stage == Cfg::kStages) { stage = 0; phase ^= 1u; }
                }
            }
        }
    } else if (warp == 1) {
        if (lane == 0 && rank == 0) {
            constexpr uint32_t idesc = make_idesc_bf16(BMT, BN);
            uint32_t stage = 0, phase = 0, buf = 0, bphase = 0;
            bool ok = true;
            for (uint32_t it = 0; it < n_my && ok; it++) {
                if (!mbar_wait(&bars->tmem_empty[buf], bphase ^ 1u, abort_flag)) { ok = false; break; }
                tc_fence_after();
                const uint32_t d_tmem = tmem_base + buf * BN;
                for (uint32_t kb = 0; kb < k_blocks; kb++) {
                    if (!mbar_wait(&bars->full[stage], phase, abort_flag)) { ok = false; break; }
                    tc_fence_after();
                    const uint32_t aaddr = base_u32 + stage * Cfg::kStageBytes;
                    const uint32_t baddr = aaddr + Cfg::kStageBytesA;
#pragma unroll
                    for (uint32_t k = 0; k < BK / 16; k++) {
                        // 16 bf16 = 32 bytes further along K inside the 128-byte swizzled row
                        const uint64_t adesc = make_smem_desc(aaddr + k * 32u, 16, 1024, 2);
                        const uint64_t bdesc = make_smem_desc(baddr + k * 32u, 16, 1024, 2);
                        if constexpr (PAIR) umma_bf16_pair(d_tmem, adesc, bdesc, idesc, (kb | k) != 0 ? 1u : 0u);
                        else umma_bf16(d_tmem, adesc, bdesc, idesc, (kb | k) != 0 ? 1u : 0u);
                    }
                    // stage reusable once these MMAs retire
                    if constexpr (PAIR) umma_commit_pair(&bars->empty[stage]); else umma_commit(&bars->empty[stage]);
                    if (++stage == Cfg::kStages) { stage = 0; phase ^= 1u; }
                }
                if (!ok) break;
                // accumulator complete
                if constexpr (PAIR) umma_commit_pair(&bars->tmem_full[buf]); else umma_commit(&bars->tmem_full[buf]);
                buf ^= 1u; if (buf == 0) bphase ^= 1u;
            }
        }
    } else {
        // 8 epilogue warps: TMEM lane quarter = warp % 4, column half = (warp - 2) / 4
        const uint32_t quarter = warp & 3u;
        const uint32_t half = (warp - 2u) >> 2;
        uint8_t* stg = epi_smem + (warp - 2u) * 2048u;   // 32 rows x 64 B, XOR-swizzled
        uint32_t buf = 0, bphase = 0, hphase = 0;
        bool ok = true;
        float lg[CH];                                     // fused head: this thread's row, partial logits over this warp's columns
        for (uint32_t it = 0; it < n_my && ok; it++) {
            uint32_t tm, tn;
            tile_of(it, tm, tn);
            // the whole warp takes the same way out: the TMEM loads below are warp-collective
            ok = __all_sync(0xFFFFFFFFu, mbar_wait(&bars->tmem_full[buf], bphase, abort_flag));
            if (!ok) break;
            tc_fence_after();
            const uint32_t row0 = tm * BMT + rank * BM + quarter * 32u;
            const uint32_t col0 = tn * BN;
            const uint32_t taddr = tmem_base + ((quarter * 32u) << 16) + buf * BN;
            if constexpr (HEAD) {
                if (half == 0) {
                    const uint32_t row = row0 + lane;
                    uint32_t v[16];
                    tmem_ld16(taddr, v);
                    tmem_ld_wait();
                    if (row < n_rows) {
                        uint32_t a = 0; float mx = 0.0f;
#pragma unroll
                        for (int c = 0; c < 16; c++) {
                            if ((uint32_t)c < C) {
                                float x = __uint_as_float(v[c]) + __ldg(bias + c);
                                logits[(size_t)row * C + c] = x;
                                if (c == 0 || x > mx) { mx = x; a = c; }
                            }
                        }
                        if (label) label[row] = (uint8_t)a;
                    }
                }
            } else if constexpr (FUSED) {
                constexpr uint32_t kHalfCols = BN / 2;
                const uint32_t row = row0 + lane;
                if (tn == 0) {
#pragma unroll
                    for (uint32_t c = 0; c < CH; c++) lg[c] = 0.0f;
                }
#pragma unroll 1
                for (uint32_t c = half * kHalfCols; c < (half + 1) * kHalfCols; c += 32) {
                    uint32_t v[32];
                    tmem_ld32(taddr + c, v);
                    tmem_ld_wait();
                    const float4* b4 = reinterpret_cast<const float4*>(bias + col0 + c);
                    const uint8_t* wq = epi_smem + (size_t)(col0 + c) * (CH <= 8 ? CH * 4 : 32);     // this chunk's first column
#pragma unroll
                    for (int pc = 0; pc < 8; pc++) {
                        const float4 bv = __ldg(b4 + pc);
                        const float bb[4] = {bv.x, bv.y, bv.z, bv.w};
#pragma unroll
                        for (int e = 0; e < 4; e += 2) {
                            // bias + ReLU + bf16 rounding exactly as the stored activations would have had
                            const uint32_t hb = bias_relu_bf16x2(v[pc * 4 + e], v[pc * 4 + e + 1], bb[e], bb[e + 1]);
                            const float a[2] = {__uint_as_float(hb << 16), __uint_as_float(hb & 0xFFFF0000u)};
#pragma unroll
                            for (int q = 0; q < 2; q++) {
                                // this column's head weights: the same address in all lanes, a broadcast
                                if constexpr (CH == 16) {
                                    const uint4* wp = reinterpret_cast<const uint4*>(wq) + (size_t)(pc * 4 + e + q) * 2;
#pragma unroll
                                    for (uint32_t g = 0; g < 2; g++) {
                                        const uint4 w = wp[g];
                                        const uint32_t ww[4] = {w.x, w.y, w.z, w.w};
#pragma unroll
                                        for (int k = 0; k < 4; k++) {
                                            lg[g * 8 + 2 * k] = fmaf(a[q], __uint_as_float(ww[k] << 16), lg[g * 8 + 2 * k]);
                                            lg[g * 8 + 2 * k + 1] = fmaf(a[q], __uint_as_float(ww[k] & 0xFFFF0000u), lg[g * 8 + 2 * k + 1]);
                                        }
                                    }
                                } else {
                                    const float2* wp = reinterpret_cast<const float2*>(wq) + (size_t)(pc * 4 + e + q) * (CH / 2);
                                    if constexpr (CH == 2) {
                                        const float2 w = wp[0];
                                        lg[0] = fmaf(a[q], w.x, lg[0]); lg[1] = fmaf(a[q], w.y, lg[1]);
                                    } else {
#pragma unroll
                                        for (uint32_t g = 0; g < CH / 4; g++) {
                                            const float4 w = reinterpret_cast<const float4*>(wp)[g];
                                            fma_pair(lg[g * 4 + 0], lg[g * 4 + 1], a[q], w.x, w.y);
                                            fma_pair(lg[g * 4 + 2], lg[g * 4 + 3], a[q], w.z, w.w);
                                        }
                                    }
                                }
                            }
                        }
                    }
                }
                if (tn + 1 == tiles_n) {
                    // the row's two halves meet: the high-half warp leaves its partial sums in the logits row, the low-half warp
                    // adds (low + high) + bias, writes the logits and the label
                    if (half == 1) {
                        if (row < n_rows) {
#pragma unroll
                            for (uint32_t c = 0; c < CH; c++) if (c < C) logits[(size_t)row * C + c] = lg[c];
                        }
                        __syncwarp();
                        if (lane == 0) mbar_arrive(&bars->head_bar);
                    } else {
                        ok = __all_sync(0xFFFFFFFFu, mbar_wait(&bars->head_bar, hphase, abort_flag));
                        if (!ok) break;
                        hphase ^= 1u;
                        if (row < n_rows) {
                            uint32_t arg = 0; float mx = 0.0f;
#pragma unroll
                            for (uint32_t c = 0; c < CH; c++) {
                                if (c < C) {
                                    const float x = (lg[c] + logits[(size_t)row * C + c]) + __ldg(head_b + c);
                                    logits[(size_t)row * C + c] = x;
                                    if (c == 0 || x > mx) { mx = x; arg = c; }
                                }
                            }
                            if (label) label[row] = (uint8_t)arg;
                        }
                    }
                }
            } else {
                constexpr uint32_t kHalfCols = BN / 2;
                const uint32_t sw = (lane >> 1) & 3u;                       // swizzle of this lane's staging row
#pragma unroll 1
                for (uint32_t c = half * kHalfCols; c < (half + 1) * kHalfCols; c += 32) {
                    uint32_t v[32];
                    tmem_ld32(taddr + c, v);
                    tmem_ld_wait();
                    const float4* b4 = reinterpret_cast<const float4*>(bias + col0 + c);
                    // bias + ReLU + bf16, staged as this lane's 64-byte row (16-byte pieces XOR-swizzled by row)
#pragma unroll
                    for (int pc = 0; pc < 4; pc++) {
                        const float4 ba = __ldg(b4 + 2 * pc), bb = __ldg(b4 + 2 * pc + 1);
                        const float bv[8] = {ba.x, ba.y, ba.z, ba.w, bb.x, bb.y, bb.z, bb.w};
                        uint32_t pk[4];
#pragma unroll
                        for (int e = 0; e < 4; e++) {
                            pk[e] = bias_relu_bf16x2(v[pc * 8 + 2 * e], v[pc * 8 + 2 * e + 1], bv[2 * e], bv[2 * e + 1]);
                        }
                        *reinterpret_cast<uint4*>(stg + lane * 64u + (((uint32_t)pc ^ sw) << 4)) = make_uint4(pk[0], pk[1], pk[2], pk[3]);
                    }
                    __syncwarp();
                    // read back 8 rows x 64 B per instruction and store full 64-byte row segments
#pragma unroll
                    for (uint32_t it = 0; it < 4; it++) {
                        const uint32_t rr = it * 8u + (lane >> 2), pp = lane & 3u;
                        const uint4 val = *reinterpret_cast<const uint4*>(stg + rr * 64u + ((pp ^ ((rr >> 1) & 3u)) << 4));
                        if (row0 + rr < n_rows)
                            *reinterpret_cast<uint4*>(out + (size_t)(row0 + rr) * N + col0 + c + pp * 8u) = val;
                    }
                    __syncwarp();
                }
            }
            tc_fence_before();
            __syncwarp();
            if (lane == 0) {
                if constexpr (PAIR) mbar_arrive_cluster(map_to_cta(smem_u32(&bars->tmem_empty[buf]), 0));
                else mbar_arrive(&bars->tmem_empty[buf]);
            }
            buf ^= 1u; if (buf == 0) bphase ^= 1u;
        }
    }

    __syncthreads();
    if (*abort_flag) {
        // a wait ran out somewhere in this block: give copies in flight time to land
        if (threadIdx.x == 0) sf_dev_set_error(st, SF_ERR_DEVICE_TIMEOUT);
        __nanosleep(200000);
        __syncthreads();
    }
    if constexpr (PAIR) cluster_sync_all();          // the partner is done with this CTA's shared memory and barriers
    tc_fence_after();
    if (warp == 1) {
        __syncwarp();
        if constexpr (PAIR) tmem_dealloc_pair(tmem_base, Cfg::kTmemCols); else tmem_dealloc(tmem_base, Cfg::kTmemCols);
    }
}

// Can this device co-schedule two-CTA clusters of this kernel at all?  Asked once per kernel and device (the smem opt-in must
// already be set); where the answer is no, or the query fails, the single-CTA kernel serves the layer instead.
template <typename Kern>
bool pairs_supported(Kern k, size_t smem, int device, int (&cache)[64]) {
    int& c = cache[device & 63];                       // 0 unknown, 1 yes, -1 no
    if (c == 0) {
        cudaLaunchConfig_t lc = {};
        lc.gridDim = dim3(2); lc.blockDim = dim3(kGemmThreads); lc.dynamicSmemBytes = smem;
        cudaLaunchAttribute at[1];
        at[0].id = cudaLaunchAttributeClusterDimension;
        at[0].val.clusterDim.x = 2; at[0].val.clusterDim.y = 1; at[0].val.clusterDim.z = 1;
        lc.attrs = at; lc.numAttrs = 1;
        int n = 0;
        const cudaError_t e = cudaOccupancyMaxActiveClusters(&n, k, &lc);
        if (e != cudaSuccess) (void)cudaGetLastError();
        c = (e == cudaSuccess && n > 0) ? 1 : -1;
    }
    return c > 0;
}

// launch as clusters of two CTAs
template <typename Kern, typename... Args>
cudaError_t launch_pairs(Kern k, uint32_t grid, size_t smem, cudaStream_t st, Args... args) {
    cudaLaunchConfig_t lc = {};
    lc.gridDim = dim3(grid); lc.blockDim = dim3(kGemmThreads); lc.dynamicSmemBytes = smem; lc.stream = st;
    cudaLaunchAttribute at[2];
    at[0].id = cudaLaunchAttributeClusterDimension;
    at[0].val.clusterDim.x = 2; at[0].val.clusterDim.y = 1; at[0].val.clusterDim.z = 1;
    at[1].id = cudaLaunchAttributeProgrammaticStreamSerialization;       // a chained launch (the kernel starts with sf_chain_enter)
    at[1].val.programmaticStreamSerializationAllowed = 1;
    lc.attrs = at; lc.numAttrs = 2;
    return cudaLaunchKernelEx(&lc, k, args...);
}

template <uint32_t BN>
int launch_gemm(sf_ctx* ctx, const void* A, const void* W, const float* bias, const uint32_t* n_rows_dev,
                uint32_t capacity, uint32_t N, uint32_t K, void* out, cudaStream_t st, uint32_t small_max)
{
    using Cfg = GemmCfg<BN>;
    CUtensorMap tmA, tmW;
    int rc = encode_tmap_bf16_2d(&tmA, A, capacity, K, BM, BK);
    if (rc != SF_OK) return rc;
    rc = encode_tmap_bf16_2d(&tmW, W, N, K, BN, BK);
    if (rc != SF_OK) return rc;
    if constexpr (BN == 256) {
        if (small_max == 0) {                          // large batches: CTA pairs on 256 x 256 tiles
            using CfgP = GemmCfg<BN, true>;
            rc = encode_tmap_bf16_2d(&tmW, W, N, K, BN / 2, BK);
            if (rc != SF_OK) return rc;
            auto kp = gemm_bias_relu_bf16_kernel<BN, MODE_HIDDEN, 8, true>;
            static bool attr_set_dev[64] = {};
            bool& attr_set = attr_set_dev[ctx->device & 63];
            if (!attr_set) { SF_CUDA(cudaFuncSetAttribute(kp, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)CfgP::kSmemBytes)); attr_set = true; }
            static int pairs_ok[64] = {};
            const uint32_t pair_tiles = ((capacity + 2 * BM - 1) / (2 * BM)) * (N / BN);
            const uint32_t grid = 2u * std::min<uint32_t>((uint32_t)ctx->num_sms / 2u, pair_tiles);
            if (pairs_supported(kp, CfgP::kSmemBytes, ctx->device, pairs_ok)) {
            SF_CUDA(launch_pairs(kp, grid, CfgP::kSmemBytes, st, tmA, tmW, bias, n_rows_dev, N, K, reinterpret_cast<__nv_bfloat16*>(out), ctx->d_state,
                                 (float*)nullptr, (uint8_t*)nullptr, 0u, 0u, reinterpret_cast<const __nv_bfloat16*>(A),
                                 reinterpret_cast<const __nv_bfloat16*>(W), capacity, (const __nv_bfloat16*)nullptr, (const float*)nullptr));
            return SF_OK;
            }
            rc = encode_tmap_bf16_2d(&tmW, W, N, K, BN, BK);      // back to the single-CTA tile
            if (rc != SF_OK) return rc;
        }
    }
    auto k = gemm_bias_relu_bf16_kernel<BN, MODE_HIDDEN>;
    static bool attr_set_dev[64] = {};                 // the opt-in is per device
    bool& attr_set = attr_set_dev[ctx->device & 63];
    if (!attr_set) { SF_CUDA(cudaFuncSetAttribute(k, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)Cfg::kSmemBytes)); attr_set = true; }
    uint32_t max_tiles = ((capacity + BM - 1) / BM) * (N / BN);
    uint32_t grid = (uint32_t)ctx->num_sms < max_tiles ? (uint32_t)ctx->num_sms : max_tiles;
    SF_CUDA(sf_launch_chained(k, grid, kGemmThreads, Cfg::kSmemBytes, st, tmA, tmW, bias, n_rows_dev, N, K, reinterpret_cast<__nv_bfloat16*>(out),
                              ctx->d_state, (float*)nullptr, (uint8_t*)nullptr, 0u, small_max, reinterpret_cast<const __nv_bfloat16*>(A),
                              reinterpret_cast<const __nv_bfloat16*>(W), capacity, (const __nv_bfloat16*)nullptr, (const float*)nullptr));
    return SF_OK;
}

// last hidden layer with the head folded into its epilogue (no activations written); W16 = the head's weights padded to 16 rows
template <uint32_t BN, uint32_t CH>
int launch_gemm_head(sf_ctx* ctx, const void* A, const void* W, const float* bias, const uint32_t* n_rows_dev, uint32_t capacity,
                     uint32_t N, uint32_t K, const void* W16, const float* head_bias, uint32_t C, float* logits, uint8_t* label, cudaStream_t st,
                     uint32_t small_max, void* small_scratch /* bf16 [16][N]: the hidden layer of a few-rows batch */)
{
    using Cfg = GemmCfg<BN>;
    constexpr uint32_t kSmem = Cfg::kSmemBytesHead16;        // 32 KB of head weights where the other modes stage 16 KB of output
    CUtensorMap tmA, tmW;
    int rc = encode_tmap_bf16_2d(&tmA, A, capacity, K, BM, BK);
    if (rc != SF_OK) return rc;
    rc = encode_tmap_bf16_2d(&tmW, W, N, K, BN, BK);
    if (rc != SF_OK) return rc;
    if constexpr (BN == 256) {                         // CTA pairs: a pair owns whole 256-row panels
        constexpr uint32_t kSmemP = GemmCfg<BN, true>::kSmemBytesHead16;
        rc = encode_tmap_bf16_2d(&tmW, W, N, K, BN / 2, BK);
        if (rc != SF_OK) return rc;
        auto kp = gemm_bias_relu_bf16_kernel<BN, MODE_HIDDEN_HEAD, CH, true>;
        static bool attr_set_dev[64] = {};
        bool& attr_set = attr_set_dev[ctx->device & 63];
        if (!attr_set) { SF_CUDA(cudaFuncSetAttribute(kp, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)kSmemP)); attr_set = true; }
        static int pairs_ok[64] = {};
        const uint32_t pair_panels = (capacity + 2 * BM - 1) / (2 * BM);
        const uint32_t grid = 2u * std::min<uint32_t>((uint32_t)ctx->num_sms / 2u, pair_panels);
        if (pairs_supported(kp, kSmemP, ctx->device, pairs_ok)) {
        SF_CUDA(launch_pairs(kp, grid, kSmemP, st, tmA, tmW, bias, n_rows_dev, N, K, reinterpret_cast<__nv_bfloat16*>(small_scratch), ctx->d_state, logits, label, C, small_max,
                             reinterpret_cast<const __nv_bfloat16*>(A), reinterpret_cast<const __nv_bfloat16*>(W), capacity,
                             reinterpret_cast<const __nv_bfloat16*>(W16), head_bias));
        return SF_OK;
        }
        rc = encode_tmap_bf16_2d(&tmW, W, N, K, BN, BK);          // back to the single-CTA tile
        if (rc != SF_OK) return rc;
    }
    auto k = gemm_bias_relu_bf16_kernel<BN, MODE_HIDDEN_HEAD, CH>;
    static bool attr_set_dev[64] = {};                 // the opt-in is per device
    bool& attr_set = attr_set_dev[ctx->device & 63];
    if (!attr_set) { SF_CUDA(cudaFuncSetAttribute(k, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)kSmem)); attr_set = true; }
    const uint32_t panels = (capacity + BM - 1) / BM;
    const uint32_t grid = (uint32_t)ctx->num_sms < panels ? (uint32_t)ctx->num_sms : panels;
    SF_CUDA(sf_launch_chained(k, grid, kGemmThreads, kSmem, st, tmA, tmW, bias, n_rows_dev, N, K, reinterpret_cast<__nv_bfloat16*>(small_scratch), ctx->d_state, logits, label, C, small_max,
                              reinterpret_cast<const __nv_bfloat16*>(A), reinterpret_cast<const __nv_bfloat16*>(W), capacity,
                              reinterpret_cast<const __nv_bfloat16*>(W16), head_bias));
    return SF_OK;
}

// last layer on the tensor cores: one 128 x 16 tile per 128 rows, W padded to 16 rows
int launch_head_tc(sf_ctx* ctx, const void* A, const void* W16, const float* bias, const uint32_t* n_rows_dev,
                   uint32_t capacity, uint32_t K, uint32_t C, float* logits, uint8_t* label, cudaStream_t st, uint32_t small_max)
{
    using Cfg = GemmCfg<16>;
    CUtensorMap tmA, tmW;
    int rc = encode_tmap_bf16_2d(&tmA, A, capacity, K, BM, BK);
    if (rc != SF_OK) return rc;
    rc = encode_tmap_bf16_2d(&tmW, W16, 16, K, 16, BK);
    if (rc != SF_OK) return rc;
    auto k = gemm_bias_relu_bf16_kernel<16, MODE_HEAD>;
    static bool attr_set_dev[64] = {};                 // the opt-in is per device
    bool& attr_set = attr_set_dev[ctx->device & 63];
    if (!attr_set) { SF_CUDA(cudaFuncSetAttribute(k, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)Cfg::kSmemBytes)); attr_set = true; }
    uint32_t max_tiles = (capacity + BM - 1) / BM;
    uint32_t grid = (uint32_t)ctx->num_sms < max_tiles ? (uint32_t)ctx->num_sms : max_tiles;
    SF_CUDA(sf_launch_chained(k, grid, kGemmThreads, Cfg::kSmemBytes, st, tmA, tmW, bias, n_rows_dev, 16u, K, (__nv_bfloat16*)nullptr, ctx->d_state, logits, label,
                              C, small_max, reinterpret_cast<const __nv_bfloat16*>(A), reinterpret_cast<const __nv_bfloat16*>(W16), capacity,
                              (const __nv_bfloat16*)nullptr, (const float*)nullptr));
    return SF_OK;
}


}  // namespace

int sf_mlp_bf16_forward(sf_ctx* ctx, const sf_slow* s, const void* rows, const uint32_t* n_rows_dev, uint32_t capacity,
                        float* logits, uint8_t* label, void* scratch, cudaStream_t st)
{
    uint32_t maxh = 0;
    for (uint32_t l = 1; l < s->n_layers; l++) if (s->dims[l] > maxh) maxh = s->dims[l];
    char* h0 = reinterpret_cast<char*>(scratch);
    char* h1 = h0 + sf_align256((size_t)capacity * maxh * 2);
    // batches that may hold only a handful of rows (the streaming path) may take the CUDA-core path inside the same kernels
    bool small = capacity <= 65536;
    for (uint32_t l = 0; l < s->n_layers; l++) if (s->dims[l] > kSmallMaxK || (s->dims[l] % 8) != 0) small = false;
    const uint32_t small_max = small ? kSmallRows : 0u;
    const void* in = rows;
    const uint32_t L = s->n_layers - 1;                  // the head
    // The head is folded into the last hidden layer (its activations are then never written or re-read; a few-rows batch
    // keeps them in a 16-row scratch and the block that finishes last adds the head): one launch less either way.
    // Not where a row panel has a single column tile (the epilogue warps' hand-over needs two tiles between two panel ends).
    const uint32_t Nl = s->dims[L], Cn = s->dims[L + 1];
    const uint32_t BNl = Nl % 256 == 0 ? 256u : (Nl % 128 == 0 ? 128u : 64u);
    const bool fuse_head = Nl <= kFusedHeadMaxN && Nl / BNl >= 2;
    sf_time_begin(ctx, SF_T_GEMM, st);
    for (uint32_t l = 0; l + 1 < s->n_layers; l++) {
        void* out = (l & 1) ? h1 : h0;
        const uint32_t K = s->dims[l], N = s->dims[l + 1];
        int rc;
        if (fuse_head && l + 1 == L) {
#define SF_FUSED_CH(BNv, CHv) launch_gemm_head<BNv, CHv>(ctx, in, s->d_W[l], s->d_b[l], n_rows_dev, capacity, N, K, s->d_W[L], s->d_b[L], Cn, logits, label, st, small_max, out)
#define SF_FUSED(BNv) (Cn <= 2 ? SF_FUSED_CH(BNv, 2) : (Cn <= 4 ? SF_FUSED_CH(BNv, 4) : (Cn <= 8 ? SF_FUSED_CH(BNv, 8) : SF_FUSED_CH(BNv, 16))))
            if (N % 256 == 0)      rc = SF_FUSED(256);
            else if (N % 128 == 0) rc = SF_FUSED(128);
            else                   rc = SF_FUSED(64);
#undef SF_FUSED
#undef SF_FUSED_CH
        }
        else if (N % 256 == 0) rc = launch_gemm<256>(ctx, in, s->d_W[l], s->d_b[l], n_rows_dev, capacity, N, K, out, st, small_max);
        else if (N % 128 == 0) rc = launch_gemm<128>(ctx, in, s->d_W[l], s->d_b[l], n_rows_dev, capacity, N, K, out, st, small_max);
        else                   rc = launch_gemm<64>(ctx, in, s->d_W[l], s->d_b[l], n_rows_dev, capacity, N, K, out, st, small_max);
        if (rc != SF_OK) return rc;
        in = out;
    }
    sf_time_end(ctx, SF_T_GEMM, st);
    if (fuse_head) return SF_OK;
    sf_time_begin(ctx, SF_T_HEAD, st);
    int rc = launch_head_tc(ctx, in, s->d_W[L], s->d_b[L], n_rows_dev, capacity, s->dims[L], s->dims[L + 1], logits, label, st, small_max);
    sf_time_end(ctx, SF_T_HEAD, st);
    return rc;
}

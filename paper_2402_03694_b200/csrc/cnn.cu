// S4 (1-D CNN slow model), one fused kernel per batch of assigned flows:
//   conv1 (k=5, 8 -> 64) + ReLU -> conv2 (k=5, 64 -> 128) + ReLU -> mean over the 128
//   positions -> linear 128 -> n_cls -> argmax.
// Both convolutions run on the tcgen05 tensor cores; nothing but the 2 KB input row and the
// logits touches HBM.
//
// Shifted ("same" padded) operands without im2col.  Activations are kept in shared memory
// in the un-swizzled core-matrix layout: for every group of 8 channels a column of 16-byte
// rows, one row per position, with zero rows above and below.  In that layout a matrix
// descriptor's start address may be moved by whole rows, so tap t of a convolution is the
// same buffer started t positions further down; the zero rows supply the padding.
//
// conv1 takes one flow's 128 positions as the M = 128 rows of a tile (N = 64 output channels;
// 8 input channels = one 16-byte row per position, so consecutive taps are consecutive rows and a
// K = 16 step covers two taps with a K-direction stride of 16 bytes).
//
// conv2 is issued the other way round, for TWO flows at once: the weights of a tap are the A
// operand (M = 128 output channels), the activations of a pair of flows are the B operand with
// N = 256 = 128 positions x 2 flows, rows interleaved (row 2p + s = position p of flow s, so a tap
// is a shift by two rows and the two flows share the zero padding rows).  On this part an
// M = 128 tcgen05.mma of K = 16 holds the tensor pipe for max(N/2, ~98) cycles, so only N = 256
// runs at the full rate; with a single flow per instruction (N = 128) a third of the pipe idles.
// The accumulator then has the output channel as its TMEM lane and (position, flow) as its
// column, so the mean over positions is a plain sum inside one thread: bias, ReLU and the bf16
// rounding of the activation are applied per element, the rounded values are added in
// position order, and no pooling pass or third contraction is needed.  The linear head
// (128 -> n_cls, 2 Kflop per flow) runs on CUDA cores from the pooled values, with every cross-thread
// sum a fixed shuffle tree (deterministic).
//
// Persistent CTAs, one per SM, loop over pairs of flows.  Warp roles:
//   warp 0        streams input rows with bulk copies into a ring
//   warp 1        issues conv2's MMAs, pair after pair, into alternating accumulators
//   warp 2        issues conv1's MMAs, three pairs ahead of the pair whose accumulator the epilogue is emptying
//   warps 3..18   epilogue: conv2 accumulator of pair k -> registers (and released) -> bias + ReLU -> bf16 -> partial
//                 sums over 32 positions; then conv1 accumulators of pair k+3 -> bias + ReLU -> bf16 -> conv2's B
//                 operand (shared memory); warp = (TMEM lane quarter, column group)
//   warps 19..22  partial sums -> mean -> linear head -> logits, argmax
// The tensor pipe queues only two or three instructions, so a thread that issues MMAs must not do anything
// else for long: hence one issuing thread per MMA stream.  TMEM holds exactly two conv2 accumulators (2 x 256
// columns): conv2 of pair k+1 starts the moment conv2 of pair k ends, while the epilogue empties the other
// accumulator at leisure.  conv1 has no columns of its own: the accumulators of pair k+3 are written into the
// buffer the epilogue has just emptied (pair k's), are pulled into registers at once, and conv2 of pair k+2 reuses
// the buffer after that.  conv1's bias reaches the epilogue as a kernel parameter (constant bank).  Every wait is
// bounded; on a timeout the block records SF_ERR_DEVICE_TIMEOUT and leaves.
#include "tc_common.cuh"
#include <stdlib.h>
#include <string.h>

namespace {
using namespace sftc;

constexpr uint32_t L = 128, CIN = 8, C1 = 64, C2 = 128, KW = 5, NCLS_MAX = 16;
constexpr uint32_t kEWarps = 16, kE3Warps = 4;
constexpr uint32_t kEFirst = 3, kE3First = kEFirst + kEWarps;
constexpr uint32_t kThreads = (kE3First + kE3Warps) * 32;       // 736
constexpr uint32_t NH1 = 3;                                 // conv1 output (= conv2 operand) buffers
constexpr uint32_t XS = 4;                                  // input-row ring depth
constexpr uint32_t X_STAGE = (2 + L + 3) * 16;              // 2 zero rows, 128 rows, 3 zero rows (tap 5 is a zero tap)
constexpr uint32_t H1_COL = 2 * (2 + L + 2) * 16;           // one 8-channel column of a PAIR's conv1 output: 264 rows, 4,224 bytes
constexpr uint32_t H1_BYTES = (C1 / 8) * H1_COL;            // 33,792
// weight blob (device and shared memory share this layout)
constexpr uint32_t W2_OFF = 0;                              // [5 taps][8 k-chunks][128 out][8] bf16
constexpr uint32_t W2_BYTES = KW * (C1 / 8) * C2 * 16;      // 81,920
constexpr uint32_t W1_OFF = W2_OFF + W2_BYTES;              // [6 taps][64 out][8] bf16 (tap 5 = 0)
constexpr uint32_t W1_BYTES = 6 * C1 * 16;                  // 6,144
constexpr uint32_t W3_OFF = W1_OFF + W1_BYTES;              // fp32 [16 classes][128], values rounded to bf16, zero beyond n_cls
constexpr uint32_t W3_BYTES = NCLS_MAX * C2 * 4;            // 8,192
constexpr uint32_t B1_OFF = W3_OFF + W3_BYTES;              // fp32 [64]
constexpr uint32_t B2_OFF = B1_OFF + C1 * 4;                // fp32 [128]
constexpr uint32_t B3_OFF = B2_OFF + C2 * 4;                // fp32 [16]
constexpr uint32_t BLOB_BYTES = B3_OFF + NCLS_MAX * 4;
// shared memory map
constexpr uint32_t SM_BLOB = 0;
constexpr uint32_t SM_H1 = SM_BLOB + BLOB_BYTES;            // NH1 pair buffers
constexpr uint32_t SM_X = SM_H1 + NH1 * H1_BYTES;           // XS stages
constexpr uint32_t PART_BYTES = 4 * 2 * C2 * 4;             // fp32 [4 position groups][2 flows][128 channels]
constexpr uint32_t SM_PART = SM_X + XS * X_STAGE;           // 2 buffers
constexpr uint32_t SM_PART2 = SM_PART + 2 * PART_BYTES;     // fp32 [4 warps][32] partial logits
constexpr uint32_t SM_BARS = SM_PART2 + kE3Warps * 32 * 4;
constexpr uint32_t SM_TOTAL = SM_BARS + 320;
static_assert(BLOB_BYTES % 16 == 0 && SM_H1 % 16 == 0 && SM_X % 16 == 0 && SM_PART % 16 == 0 && SM_BARS % 8 == 0, "alignment");
static_assert(SM_TOTAL <= 232448, "shared memory");
// TMEM columns: two conv2 accumulators of 256 columns; conv1's accumulators of a pair (2 x 64 columns) borrow the
// first half of the conv2 accumulator that is idle at the time
constexpr uint32_t TM_D2 = 256;                             // columns per conv2 accumulator

struct Bars {
    uint64_t w_full;
    uint64_t x_full[XS], x_empty[XS];
    uint64_t d1_full[2], d1_empty[2];          // conv1 accumulators of pair j: index j & 1
    uint64_t h1_full[NH1], h1_empty[NH1];      // conv2 operand of pair j: index j % NH1
    uint64_t d2_full[2], d2_empty[2];          // conv2 accumulator of pair p: index p & 1
    uint64_t c1_issued;                        // conv1 of a pair has been handed to the tensor pipe
    uint64_t part_full[2], part_empty[2];
    uint32_t tmem_base, abort_flag;
};
static_assert(sizeof(Bars) <= 320, "barrier block");

__device__ __forceinline__ void named_barrier_sync(uint32_t id, uint32_t count) {
    asm volatile("bar.sync %0, %1;" ::"r"(id), "r"(count) : "memory");
}

// Sum over the 32 lanes of each of 32 per-lane values; lane l ends up with value l's total.
// The order of additions is a fixed tree, so the result is reproducible run to run.
__device__ __forceinline__ float transpose_reduce32(float (&v)[32], uint32_t lane) {
#pragma unroll
    for (int off = 16; off >= 1; off >>= 1) {
        const bool up = (lane & off) != 0;
#pragma unroll
        for (int j = 0; j < off; j++) {
            const float keep = up ? v[j + off] : v[j];
            const float send = up ? v[j] : v[j + off];
            v[j] = keep + __shfl_xor_sync(0xFFFFFFFFu, send, off);
        }
    }
    return v[0];
}

// {high half: bf16(max(hi, 0)), low half: bf16(max(lo, 0))}, round to nearest even
__device__ __forceinline__ uint32_t relu_bf16x2(float hi, float lo) {
    uint32_t d;
    asm("cvt.rn.relu.bf16x2.f32 %0, %1, %2;" : "=r"(d) : "f"(hi), "f"(lo));
    return d;
}
__device__ __forceinline__ uint32_t pack_relu_bf16(uint32_t a, uint32_t b, float ba, float bb) {
    return relu_bf16x2(__uint_as_float(b) + bb, __uint_as_float(a) + ba);     // a in the low half
}

struct Bias1 { float v[C1]; };

__global__ void __launch_bounds__(kThreads, 1)
cnn_fused_kernel(const __nv_bfloat16* __restrict__ rows, const uint32_t* __restrict__ n_rows_dev,
                 const unsigned char* __restrict__ blob, const __grid_constant__ Bias1 b1, uint32_t n_cls,
                 float* __restrict__ logits, uint8_t* __restrict__ label, sf_dev_state* st, uint32_t capacity)
{
    extern __shared__ __align__(128) uint8_t smem[];
    Bars* bars = reinterpret_cast<Bars*>(smem + SM_BARS);
    volatile uint32_t* abort_flag = &bars->abort_flag;
    const uint32_t sbase = smem_u32(smem);
    const uint32_t warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
    const uint32_t n_rows = sf_clamp_rows(*n_rows_dev, capacity, st);      // the caller's word, bounded by what the buffers hold
    // flows of this CTA: blockIdx.x, blockIdx.x + gridDim.x, ...; flow m of the CTA is slot (m & 1) of pair (m >> 1)
    const uint32_t n_mine = (n_rows > blockIdx.x) ? (n_rows - blockIdx.x + gridDim.x - 1) / gridDim.x : 0;
    const uint32_t n_pairs = (n_mine + 1) >> 1;

    // zero everything that acts as padding (and the rest of the activation buffers: the unused
    // slot of an odd last pair is multiplied like any other and must hold finite numbers)
    for (uint32_t i = threadIdx.x; i < (NH1 * H1_BYTES + XS * X_STAGE) / 16; i += kThreads)
        reinterpret_cast<uint4*>(smem + SM_H1)[i] = make_uint4(0, 0, 0, 0);
    if (threadIdx.x == 0) {
        mbar_init(&bars->w_full, 1);
        for (uint32_t s = 0; s < XS; s++) { mbar_init(&bars->x_full[s], 1); mbar_init(&bars->x_empty[s], 1); }
        for (uint32_t b = 0; b < 2; b++) {
            mbar_init(&bars->d1_full[b], 1); mbar_init(&bars->d1_empty[b], kEWarps);
            mbar_init(&bars->d2_full[b], 1); mbar_init(&bars->d2_empty[b], kEWarps);
            mbar_init(&bars->part_full[b], kEWarps); mbar_init(&bars->part_empty[b], kE3Warps);
        }
        for (uint32_t b = 0; b < NH1; b++) { mbar_init(&bars->h1_full[b], kEWarps); mbar_init(&bars->h1_empty[b], 1); }
        mbar_init(&bars->c1_issued, 1);
        bars->abort_flag = 0;
        fence_barrier_init();
    }
    fence_proxy_async();                       // the zero fill must be visible to the tensor-core reads
    if (warp == 1) tmem_alloc(&bars->tmem_base, 512);
    tc_fence_before();
    __syncthreads();
    tc_fence_after();
    const uint32_t tmem_base = bars->tmem_base;
    const uint32_t q = warp & 3u;                    // TMEM lane quarter an epilogue warp may read

    if (warp == 0) {
        if (lane == 0 && n_mine > 0) {
            mbar_expect_tx(&bars->w_full, BLOB_BYTES);
            bulk_load(smem + SM_BLOB, blob, BLOB_BYTES, &bars->w_full);
            for (uint32_t m = 0; m < n_mine; m++) {
                const uint32_t s = m % XS, ph = (m / XS) & 1u;
                if (!mbar_wait_relaxed(&bars->x_empty[s], ph ^ 1u, abort_flag)) break;
                const uint32_t r = blockIdx.x + m * gridDim.x;
                mbar_expect_tx(&bars->x_full[s], L * CIN * 2);
                bulk_load(smem + SM_X + s * X_STAGE + 32, rows + (size_t)r * L * CIN, L * CIN * 2, &bars->x_full[s]);
            }
        }
    } else if (warp == 1) {
        // ---- conv2: weights of tap t (A, M = 128 output channels) x the pair's activations (B, N = 256) ----
        if (lane == 0 && n_mine > 0) {
            constexpr uint32_t idesc2 = make_idesc_bf16(C2, 2 * L);
            // descriptor = constant fields + (address >> 4) in the low bits: build the bases once, add offsets per MMA
            const uint64_t dH1 = make_smem_desc(sbase + SM_H1, H1_COL, 128, 0);
            const uint64_t dW2 = make_smem_desc(sbase + SM_BLOB + W2_OFF, C2 * 16u, 128, 0);
            bool ok = mbar_wait(&bars->w_full, 0, abort_flag);
            for (uint32_t p = 0; p < n_pairs && ok; p++) {
                const uint32_t b = p & 1u, hb = p % NH1;
                if (!mbar_wait(&bars->h1_full[hb], (p / NH1) & 1u, abort_flag)) break;
                // the accumulator is free once conv1 of pair p + 1, which borrowed it, sits in registers (that conv1 was
                // itself issued after conv2 of pair p - 2 had been emptied); without a pair p + 1 wait for pair p - 2 directly
                if (p + 1 < n_pairs) { if (!mbar_wait(&bars->d1_empty[(p + 1) & 1u], ((p + 1) >> 1) & 1u, abort_flag)) break; }
                else if (p >= 2) { if (!mbar_wait(&bars->d2_empty[b], ((p - 2) >> 1) & 1u, abort_flag)) break; }
                tc_fence_after();
                const uint64_t bh = dH1 + (uint64_t)((hb * H1_BYTES) >> 4);
#pragma unroll
                for (uint32_t t = 0; t < KW; t++) {
                    // Give way once per pair: this thread refills the pipe's short queue the moment a slot frees, and conv1 of
                    // pair p + 2 (issued by the other thread as soon as the epilogue has emptied the previous accumulator) would
                    // otherwise get in only after this pair's last MMA - too late for the next pair.  Only a matter of timing:
                    // no result depends on this wait.
                    if (t == 4 && p >= 1 && p + 2 < n_pairs && !mbar_wait(&bars->c1_issued, (p + 2) & 1u, abort_flag)) { ok = false; break; }
#pragma unroll
                    for (uint32_t k = 0; k < C1 / 16; k++)      // the activations two rows per tap further down
                        umma_bf16(tmem_base + b * TM_D2, dW2 + ((t * ((C1 / 8) * C2 * 16u) + (2u * k) * (C2 * 16u)) >> 4),
                                  bh + (((2u * k) * H1_COL + t * 32u) >> 4), idesc2, (t | k) != 0 ? 1u : 0u);
                }
                if (!ok) break;
                umma_commit(&bars->d2_full[b]);
                umma_commit(&bars->h1_empty[hb]);
            }
        }
    } else if (warp == 2) {
        // ---- conv1: one flow's positions (A, M = 128) x the weights of two taps (B, N = 64) ----
        if (lane == 0 && n_mine > 0) {
            constexpr uint32_t idesc1 = make_idesc_bf16(128, C1);
            const uint64_t dX = make_smem_desc(sbase + SM_X, 16, 128, 0);
            const uint64_t dW1 = make_smem_desc(sbase + SM_BLOB + W1_OFF, C1 * 16u, 128, 0);
            bool ok = mbar_wait(&bars->w_full, 0, abort_flag);
            for (uint32_t j = 0; j < n_pairs && ok; j++) {
                const uint32_t n_fl = (2u * j + 1u < n_mine) ? 2u : 1u;
                for (uint32_t s = 0; s < n_fl && ok; s++) {
                    const uint32_t m = 2u * j + s;
                    ok = mbar_wait(&bars->x_full[m % XS], (m / XS) & 1u, abort_flag);
                }
                // the accumulators go into conv2's buffer (j + 1) & 1: pair j - 2's conv1 results must have left it, and so
                // must conv2 of pair j - 3
                if (ok && j >= 2) ok = mbar_wait(&bars->d1_empty[j & 1u], ((j - 2) >> 1) & 1u, abort_flag);
                if (ok && j >= 3) ok = mbar_wait(&bars->d2_empty[(j + 1) & 1u], ((j - 3) >> 1) & 1u, abort_flag);
                if (!ok) break;
                tc_fence_after();
                for (uint32_t s = 0; s < n_fl; s++) {
                    const uint32_t xs = (2u * j + s) % XS;
                    const uint64_t ax = dX + (uint64_t)((xs * X_STAGE) >> 4);
#pragma unroll
                    for (uint32_t k = 0; k < 3; k++)         // taps (2k, 2k+1): rows shifted by 2k, next tap = next row
                        umma_bf16(tmem_base + ((j + 1) & 1u) * TM_D2 + s * C1, ax + ((k * 32u) >> 4), dW1 + ((k * 2u * (C1 * 16u)) >> 4),
                                  idesc1, k != 0 ? 1u : 0u);
                    umma_commit(&bars->x_empty[xs]);
                }
                umma_commit(&bars->d1_full[j & 1u]);
                mbar_arrive(&bars->c1_issued);
            }
        }
    } else if (n_mine > 0 && warp < kE3First) {
        // ---- epilogue warps: (TMEM lane quarter q, column group cg) ----
        const uint32_t cg = (warp - kEFirst) >> 2;
        bool ok = __all_sync(0xFFFFFFFFu, mbar_wait_relaxed(&bars->w_full, 0, abort_flag));
        const float bias2 = ok ? reinterpret_cast<const float*>(smem + SM_BLOB + B2_OFF)[q * 32u + lane] : 0.0f;

        // conv1 accumulators of pair j [position = lane][channels 16cg .. 16cg+15] of both flows -> conv2's B operand
        auto conv1_out = [&](uint32_t j) -> bool {
            const uint32_t hb = j % NH1, n_fl = (2u * j + 1u < n_mine) ? 2u : 1u;
            bool w = mbar_wait_relaxed(&bars->d1_full[j & 1u], (j >> 1) & 1u, abort_flag) &&
                     mbar_wait_relaxed(&bars->h1_empty[hb], ((j / NH1) & 1u) ^ 1u, abort_flag);
            if (!__all_sync(0xFFFFFFFFu, w)) return false;
            tc_fence_after();
            const uint32_t taddr = tmem_base + ((q * 32u) << 16) + ((j + 1) & 1u) * TM_D2 + cg * 16u;
            uint32_t v[2][16];
            tmem_ld16(taddr, v[0]);
            if (n_fl > 1) tmem_ld16(taddr + C1, v[1]);
            tmem_ld_wait();
            tc_fence_before();
            __syncwarp();
            if (lane == 0) mbar_arrive(&bars->d1_empty[j & 1u]);     // the accumulators are in registers: the buffer is conv2's again
            const uint32_t p = q * 32u + lane;                       // position
#pragma unroll
            for (int s = 0; s < 2; s++) {
                if ((uint32_t)s < n_fl) {
                    uint8_t* hrow = smem + SM_H1 + hb * H1_BYTES + (2u * cg) * H1_COL + (2u * (p + 2u) + s) * 16u;
#pragma unroll
                    for (int h = 0; h < 2; h++) {                    // two columns of 8 channels
                        uint32_t pk[4];
#pragma unroll
                        for (int e = 0; e < 4; e++)
                            pk[e] = pack_relu_bf16(v[s][h * 8 + e * 2], v[s][h * 8 + e * 2 + 1], b1.v[cg * 16u + h * 8 + e * 2],
                                                   b1.v[cg * 16u + h * 8 + e * 2 + 1]);
                        *reinterpret_cast<uint4*>(hrow + h * H1_COL) = make_uint4(pk[0], pk[1], pk[2], pk[3]);
                    }
                }
            }
            fence_proxy_async();                                 // activations -> visible to the MMA's shared-memory reads
            __syncwarp();
            if (lane == 0) mbar_arrive(&bars->h1_full[hb]);
            return true;
        };
        // conv2 accumulator of pair k [channel = lane][positions 32cg .. 32cg+31 of both flows] -> sums over those positions
        auto conv2_out = [&](uint32_t k) -> bool {
            const uint32_t b = k & 1u;
            if (!__all_sync(0xFFFFFFFFu, mbar_wait(&bars->d2_full[b], (k >> 1) & 1u, abort_flag))) return false;
            tc_fence_after();
            const uint32_t taddr = tmem_base + ((q * 32u) << 16) + b * TM_D2 + cg * 64u;
            uint32_t v0[32], v1[32];
            tmem_ld32(taddr, v0);
            tmem_ld32(taddr + 32, v1);
            tmem_ld_wait();
            tc_fence_before();
            __syncwarp();
            if (lane == 0) mbar_arrive(&bars->d2_empty[b]);          // the accumulator is in registers: conv1 of pair k + 3 may borrow it
            float s0 = 0.0f, s1 = 0.0f;
#pragma unroll
            for (int j = 0; j < 16; j++) {                // columns 2j, 2j+1 = position 32cg+j of flows 0, 1
                const uint32_t h = relu_bf16x2(__uint_as_float(v0[2 * j + 1]) + bias2, __uint_as_float(v0[2 * j]) + bias2);
                s0 += __uint_as_float(h << 16);
                s1 += __uint_as_float(h & 0xFFFF0000u);
            }
#pragma unroll
            for (int j = 0; j < 16; j++) {
                const uint32_t h = relu_bf16x2(__uint_as_float(v1[2 * j + 1]) + bias2, __uint_as_float(v1[2 * j]) + bias2);
                s0 += __uint_as_float(h << 16);
                s1 += __uint_as_float(h & 0xFFFF0000u);
            }
            if (!__all_sync(0xFFFFFFFFu, mbar_wait_relaxed(&bars->part_empty[b], ((k >> 1) & 1u) ^ 1u, abort_flag))) return false;
            float* part = reinterpret_cast<float*>(smem + SM_PART + b * PART_BYTES) + cg * 2u * C2;
            part[q * 32u + lane] = s0;
            part[C2 + q * 32u + lane] = s1;
            __syncwarp();
            if (lane == 0) mbar_arrive(&bars->part_full[b]);
            return true;
        };
        for (uint32_t j = 0; j < 3 && j < n_pairs && ok; j++) ok = conv1_out(j);
        for (uint32_t k = 0; k < n_pairs && ok; k++) {
            ok = conv2_out(k);
            if (ok && k + 3 < n_pairs) ok = conv1_out(k + 3);
        }
    } else if (n_mine > 0) {
        // ---- E3: partial sums -> mean -> linear head -> logits, argmax -----------------
        const uint32_t ew = warp - kE3First;
        const uint32_t ch = ew * 32u + lane;                              // 0..127
        float* part2 = reinterpret_cast<float*>(smem + SM_PART2);
        bool ok = __all_sync(0xFFFFFFFFu, mbar_wait_relaxed(&bars->w_full, 0, abort_flag));
        float w3r[NCLS_MAX];
#pragma unroll
        for (int c = 0; c < (int)NCLS_MAX; c++) w3r[c] = ok ? reinterpret_cast<const float*>(smem + SM_BLOB + W3_OFF)[c * C2 + ch] : 0.0f;
        const float* b3 = reinterpret_cast<const float*>(smem + SM_BLOB + B3_OFF);
        for (uint32_t i = 0; i < n_pairs && ok; i++) {
            const uint32_t b = i & 1u;
            ok = __all_sync(0xFFFFFFFFu, mbar_wait_relaxed(&bars->part_full[b], (i >> 1) & 1u, abort_flag));
            if (!ok) break;
            const float* part = reinterpret_cast<const float*>(smem + SM_PART + b * PART_BYTES);
            float pooled[2];
#pragma unroll
            for (int s = 0; s < 2; s++)                                   // position groups in order, then the mean (an exact scaling)
                pooled[s] = (((part[s * C2 + ch] + part[(2 + s) * C2 + ch]) + part[(4 + s) * C2 + ch]) + part[(6 + s) * C2 + ch]) * (1.0f / 128.0f);
            __syncwarp();
            if (lane == 0) mbar_arrive(&bars->part_empty[b]);
            float x[32];
#pragma unroll
            for (int s = 0; s < 2; s++)
#pragma unroll
                for (int c = 0; c < (int)NCLS_MAX; c++) x[s * 16 + c] = pooled[s] * w3r[c];
            const float tot = transpose_reduce32(x, lane);                // this warp's 32 channels; lane = flow slot * 16 + class
            part2[ew * 32u + lane] = tot;
            named_barrier_sync(1, kE3Warps * 32);
            if (ew == 0) {
                const uint32_t s = lane >> 4, c = lane & 15u, m = 2u * i + s;
                const uint32_t r = blockIdx.x + m * gridDim.x;
                float lg = -3.0e38f;
                if (c < n_cls && m < n_mine) {
                    lg = ((part2[lane] + part2[32 + lane]) + part2[64 + lane]) + part2[96 + lane] + b3[c];
                    logits[(size_t)r * n_cls + c] = lg;
                }
                // argmax over the 16 lanes of a flow slot, lowest index on ties
                float best = lg; uint32_t arg = c;
#pragma unroll
                for (int o = 8; o >= 1; o >>= 1) {
                    const float ob = __shfl_xor_sync(0xFFFFFFFFu, best, o);
                    const uint32_t oa = __shfl_xor_sync(0xFFFFFFFFu, arg, o);
                    if (ob > best || (ob == best && oa < arg)) { best = ob; arg = oa; }
                }
                if (c == 0 && m < n_mine && label) label[r] = (uint8_t)arg;
            }
            named_barrier_sync(1, kE3Warps * 32);                     // part2 is free again
        }
    }

    __syncthreads();
    if (*abort_flag) {
        if (threadIdx.x == 0) sf_dev_set_error(st, SF_ERR_DEVICE_TIMEOUT);
        __nanosleep(200000);
        __syncthreads();
    }
    tc_fence_after();
    if (warp == 1) { __syncwarp(); tmem_dealloc(tmem_base, 512); }
}

uint16_t bf16_bits(float x) {
    uint32_t u; memcpy(&u, &x, 4);
    uint32_t low = u & 0xFFFFu, up = u >> 16;
    if (low > 0x8000u || (low == 0x8000u && (up & 1u))) up++;
    return (uint16_t)up;
}

}  // namespace

int sf_cnn_prepare(sf_slow* s, const float* w1, const float* b1, const float* w2, const float* b2,
                   const float* w3, const float* b3)
{
    unsigned char* h = (unsigned char*)calloc(1, BLOB_BYTES);
    if (!h) return SF_ERR_ALLOC;
    uint16_t* W2 = reinterpret_cast<uint16_t*>(h + W2_OFF);
    for (uint32_t t = 0; t < KW; t++)
        for (uint32_t j = 0; j < C1 / 8; j++)
            for (uint32_t n = 0; n < C2; n++)
                for (uint32_t e = 0; e < 8; e++)
                    W2[((t * (C1 / 8) + j) * C2 + n) * 8 + e] = bf16_bits(w2[((size_t)n * KW + t) * C1 + j * 8 + e]);
    uint16_t* W1 = reinterpret_cast<uint16_t*>(h + W1_OFF);
    for (uint32_t t = 0; t < KW; t++)
        for (uint32_t n = 0; n < C1; n++)
            for (uint32_t e = 0; e < CIN; e++)
                W1[(t * C1 + n) * 8 + e] = bf16_bits(w1[((size_t)n * KW + t) * CIN + e]);
    // head weights rounded to bf16 (the model's precision), kept as fp32 for the CUDA-core head
    float* W3 = reinterpret_cast<float*>(h + W3_OFF);
    for (uint32_t c = 0; c < s->n_cls; c++)
        for (uint32_t k = 0; k < C2; k++) {
            uint32_t bits = (uint32_t)bf16_bits(w3[(size_t)c * C2 + k]) << 16;
            memcpy(&W3[c * C2 + k], &bits, 4);
        }
    memcpy(h + B1_OFF, b1, C1 * 4);
    memcpy(s->h_cnn_b1, b1, C1 * 4);
    memcpy(h + B2_OFF, b2, C2 * 4);
    memcpy(h + B3_OFF, b3, s->n_cls * 4);
    cudaError_t e = cudaMalloc(&s->d_w1, BLOB_BYTES);
    if (e == cudaSuccess) e = cudaMemcpy(s->d_w1, h, BLOB_BYTES, cudaMemcpyHostToDevice);
    free(h);
    if (e != cudaSuccess) return sf_set_cuda_error(e, "sf_cnn_prepare");
    return SF_OK;
}

int sf_cnn_bf16_forward(sf_ctx* ctx, const sf_slow* s, const void* rows, const uint32_t* n_rows_dev, uint32_t capacity,
                        float* logits, uint8_t* label, void* scratch, cudaStream_t st)
{
    (void)scratch;
    static bool attr_set_dev[64] = {};                 // the opt-in is per device
    bool& attr_set = attr_set_dev[ctx->device & 63];
    if (!attr_set) { SF_CUDA(cudaFuncSetAttribute(cnn_fused_kernel, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)SM_TOTAL)); attr_set = true; }
    uint32_t grid = (uint32_t)ctx->num_sms < capacity ? (uint32_t)ctx->num_sms : capacity;
    sf_time_begin(ctx, SF_T_GEMM, st);
    cnn_fused_kernel<<<grid, kThreads, SM_TOTAL, st>>>(reinterpret_cast<const __nv_bfloat16*>(rows), n_rows_dev,
                                                     reinterpret_cast<const unsigned char*>(s->d_w1), *reinterpret_cast<const Bias1*>(s->h_cnn_b1), s->n_cls,
                                                     logits, label, ctx->d_state, capacity);
    sf_time_end(ctx, SF_T_GEMM, st);
    SF_LAUNCH_CHECK("cnn_fused_kernel");
    return SF_OK;
}

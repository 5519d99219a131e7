// S4 (1-D CNN slow model), one fused kernel per batch of assigned flows:
//   conv1 (k=5, 8 -> 64) + ReLU -> conv2 (k=5, 64 -> 128) + ReLU -> mean over the 128
//   positions -> linear 128 -> n_cls -> argmax.
// All three contractions run on the tcgen05 tensor cores with one flow's 128 positions as
// the M = 128 rows of a tile; nothing but the 2 KB input row and the logits touches HBM.
//
// Shifted ("same" padded) operands without im2col.  Activations are kept in shared memory
// in the un-swizzled core-matrix layout: for every group of 8 channels a column of 16-byte
// rows, one row per position, with zero rows above and below.  In that layout a matrix
// descriptor's start address may be moved by whole rows, so tap t of a convolution is the
// same buffer started t rows further down; the zero rows supply the padding.  For conv1
// (8 input channels = one 16-byte row per position) consecutive taps are consecutive rows,
// so a K = 16 step (two taps) uses a K-direction stride of 16 bytes.
//
// Pooling and the linear head are one more MMA: mean_p(h2[p][:]) . W3^T = sum_p (h2[p][:] .
// (W3/128)^T), i.e. a [128 positions] x [16 classes] product over the 128 channels followed
// by a sum over positions (TMEM lanes), which a shuffle tree and four partial sums finish in a
// fixed order (deterministic).
//
// Persistent CTAs, one per SM, loop over flows.  Warp roles:
//   warp 0        streams input rows with bulk copies into a ring
//   warp 1        issues the MMAs in the order conv1(i+2), conv2(i), head(i-2)
//   warps 2..5    E1: conv1 accumulators -> bias + ReLU -> bf16 -> conv2's A operand (shared memory)
//   warps 6..21   E2: conv2 accumulators -> bias + ReLU -> bf16 -> the head's A operand
//   warps 22..25  E3: head accumulators -> sum over positions -> + bias -> logits, argmax
// Every accumulator and activation buffer is double (conv1: triple) buffered, so the three epilogues and the
// tensor pipe overlap.  Every wait is bounded; on a timeout the block records
// SF_ERR_DEVICE_TIMEOUT and leaves.
#include "tc_common.cuh"
#include <stdlib.h>
#include <string.h>

namespace {
using namespace sftc;

constexpr uint32_t L = 128, CIN = 8, C1 = 64, C2 = 128, KW = 5, NCLS_MAX = 16;
constexpr uint32_t kE1Warps = 4, kE2Warps = 16, kE3Warps = 4;
constexpr uint32_t kE1First = 2, kE2First = kE1First + kE1Warps, kE3First = kE2First + kE2Warps;
constexpr uint32_t kThreads = (kE3First + kE3Warps) * 32;       // 832
constexpr uint32_t XS = 4;                                  // input-row ring depth
constexpr uint32_t X_STAGE = (2 + L + 3) * 16;              // 2 zero rows, 128 rows, 3 zero rows (tap 5 is a zero tap)
constexpr uint32_t H1_COL = (2 + L + 2) * 16;               // one 8-channel column of conv1's output: 2112 bytes
constexpr uint32_t H1_BYTES = (C1 / 8) * H1_COL;            // 16,896
constexpr uint32_t H2_COL = L * 16;                         // one 8-channel column of conv2's output: 2048 bytes
constexpr uint32_t H2_BYTES = (C2 / 8) * H2_COL;            // 32,768
// weight blob (device and shared memory share this layout)
constexpr uint32_t W2_OFF = 0;                              // [5 taps][8 k-chunks][128 n][8] bf16
constexpr uint32_t W2_BYTES = KW * (C1 / 8) * C2 * 16;      // 81,920
constexpr uint32_t W1_OFF = W2_OFF + W2_BYTES;              // [6 taps][64 n][8] bf16 (tap 5 = 0)
constexpr uint32_t W1_BYTES = 6 * C1 * 16;                  // 6,144
constexpr uint32_t W3_OFF = W1_OFF + W1_BYTES;              // [16 k-chunks][16 classes][8] bf16, scaled by 1/128
constexpr uint32_t W3_BYTES = (C2 / 8) * NCLS_MAX * 16;     // 4,096
constexpr uint32_t B1_OFF = W3_OFF + W3_BYTES;              // fp32 [64]
constexpr uint32_t B2_OFF = B1_OFF + C1 * 4;                // fp32 [128]
constexpr uint32_t B3_OFF = B2_OFF + C2 * 4;                // fp32 [16]
constexpr uint32_t BLOB_BYTES = B3_OFF + NCLS_MAX * 4;
// shared memory map
constexpr uint32_t SM_BLOB = 0;
constexpr uint32_t NB1 = 3;                                 // conv1 accumulator / activation buffers (conv1 runs two flows ahead)
constexpr uint32_t SM_H1 = SM_BLOB + BLOB_BYTES;            // NB1 buffers
constexpr uint32_t SM_H2 = SM_H1 + NB1 * H1_BYTES;          // 2 buffers
constexpr uint32_t SM_X = SM_H2 + 2 * H2_BYTES;             // XS stages
constexpr uint32_t SM_PART = SM_X + XS * X_STAGE;           // fp32 [4 warps][16] partial logits
constexpr uint32_t SM_BARS = SM_PART + 4 * NCLS_MAX * 4;
constexpr uint32_t SM_TOTAL = SM_BARS + 320;
static_assert(BLOB_BYTES % 16 == 0 && SM_H1 % 16 == 0 && SM_H2 % 16 == 0 && SM_X % 16 == 0 && SM_BARS % 8 == 0, "alignment");
static_assert(SM_TOTAL <= 232448, "shared memory");
// TMEM columns: conv1 accumulators [3][64], conv2 [2][128], head [2][16]
constexpr uint32_t TM_D1 = 0, TM_D2 = 192, TM_D4 = 448;

struct Bars {
    uint64_t w_full;
    uint64_t x_full[XS], x_empty[XS];
    uint64_t d1_full[NB1], d1_empty[NB1], h1_full[NB1], h1_empty[NB1];
    uint64_t d2_full[2], d2_empty[2], h2_full[2], h2_empty[2];
    uint64_t d4_full[2], d4_empty[2];
    uint32_t tmem_base, abort_flag;
};
static_assert(sizeof(Bars) <= 320, "barrier block");

__device__ __forceinline__ void named_barrier_sync(uint32_t id, uint32_t count) {
    asm volatile("bar.sync %0, %1;" ::"r"(id), "r"(count) : "memory");
}

// sum over the 32 lanes of each of 16 per-lane values; lanes l and l+16 end up with column (l & 15)'s
// total.  The order of additions is a fixed tree, so the result is reproducible run to run.
__device__ __forceinline__ float transpose_reduce16(float (&v)[16], uint32_t lane) {
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
    return v[0];
}

__device__ __forceinline__ uint32_t pack_relu_bf16(uint32_t a, uint32_t b, float ba, float bb) {
    __nv_bfloat162 h = __floats2bfloat162_rn(fmaxf(__uint_as_float(a) + ba, 0.0f), fmaxf(__uint_as_float(b) + bb, 0.0f));
    return *reinterpret_cast<uint32_t*>(&h);
}

__global__ void __launch_bounds__(kThreads, 1)
cnn_fused_kernel(const __nv_bfloat16* __restrict__ rows, const uint32_t* __restrict__ n_rows_dev,
                 const unsigned char* __restrict__ blob, uint32_t n_cls,
                 float* __restrict__ logits, uint8_t* __restrict__ label, sf_dev_state* st)
{
    extern __shared__ __align__(128) uint8_t smem[];
    Bars* bars = reinterpret_cast<Bars*>(smem + SM_BARS);
    volatile uint32_t* abort_flag = &bars->abort_flag;
    const uint32_t sbase = smem_u32(smem);
    const uint32_t warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
    const uint32_t n_rows = *n_rows_dev;
    // flows of this CTA: blockIdx.x, blockIdx.x + gridDim.x, ...
    const uint32_t n_mine = (n_rows > blockIdx.x) ? (n_rows - blockIdx.x + gridDim.x - 1) / gridDim.x : 0;

    // zero everything that acts as padding (and the rest of the activation buffers)
    for (uint32_t i = threadIdx.x; i < (NB1 * H1_BYTES + 2 * H2_BYTES + XS * X_STAGE) / 16; i += kThreads)
        reinterpret_cast<uint4*>(smem + SM_H1)[i] = make_uint4(0, 0, 0, 0);
    if (threadIdx.x == 0) {
        mbar_init(&bars->w_full, 1);
        for (uint32_t s = 0; s < XS; s++) { mbar_init(&bars->x_full[s], 1); mbar_init(&bars->x_empty[s], 1); }
        for (uint32_t b = 0; b < NB1; b++) {
            mbar_init(&bars->d1_full[b], 1); mbar_init(&bars->d1_empty[b], kE1Warps);
            mbar_init(&bars->h1_full[b], kE1Warps); mbar_init(&bars->h1_empty[b], 1);
        }
        for (uint32_t b = 0; b < 2; b++) {
            mbar_init(&bars->d2_full[b], 1); mbar_init(&bars->d2_empty[b], kE2Warps);
            mbar_init(&bars->h2_full[b], kE2Warps); mbar_init(&bars->h2_empty[b], 1);
            mbar_init(&bars->d4_full[b], 1); mbar_init(&bars->d4_empty[b], kE3Warps);
        }
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
    const uint32_t p = q * 32u + lane;               // position handled by an epilogue thread

    if (warp == 0) {
        if (lane == 0 && n_mine > 0) {
            mbar_expect_tx(&bars->w_full, BLOB_BYTES);
            bulk_load(smem + SM_BLOB, blob, BLOB_BYTES, &bars->w_full);
            for (uint32_t i = 0; i < n_mine; i++) {
                const uint32_t s = i % XS, ph = (i / XS) & 1u;
                if (!mbar_wait_relaxed(&bars->x_empty[s], ph ^ 1u, abort_flag)) break;
                const uint32_t r = blockIdx.x + i * gridDim.x;
                mbar_expect_tx(&bars->x_full[s], L * CIN * 2);
                bulk_load(smem + SM_X + s * X_STAGE + 32, rows + (size_t)r * L * CIN, L * CIN * 2, &bars->x_full[s]);
            }
        }
    } else if (warp == 1) {
        if (lane == 0 && n_mine > 0) {
            constexpr uint32_t idesc1 = make_idesc_bf16(128, C1);
            constexpr uint32_t idesc2 = make_idesc_bf16(128, C2);
            constexpr uint32_t idesc4 = make_idesc_bf16(128, NCLS_MAX);
            // descriptor = constant fields + (address >> 4) in the low bits: build the bases once, add offsets per MMA
            const uint64_t dX = make_smem_desc(sbase + SM_X, 16, 128, 0);
            const uint64_t dW1 = make_smem_desc(sbase + SM_BLOB + W1_OFF, C1 * 16u, 128, 0);
            const uint64_t dH1 = make_smem_desc(sbase + SM_H1, H1_COL, 128, 0);
            const uint64_t dW2 = make_smem_desc(sbase + SM_BLOB + W2_OFF, C2 * 16u, 128, 0);
            const uint64_t dH2 = make_smem_desc(sbase + SM_H2, H2_COL, 128, 0);
            const uint64_t dW3 = make_smem_desc(sbase + SM_BLOB + W3_OFF, NCLS_MAX * 16u, 128, 0);
            bool ok = mbar_wait(&bars->w_full, 0, abort_flag);
            auto conv1 = [&](uint32_t i) -> bool {
                const uint32_t s = i % XS, xph = (i / XS) & 1u, b = i % NB1, ph = (i / NB1) & 1u;
                if (!mbar_wait(&bars->x_full[s], xph, abort_flag)) return false;
                if (!mbar_wait(&bars->d1_empty[b], ph ^ 1u, abort_flag)) return false;
                tc_fence_after();
                const uint64_t ax = dX + (uint64_t)((s * X_STAGE) >> 4);
#pragma unroll
                for (uint32_t k = 0; k < 3; k++)             // taps (2k, 2k+1): rows shifted by 2k, next tap = next row
                    umma_bf16(tmem_base + TM_D1 + b * C1, ax + ((k * 32u) >> 4), dW1 + ((k * 2u * (C1 * 16u)) >> 4), idesc1,
                              k != 0 ? 1u : 0u);
                umma_commit(&bars->x_empty[s]);
                umma_commit(&bars->d1_full[b]);
                return true;
            };
            auto conv2 = [&](uint32_t i) -> bool {
                const uint32_t b = i & 1u, ph = (i >> 1) & 1u, b1i = i % NB1, ph1 = (i / NB1) & 1u;
                if (!mbar_wait(&bars->h1_full[b1i], ph1, abort_flag)) return false;
                if (!mbar_wait(&bars->d2_empty[b], ph ^ 1u, abort_flag)) return false;
                tc_fence_after();
                const uint64_t ah = dH1 + (uint64_t)((b1i * H1_BYTES) >> 4);
#pragma unroll
                for (uint32_t t = 0; t < KW; t++) {
#pragma unroll
                    for (uint32_t k = 0; k < C1 / 16; k++)
                        umma_bf16(tmem_base + TM_D2 + b * C2, ah + (((2u * k) * H1_COL + t * 16u) >> 4),
                                  dW2 + ((t * ((C1 / 8) * C2 * 16u) + (2u * k) * (C2 * 16u)) >> 4), idesc2, (t | k) != 0 ? 1u : 0u);
                }
                umma_commit(&bars->h1_empty[b1i]);
                umma_commit(&bars->d2_full[b]);
                return true;
            };
            auto head = [&](uint32_t i) -> bool {
                const uint32_t b = i & 1u, ph = (i >> 1) & 1u;
                if (!mbar_wait(&bars->h2_full[b], ph, abort_flag)) return false;
                if (!mbar_wait(&bars->d4_empty[b], ph ^ 1u, abort_flag)) return false;
                tc_fence_after();
                const uint64_t ah = dH2 + (uint64_t)((b * H2_BYTES) >> 4);
#pragma unroll
                for (uint32_t k = 0; k < C2 / 16; k++)
                    umma_bf16(tmem_base + TM_D4 + b * NCLS_MAX, ah + (((2u * k) * H2_COL) >> 4),
                              dW3 + (((2u * k) * (NCLS_MAX * 16u)) >> 4), idesc4, k != 0 ? 1u : 0u);
                umma_commit(&bars->h2_empty[b]);
                umma_commit(&bars->d4_full[b]);
                return true;
            };
            // conv1 runs two flows ahead and the head two flows behind conv2, so that each epilogue has two
            // conv2 periods to turn its accumulator into the next operand
            if (ok) ok = conv1(0);
            if (ok && n_mine > 1) ok = conv1(1);
            for (uint32_t i = 0; i < n_mine && ok; i++) {
                if (i + 2 < n_mine) ok = conv1(i + 2);
                if (ok) ok = conv2(i);
                if (ok && i >= 2) ok = head(i - 2);
            }
            if (ok && n_mine >= 2) ok = head(n_mine - 2);
            if (ok) ok = head(n_mine - 1);
        }
    } else if (n_mine > 0 && warp < kE2First) {
        // ---- E1: conv1 accumulators -> conv2's A operand -------------------------------
        const float* b1 = reinterpret_cast<const float*>(smem + SM_BLOB + B1_OFF);
        bool ok = __all_sync(0xFFFFFFFFu, mbar_wait_relaxed(&bars->w_full, 0, abort_flag));
        for (uint32_t i = 0; i < n_mine && ok; i++) {
            const uint32_t b = i % NB1, ph = (i / NB1) & 1u;
            bool w = mbar_wait_relaxed(&bars->d1_full[b], ph, abort_flag) && mbar_wait_relaxed(&bars->h1_empty[b], ph ^ 1u, abort_flag);
            ok = __all_sync(0xFFFFFFFFu, w);
            if (!ok) break;
            tc_fence_after();
            const uint32_t taddr = tmem_base + ((q * 32u) << 16) + TM_D1 + b * C1;
            uint8_t* hrow = smem + SM_H1 + b * H1_BYTES + (p + 2u) * 16u;
            uint32_t v0[32], v1[32];
            tmem_ld32(taddr, v0);
            tmem_ld32(taddr + 32, v1);
            tmem_ld_wait();
            tc_fence_before();
            __syncwarp();
            if (lane == 0) mbar_arrive(&bars->d1_empty[b]);      // the accumulator is in registers: conv1 may reuse it
#pragma unroll
            for (int j = 0; j < 8; j++) {                // 8 columns of 8 channels
                uint32_t pk[4];
#pragma unroll
                for (int e = 0; e < 4; e++) {
                    const int c = (j & 3) * 8 + e * 2;
                    const uint32_t a = (j < 4) ? v0[c] : v1[c], bq = (j < 4) ? v0[c + 1] : v1[c + 1];
                    pk[e] = pack_relu_bf16(a, bq, b1[j * 8 + e * 2], b1[j * 8 + e * 2 + 1]);
                }
                *reinterpret_cast<uint4*>(hrow + j * H1_COL) = make_uint4(pk[0], pk[1], pk[2], pk[3]);
            }
            fence_proxy_async();                         // activations -> visible to the MMA's shared-memory reads
            __syncwarp();
            if (lane == 0) mbar_arrive(&bars->h1_full[b]);
        }
    } else if (n_mine > 0 && warp < kE3First) {
        // ---- E2: conv2 accumulators -> the head's A operand ----------------------------
        const uint32_t g = (warp - kE2First) >> 2;        // 32 of the 128 conv2 channels
        const float* b2 = reinterpret_cast<const float*>(smem + SM_BLOB + B2_OFF);
        bool ok = __all_sync(0xFFFFFFFFu, mbar_wait_relaxed(&bars->w_full, 0, abort_flag));
        for (uint32_t i = 0; i < n_mine && ok; i++) {
            const uint32_t b = i & 1u, ph = (i >> 1) & 1u;
            bool w = mbar_wait_relaxed(&bars->d2_full[b], ph, abort_flag) && mbar_wait_relaxed(&bars->h2_empty[b], ph ^ 1u, abort_flag);
            ok = __all_sync(0xFFFFFFFFu, w);
            if (!ok) break;
            tc_fence_after();
            const uint32_t c0 = g * 32u;
            uint32_t v[32];
            tmem_ld32(tmem_base + ((q * 32u) << 16) + TM_D2 + b * C2 + c0, v);
            tmem_ld_wait();
            tc_fence_before();
            __syncwarp();
            if (lane == 0) mbar_arrive(&bars->d2_empty[b]);      // the accumulator is in registers: conv2 may reuse it
            uint8_t* hrow = smem + SM_H2 + b * H2_BYTES + p * 16u;
#pragma unroll
            for (int j = 0; j < 4; j++) {
                uint32_t pk[4];
#pragma unroll
                for (int e = 0; e < 4; e++) {
                    const int c = j * 8 + e * 2;
                    pk[e] = pack_relu_bf16(v[c], v[c + 1], b2[c0 + c], b2[c0 + c + 1]);
                }
                *reinterpret_cast<uint4*>(hrow + ((c0 >> 3) + j) * H2_COL) = make_uint4(pk[0], pk[1], pk[2], pk[3]);
            }
            fence_proxy_async();
            __syncwarp();
            if (lane == 0) mbar_arrive(&bars->h2_full[b]);
        }
    } else if (n_mine > 0) {
        // ---- E3: head accumulators [position][class] -> sum over positions -> logits ----
        const uint32_t et = (warp - kE3First) * 32u + lane;           // 0..127
        const float* b3 = reinterpret_cast<const float*>(smem + SM_BLOB + B3_OFF);
        float* part = reinterpret_cast<float*>(smem + SM_PART);
        bool ok = __all_sync(0xFFFFFFFFu, mbar_wait_relaxed(&bars->w_full, 0, abort_flag));
        for (uint32_t i = 0; i < n_mine && ok; i++) {
            const uint32_t b = i & 1u, ph = (i >> 1) & 1u;
            ok = __all_sync(0xFFFFFFFFu, mbar_wait_relaxed(&bars->d4_full[b], ph, abort_flag));
            if (!ok) break;
            tc_fence_after();
            uint32_t v[16];
            tmem_ld16(tmem_base + ((q * 32u) << 16) + TM_D4 + b * NCLS_MAX, v);
            tmem_ld_wait();
            tc_fence_before();
            __syncwarp();
            if (lane == 0) mbar_arrive(&bars->d4_empty[b]);
            float x[16];
#pragma unroll
            for (int c = 0; c < 16; c++) x[c] = __uint_as_float(v[c]);
            const float tot = transpose_reduce16(x, lane);            // this warp's 32 positions, class lane & 15
            if (lane < 16) part[(warp - kE3First) * NCLS_MAX + lane] = tot;
            named_barrier_sync(1, kE3Warps * 32);
            const uint32_t r = blockIdx.x + i * gridDim.x;
            if (et < 32) {                                            // first E3 warp: lane c < n_cls finishes class c
                float lg = -3.0e38f;
                if (lane < n_cls) {
                    lg = ((part[lane] + part[NCLS_MAX + lane]) + part[2 * NCLS_MAX + lane]) + part[3 * NCLS_MAX + lane] + b3[lane];
                    logits[(size_t)r * n_cls + lane] = lg;
                }
                // argmax, lowest index on ties
                float best = lg; uint32_t arg = lane;
#pragma unroll
                for (int o = 16; o >= 1; o >>= 1) {
                    const float ob = __shfl_xor_sync(0xFFFFFFFFu, best, o);
                    const uint32_t oa = __shfl_xor_sync(0xFFFFFFFFu, arg, o);
                    if (ob > best || (ob == best && oa < arg)) { best = ob; arg = oa; }
                }
                if (lane == 0 && label) label[r] = (uint8_t)arg;
            }
            named_barrier_sync(1, kE3Warps * 32);                     // part is free again
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
    // head weights rounded to bf16, then scaled by 2^-7 (exact) so that the MMA yields the mean's contribution
    uint16_t* W3 = reinterpret_cast<uint16_t*>(h + W3_OFF);
    for (uint32_t c = 0; c < s->n_cls; c++)
        for (uint32_t k = 0; k < C2; k++) {
            uint32_t bits = (uint32_t)bf16_bits(w3[(size_t)c * C2 + k]) << 16;
            float f; memcpy(&f, &bits, 4);
            W3[((k / 8) * NCLS_MAX + c) * 8 + (k % 8)] = bf16_bits(f * (1.0f / 128.0f));
        }
    memcpy(h + B1_OFF, b1, C1 * 4);
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
                                                     reinterpret_cast<const unsigned char*>(s->d_w1), s->n_cls,
                                                     logits, label, ctx->d_state);
    sf_time_end(ctx, SF_T_GEMM, st);
    SF_LAUNCH_CHECK("cnn_fused_kernel");
    return SF_OK;
}

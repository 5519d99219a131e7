// S1: per-flow statistical features of the first N packet headers.
//
// One thread per flow.  A thread streams its packets in chunks of 8 (16-byte
// vector loads of the uint16 sizes and uint32 inter-arrival times when the row
// pitch allows it), keeps one integer accumulator set per feature group in
// registers, converts once at the end, and the block hands its [flows][F] tile to
// global memory through shared memory so that the stores are fully coalesced.
// All statistics come from exact integer sums (128-bit for the variance numerator
// of inter-arrival times); each fp32 value is produced by exactly one rounding
// (integer -> fp32 RNE) or one IEEE division, so results are reproducible bit for bit.
#include "common.cuh"

namespace {

constexpr int kFlowsPerBlock = 128;

struct Acc {
    uint32_t cnt, mn, mx, first, last;
    uint64_t s1;        // sum
    uint64_t s2lo;      // sum of squares, low 64 bits
    uint32_t s2hi;      // high part (only inter-arrival times can carry into it)
};

__device__ __forceinline__ void acc_init(Acc& a) {
    a.cnt = 0; a.mn = 0xFFFFFFFFu; a.mx = 0; a.first = 0; a.last = 0; a.s1 = 0; a.s2lo = 0; a.s2hi = 0;
}

template <bool WIDE>
__device__ __forceinline__ void acc_add(Acc& a, uint32_t x, bool take) {
    if (take) {
        if (a.cnt == 0) a.first = x;
        a.mn = min(a.mn, x);
        a.mx = max(a.mx, x);
        a.last = x;
        a.s1 += x;
        uint64_t sq = (uint64_t)x * (uint64_t)x;
        uint64_t lo = a.s2lo + sq;
        if (WIDE) a.s2hi += (lo < sq) ? 1u : 0u;
        a.s2lo = lo;
        a.cnt += 1;
    }
}

// exact unsigned 128-bit value (hi:lo) -> fp32, round to nearest even.
// Above 64 bits: normalise into a 64-bit window, OR the dropped bits into a
// sticky bit (it sits far below the rounding position), convert once, and scale
// by an exact power of two.
__device__ __forceinline__ float u128_to_f32(uint64_t hi, uint64_t lo) {
    if (hi == 0) return __ull2float_rn(lo);
    int s = 64 - __clzll((long long)hi);                     // 1..64
    uint64_t w = (s == 64) ? hi : ((hi << (64 - s)) | (lo >> s));
    uint64_t dropped = (s == 64) ? lo : (lo << (64 - s));
    w |= (dropped != 0) ? 1ull : 0ull;
    float f = __ull2float_rn(w);
    return __fmul_rn(f, __uint_as_float((uint32_t)(127 + s) << 23));   // * 2^s, exact
}

__device__ __forceinline__ void acc_finish(const Acc& a, float* o) {
    if (a.cnt == 0) {
#pragma unroll
        for (int k = 0; k < 8; k++) o[k] = 0.0f;
        return;
    }
    float fc = __uint2float_rn(a.cnt);
    float fs = __ull2float_rn(a.s1);
    // V = cnt * S2 - S1^2 as an exact 128-bit integer
    uint64_t c = a.cnt;
    uint64_t p_lo = c * a.s2lo;
    uint64_t p_hi = __umul64hi(c, a.s2lo) + c * (uint64_t)a.s2hi;
    uint64_t q_lo = a.s1 * a.s1;
    uint64_t q_hi = __umul64hi(a.s1, a.s1);
    uint64_t v_lo = p_lo - q_lo;
    uint64_t v_hi = p_hi - q_hi - ((p_lo < q_lo) ? 1ull : 0ull);
    o[0] = fc;
    o[1] = fs;
    o[2] = __uint2float_rn(a.mn);
    o[3] = __uint2float_rn(a.mx);
    o[4] = __fdiv_rn(fs, fc);
    o[5] = __fdiv_rn(u128_to_f32(v_hi, v_lo), __uint2float_rn(a.cnt * a.cnt));
    o[6] = __uint2float_rn(a.first);
    o[7] = __uint2float_rn(a.last);
}

template <int G>
__device__ __forceinline__ void packet(Acc (&A)[G], uint32_t sz, uint32_t ia, uint32_t i, uint32_t dirw) {
    bool d = (dirw >> i) & 1u;
    bool turn = (i >= 1) && (((dirw >> (i - 1)) & 1u) != (uint32_t)d);
    acc_add<false>(A[0], sz, true);
    if (G > 1) acc_add<true>(A[1], ia, true);
    if (G > 2) acc_add<false>(A[2], sz, !d);
    if (G > 3) acc_add<false>(A[3], sz, d);
    if (G > 4) acc_add<true>(A[4], ia, !d);
    if (G > 5) acc_add<true>(A[5], ia, d);
    if (G > 6) acc_add<false>(A[6], sz, turn);
    if (G > 7) acc_add<true>(A[7], ia, turn);
}

// VEC: row pitch is a multiple of 8 packets, so size rows are 16-byte aligned
// and inter-arrival rows 32-byte aligned.
template <int G, bool VEC>
__global__ void __launch_bounds__(kFlowsPerBlock)
extract_kernel(const uint16_t* __restrict__ size, const uint32_t* __restrict__ iat,
               const uint32_t* __restrict__ dir_bits, const uint8_t* __restrict__ n_valid,
               uint32_t n, uint32_t pitch, uint32_t N, float* __restrict__ feat, const uint32_t* __restrict__ n_dev)
{
    constexpr int F = 8 * G;
    constexpr int STRIDE = F + 1;                  // odd stride: conflict-free row writes
    extern __shared__ float tile[];                // [kFlowsPerBlock][STRIDE]
    if (n_dev) n = min(n, *n_dev);               // optional device-side flow count (streaming path)
    const uint32_t f0 = blockIdx.x * kFlowsPerBlock;
    if (f0 >= n) return;
    const uint32_t f = f0 + threadIdx.x;

    if (f < n) {
        Acc A[G];
#pragma unroll
        for (int g = 0; g < G; g++) acc_init(A[g]);
        uint32_t m = N;
        if (n_valid) m = min(m, (uint32_t)n_valid[f]);
        // N <= 32: all direction bits of the window are in the row's first word
        const uint32_t dirw = dir_bits[(size_t)f * ((pitch + 31) >> 5)];
        const uint16_t* srow = size + (size_t)f * pitch;
        const uint32_t* irow = iat + (size_t)f * pitch;
        if (VEC) {
            for (uint32_t base = 0; base < m; base += 8) {
                uint4 s4 = __ldg(reinterpret_cast<const uint4*>(srow + base));
                uint4 a4 = __ldg(reinterpret_cast<const uint4*>(irow + base));
                uint4 b4 = __ldg(reinterpret_cast<const uint4*>(irow + base + 4));
                uint32_t sz[8] = {s4.x & 0xFFFFu, s4.x >> 16, s4.y & 0xFFFFu, s4.y >> 16,
                                  s4.z & 0xFFFFu, s4.z >> 16, s4.w & 0xFFFFu, s4.w >> 16};
                uint32_t ia[8] = {a4.x, a4.y, a4.z, a4.w, b4.x, b4.y, b4.z, b4.w};
#pragma unroll
                for (int j = 0; j < 8; j++)
                    if (base + j < m) packet<G>(A, sz[j], ia[j], base + j, dirw);
            }
        } else {
            for (uint32_t i = 0; i < m; i++) packet<G>(A, srow[i], irow[i], i, dirw);
        }
        float* o = tile + threadIdx.x * STRIDE;
#pragma unroll
        for (int g = 0; g < G; g++) acc_finish(A[g], o + 8 * g);
    }
    __syncthreads();
    const uint32_t rows = min((uint32_t)kFlowsPerBlock, n - f0);
    const uint32_t total = rows * F;
    float* dst = feat + (size_t)f0 * F;
    for (uint32_t e = threadIdx.x; e < total; e += kFlowsPerBlock) {
        uint32_t r = e / F, c = e - r * F;
        dst[e] = tile[r * STRIDE + c];
    }
}

template <int G>
int launch_g(const sf_packets* pk, uint32_t N, float* feat, cudaStream_t st, const uint32_t* n_dev) {
    const uint32_t n = pk->n_flows;
    const bool vec = (pk->pitch_pkts % 8 == 0) && (((uintptr_t)pk->size & 15) == 0) && (((uintptr_t)pk->iat_us & 15) == 0);
    const size_t smem = (size_t)kFlowsPerBlock * (8 * G + 1) * sizeof(float);
    const uint32_t grid = (n + kFlowsPerBlock - 1) / kFlowsPerBlock;
    if (vec)
        extract_kernel<G, true><<<grid, kFlowsPerBlock, smem, st>>>(pk->size, pk->iat_us, pk->dir_bits, pk->n_valid, n, pk->pitch_pkts, N, feat, n_dev);
    else
        extract_kernel<G, false><<<grid, kFlowsPerBlock, smem, st>>>(pk->size, pk->iat_us, pk->dir_bits, pk->n_valid, n, pk->pitch_pkts, N, feat, n_dev);
    SF_LAUNCH_CHECK("extract_kernel");
    return SF_OK;
}

}  // namespace

int sf_launch_extract(const sf_packets* pk, uint32_t N, uint32_t F, float* feat, cudaStream_t st, const uint32_t* n_dev) {
    if (pk->n_flows == 0) return SF_OK;
    switch (F / 8) {
    case 1: return launch_g<1>(pk, N, feat, st, n_dev);
    case 2: return launch_g<2>(pk, N, feat, st, n_dev);
    case 3: return launch_g<3>(pk, N, feat, st, n_dev);
    case 4: return launch_g<4>(pk, N, feat, st, n_dev);
    case 5: return launch_g<5>(pk, N, feat, st, n_dev);
    case 6: return launch_g<6>(pk, N, feat, st, n_dev);
    case 7: return launch_g<7>(pk, N, feat, st, n_dev);
    case 8: return launch_g<8>(pk, N, feat, st, n_dev);
    }
    return SF_ERR_UNSUPPORTED;
}

extern "C" int sf_extract_features(sf_ctx* ctx, const sf_packets* pk, uint32_t N, uint32_t F,
                                   float* feat_out, void* stream)
{
    if (!ctx || !pk || !feat_out) return SF_ERR_ARG;
    if (!pk->size || !pk->iat_us || !pk->dir_bits) return SF_ERR_ARG;
    if (N < 1 || N > 32 || N > pk->pitch_pkts) return SF_ERR_ARG;
    if (F < 8 || F > 64 || (F % 8) != 0) return SF_ERR_ARG;
    SF_CUDA(cudaSetDevice(ctx->device));
    sf_time_new_record(ctx);
    sf_time_begin(ctx, SF_T_EXTRACT, (cudaStream_t)stream);
    int rc = sf_launch_extract(pk, N, F, feat_out, (cudaStream_t)stream);
    sf_time_end(ctx, SF_T_EXTRACT, (cudaStream_t)stream);
    return rc;
}

// S1: per-flow statistical features of the first N packet headers.
//
// One thread per flow.  A thread streams its packets in chunks of 8 (16-byte
// vector loads of the uint16 sizes and uint32 inter-arrival times when the row
// pitch allows it), keeps one integer accumulator set per feature group in
// registers (subset membership, counts, first and last come from bit masks of the
// direction word), converts once at the end, and the block hands its [flows][F] tile to
// global memory through shared memory so that the stores are fully coalesced.
// All statistics come from exact integer sums (128-bit for the variance numerator
// of inter-arrival times); each fp32 value is produced by exactly one rounding
// (integer -> fp32 RNE) or one IEEE division, so results are reproducible bit for bit.
#include "common.cuh"

namespace {

constexpr int kFlowsPerBlock = 32;       // one warp per block: small blocks schedule better here than 64- or 128-flow ones (measured)

// Integer accumulators of one (quantity, subset) group.  Counts, first and last come from
// the subset's bit mask (popcount / lowest / highest set bit), so the per-packet work is
// two selects, a min, a max and the exact sums.
struct Acc {
    uint32_t mn, mx;
    uint64_t s1;        // sum
    uint64_t s2lo;      // sum of squares, low 64 bits
    uint32_t s2hi;      // high part (only inter-arrival times can carry into it)
};

__device__ __forceinline__ void acc_init(Acc& a) { a.mn = 0xFFFFFFFFu; a.mx = 0; a.s1 = 0; a.s2lo = 0; a.s2hi = 0; }

// sizes (16 bit): the square fits 32 bits and the sums never carry out of 64 bits
__device__ __forceinline__ void add_size(Acc& a, uint32_t x, bool take) {
    const uint32_t x0 = take ? x : 0u, xm = take ? x : 0xFFFFFFFFu;
    a.mn = min(a.mn, xm);
    a.mx = max(a.mx, x0);
    a.s1 += x0;
    a.s2lo += (uint64_t)(x0 * x0);
}
// inter-arrival times (32 bit): 64-bit squares, 128-bit sum of squares
__device__ __forceinline__ void add_iat(Acc& a, uint32_t x, bool take) {
    const uint32_t x0 = take ? x : 0u, xm = take ? x : 0xFFFFFFFFu;
    a.mn = min(a.mn, xm);
    a.mx = max(a.mx, x0);
    a.s1 += x0;
    const uint64_t sq = (uint64_t)x0 * (uint64_t)x0;
    const uint64_t lo = a.s2lo + sq;
    a.s2hi += (lo < sq) ? 1u : 0u;
    a.s2lo = lo;
}
// min / max only (the sums of the complementary subset come from a subtraction)
__device__ __forceinline__ void add_minmax(Acc& a, uint32_t x, bool take) {
    a.mn = min(a.mn, take ? x : 0xFFFFFFFFu);
    a.mx = max(a.mx, take ? x : 0u);
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

// eight slots of one group: cnt, sum, min, max, mean, var, first, last
__device__ __forceinline__ void finish(uint32_t cnt, uint32_t mn, uint32_t mx, uint64_t s1, uint64_t s2lo, uint64_t s2hi,
                                       uint32_t first, uint32_t last, float* o) {
    float4* o4 = reinterpret_cast<float4*>(o);       // 16-byte stores: conflict-free across a quarter warp
    if (cnt == 0) {
        o4[0] = make_float4(0.0f, 0.0f, 0.0f, 0.0f);
        o4[1] = make_float4(0.0f, 0.0f, 0.0f, 0.0f);
        return;
    }
    const float fc = __uint2float_rn(cnt);
    const float fs = __ull2float_rn(s1);
    // V = cnt * S2 - S1^2 as an exact 128-bit integer
    const uint64_t c = cnt;
    const uint64_t p_lo = c * s2lo;
    const uint64_t p_hi = __umul64hi(c, s2lo) + c * s2hi;
    const uint64_t q_lo = s1 * s1;
    const uint64_t q_hi = __umul64hi(s1, s1);
    const uint64_t v_lo = p_lo - q_lo;
    const uint64_t v_hi = p_hi - q_hi - ((p_lo < q_lo) ? 1ull : 0ull);
    o4[0] = make_float4(fc, fs, __uint2float_rn(mn), __uint2float_rn(mx));
    o4[1] = make_float4(__fdiv_rn(fs, fc), __fdiv_rn(u128_to_f32(v_hi, v_lo), __uint2float_rn(cnt * cnt)),
                        __uint2float_rn(first), __uint2float_rn(last));
}

// Groups: g0 size/all, g1 iat/all, g2 size/fwd, g3 size/bwd, g4 iat/fwd, g5 iat/bwd, g6 size/turn, g7 iat/turn.
// Sums of the backward subsets are (all - forward): exact, because everything is an integer.
template <int G>
__device__ __forceinline__ void packet(Acc (&A)[8], uint32_t sz, uint32_t ia, uint32_t i, uint32_t fwd_mask, uint32_t turn_mask) {
    const bool f = (fwd_mask >> i) & 1u;
    const bool tn = (turn_mask >> i) & 1u;
    add_size(A[0], sz, true);
    if (G > 1) add_iat(A[1], ia, true);
    if (G > 2) add_size(A[2], sz, f);
    if (G > 3) add_minmax(A[3], sz, !f);
    if (G > 4) add_iat(A[4], ia, f);
    if (G > 5) add_minmax(A[5], ia, !f);
    if (G > 6) add_size(A[6], sz, tn);
    if (G > 7) add_iat(A[7], ia, tn);
}

// VEC: row pitch is a multiple of 8 packets, so size rows are 16-byte aligned
// and inter-arrival rows 32-byte aligned.
template <int G, bool VEC>
__global__ void __launch_bounds__(kFlowsPerBlock)
extract_kernel(const uint16_t* __restrict__ size, const uint32_t* __restrict__ iat,
               const uint32_t* __restrict__ dir_bits, const uint8_t* __restrict__ n_valid,
               uint32_t n, uint32_t pitch, uint32_t N, float* __restrict__ feat, const uint32_t* __restrict__ n_dev,
               const uint32_t* __restrict__ row_ids)
{
    constexpr int F = 8 * G;
    constexpr int STRIDE = F + 4;                  // 16-byte aligned rows; 8 lanes x 16 B land in distinct bank groups
    extern __shared__ __align__(16) float tile[];                // [kFlowsPerBlock][STRIDE]
    if (n_dev) n = min(n, *n_dev);               // optional device-side flow count (streaming path)
    const uint32_t f0 = blockIdx.x * kFlowsPerBlock;
    if (f0 >= n) return;
    const uint32_t f = f0 + threadIdx.x;

    if (f < n) {
        const size_t fr = row_ids ? row_ids[f] : f;      // optional indirection: flow f's packets sit in row row_ids[f] of the planes
        Acc A[8];
#pragma unroll
        for (int g = 0; g < 8; g++) acc_init(A[g]);
        uint32_t m = N;
        if (n_valid) m = min(m, (uint32_t)n_valid[fr]);
        // N <= 32: all direction bits of the window are in the row's first word
        const uint32_t dirw = dir_bits[fr * ((pitch + 31) >> 5)];
        const uint32_t all_mask = (m >= 32) ? 0xFFFFFFFFu : ((1u << m) - 1u);
        const uint32_t fwd_mask = ~dirw & all_mask;
        const uint32_t bwd_mask = dirw & all_mask;
        const uint32_t turn_mask = (dirw ^ (dirw << 1)) & ~1u & all_mask;        // packet i >= 1 whose direction differs from i-1
        const uint16_t* srow = size + fr * pitch;
        const uint32_t* irow = iat + fr * pitch;
        if (VEC) {
            // issue every load of the window first (N <= 32: at most four chunks of eight packets), then reduce
            uint4 s4[4], a4[4], b4[4];
#pragma unroll
            for (int ch = 0; ch < 4; ch++) {
                if ((uint32_t)ch * 8 < m) {
                    s4[ch] = __ldg(reinterpret_cast<const uint4*>(srow + ch * 8));
                    a4[ch] = __ldg(reinterpret_cast<const uint4*>(irow + ch * 8));
                    b4[ch] = __ldg(reinterpret_cast<const uint4*>(irow + ch * 8 + 4));
                }
            }
#pragma unroll
            for (int ch = 0; ch < 4; ch++) {
                if ((uint32_t)ch * 8 < m) {
                    const uint32_t sz[8] = {s4[ch].x & 0xFFFFu, s4[ch].x >> 16, s4[ch].y & 0xFFFFu, s4[ch].y >> 16,
                                            s4[ch].z & 0xFFFFu, s4[ch].z >> 16, s4[ch].w & 0xFFFFu, s4[ch].w >> 16};
                    const uint32_t ia[8] = {a4[ch].x, a4[ch].y, a4[ch].z, a4[ch].w, b4[ch].x, b4[ch].y, b4[ch].z, b4[ch].w};
#pragma unroll
                    for (int j = 0; j < 8; j++)
                        if ((uint32_t)(ch * 8 + j) < m) packet<G>(A, sz[j], ia[j], ch * 8 + j, fwd_mask, turn_mask);
                }
            }
        } else {
            for (uint32_t i = 0; i < m; i++) packet<G>(A, srow[i], irow[i], i, fwd_mask, turn_mask);
        }
        float* o = tile + threadIdx.x * STRIDE;
#pragma unroll
        for (int g = 0; g < G; g++) {
            const uint32_t mask = (g < 2) ? all_mask : (g == 2 || g == 4) ? fwd_mask : (g == 3 || g == 5) ? bwd_mask : turn_mask;
            const bool is_size = (g == 0 || g == 2 || g == 3 || g == 6);
            const uint32_t cnt = __popc(mask);
            uint32_t first = 0, last = 0;
            if (cnt) {                               // the row was just read: these hit in L1
                const uint32_t i0 = __ffs(mask) - 1, i1 = 31 - __clz(mask);
                first = is_size ? (uint32_t)srow[i0] : irow[i0];
                last = is_size ? (uint32_t)srow[i1] : irow[i1];
            }
            uint64_t s1 = A[g].s1, s2lo = A[g].s2lo, s2hi = A[g].s2hi;
            if (g == 3 || g == 5) {                  // backward = all - forward
                const Acc& all = A[g == 3 ? 0 : 1];
                const Acc& fw = A[g == 3 ? 2 : 4];
                s1 = all.s1 - fw.s1;
                s2lo = all.s2lo - fw.s2lo;
                s2hi = (uint64_t)all.s2hi - fw.s2hi - ((all.s2lo < fw.s2lo) ? 1u : 0u);
            }
            finish(cnt, A[g].mn, A[g].mx, s1, s2lo, s2hi, first, last, o + 8 * g);
        }
    }
    __syncthreads();
    const uint32_t rows = min((uint32_t)kFlowsPerBlock, n - f0);
    const uint32_t total4 = rows * (F / 4);
    float4* dst = reinterpret_cast<float4*>(feat + (size_t)f0 * F);
    for (uint32_t e = threadIdx.x; e < total4; e += kFlowsPerBlock) {
        const uint32_t r = e / (F / 4), c = e - r * (F / 4);
        dst[e] = *reinterpret_cast<const float4*>(tile + r * STRIDE + 4 * c);
    }
}

template <int G>
int launch_g(const sf_packets* pk, uint32_t N, float* feat, cudaStream_t st, const uint32_t* n_dev, const uint32_t* row_ids) {
    const uint32_t n = pk->n_flows;
    const bool vec = (pk->pitch_pkts % 8 == 0) && (((uintptr_t)pk->size & 15) == 0) && (((uintptr_t)pk->iat_us & 15) == 0);
    const size_t smem = (size_t)kFlowsPerBlock * (8 * G + 4) * sizeof(float);
    const uint32_t grid = (n + kFlowsPerBlock - 1) / kFlowsPerBlock;
    if (vec)
        extract_kernel<G, true><<<grid, kFlowsPerBlock, smem, st>>>(pk->size, pk->iat_us, pk->dir_bits, pk->n_valid, n, pk->pitch_pkts, N, feat, n_dev, row_ids);
    else
        extract_kernel<G, false><<<grid, kFlowsPerBlock, smem, st>>>(pk->size, pk->iat_us, pk->dir_bits, pk->n_valid, n, pk->pitch_pkts, N, feat, n_dev, row_ids);
    SF_LAUNCH_CHECK("extract_kernel");
    return SF_OK;
}

}  // namespace

int sf_launch_extract(const sf_packets* pk, uint32_t N, uint32_t F, float* feat, cudaStream_t st, const uint32_t* n_dev,
                      const uint32_t* row_ids) {
    if (pk->n_flows == 0) return SF_OK;
    switch (F / 8) {
    case 1: return launch_g<1>(pk, N, feat, st, n_dev, row_ids);
    case 2: return launch_g<2>(pk, N, feat, st, n_dev, row_ids);
    case 3: return launch_g<3>(pk, N, feat, st, n_dev, row_ids);
    case 4: return launch_g<4>(pk, N, feat, st, n_dev, row_ids);
    case 5: return launch_g<5>(pk, N, feat, st, n_dev, row_ids);
    case 6: return launch_g<6>(pk, N, feat, st, n_dev, row_ids);
    case 7: return launch_g<7>(pk, N, feat, st, n_dev, row_ids);
    case 8: return launch_g<8>(pk, N, feat, st, n_dev, row_ids);
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

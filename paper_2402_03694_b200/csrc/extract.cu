// S1: per-flow statistical features of the first N packet headers.
//
// One thread per flow.  A thread loads its packets in chunks of 8 (16-byte vector loads of
// the uint16 sizes and uint32 inter-arrival times when the row pitch allows it; the next chunk
// is fetched while the current one is reduced, and the chunk loop is not unrolled, so that its
// body stays in the instruction cache and the register count stays below 100) and keeps one
// integer accumulator set per feature group in registers.  Subset membership (forward,
// backward, direction change) comes from the direction word: a packet's bit becomes one
// predicate per word, under which the subset's min, max and sums are updated without selects
// or branches.  The 96-bit sum of squared inter-arrival times is kept as two 64-bit sums (of
// the low and of the high words of the 64-bit squares) and joined at the end.  Counts, first
// and last come from the masks (popcount / lowest / highest set bit).  Sums of the backward
// subsets are (all - forward): exact, because everything is an integer.
// Each fp32 value is produced by exactly one rounding (integer -> fp32 RNE) or one IEEE
// division, so results are reproducible bit for bit.  The block hands its [flows][F] tile to
// global memory through shared memory so that the stores are fully coalesced.
// The kernel is bound by integer issue, not by HBM: min/max/add/logic and the multiply-adds run on
// two half-rate pipes, and a 64-bit accumulation costs three instructions on this target.
#include "extract_device.cuh"

namespace {

constexpr int kFlowsPerBlock = 32;       // one warp per block: small blocks schedule better here than 64- or 128-flow ones (measured)

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
        uint32_t m = N;
        if (n_valid) m = min(m, (uint32_t)n_valid[fr]);
        // N <= 32: all direction bits of the window are in the row's first word
        const uint32_t dirw = dir_bits[fr * ((pitch + 31) >> 5)];
        sfx::extract_flow<G, VEC>(size, iat, fr, pitch, m, dirw, sfx::RowOut{tile + threadIdx.x * STRIDE});
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

// S3: uncertainty score + threshold + ordered compaction + wide-row gather, and
// S5: merge of fast and slow answers.
//
// Four small kernels on one stream, no host round trip:
//   score_kernel   per flow: argmax, score (least confidence or |margin|), decision;
//                  per 1024-flow block the number of assigned flows
//   scan_kernel    one block: exclusive scan of the block counts, total -> n_esc
//   scatter_kernel per block: ballot + popc ranks -> ascending flow ids
//   gather_kernel  one warp per assigned flow: header planes -> scaled fields ->
//                  bf16 (RNE) or fp32 row, 16-byte stores, 1 KB contiguous per warp pass
#include "common.cuh"

namespace {

constexpr int kScoreBlock = 1024;

template <int RULE>
__global__ void __launch_bounds__(kScoreBlock)
score_kernel(const float* __restrict__ fast_out, uint32_t n, uint32_t C, const float* __restrict__ tau,
             uint8_t* __restrict__ decision, uint8_t* __restrict__ label, float* __restrict__ score,
             uint32_t* __restrict__ block_counts, const uint32_t* __restrict__ n_dev = nullptr)
{
    __shared__ uint32_t warp_cnt[kScoreBlock / 32];
    if (n_dev) n = min(n, *n_dev);               // optional device-side flow count (streaming path)
    const uint32_t f = blockIdx.x * kScoreBlock + threadIdx.x;
    bool esc = false;
    if (f < n) {
        float u; uint32_t a;
        if (RULE == SF_ABSMARGIN_LT) {
            float m = fast_out[f];
            u = fabsf(m);
            a = (m > 0.0f) ? 1u : 0u;
            esc = u < __ldg(tau);
        } else {
            const float* p = fast_out + (size_t)f * C;
            float mx = p[0]; a = 0;
            for (uint32_t c = 1; c < C; c++) { float v = p[c]; if (v > mx) { mx = v; a = c; } }
            if (RULE == SF_ENTROPY_GT) {
                // H = -sum p ln p (Sec. 3.2); fp32 logf, so this score is compared by tolerance, not bit for bit
                float h = 0.0f;
                for (uint32_t c = 0; c < C; c++) { float v = p[c]; if (v > 0.0f) h -= v * logf(v); }
                u = h;
            } else if (RULE == SF_SOFTMAX_LC_GT) {
                // least confidence of softmax(margins): 1 - 1 / sum_j exp(m_j - m_max); fp32 expf, compared by tolerance
                float sum = 0.0f;
                for (uint32_t c = 0; c < C; c++) sum += expf(p[c] - mx);
                u = 1.0f - 1.0f / sum;
            } else {
                u = __fsub_rn(1.0f, mx);
            }
            esc = u > __ldg(tau + a);
        }
        if (decision) decision[f] = esc ? 1 : 0;
        if (label) label[f] = (uint8_t)a;
        if (score) score[f] = u;
    }
    uint32_t b = __ballot_sync(0xFFFFFFFFu, esc);
    if ((threadIdx.x & 31) == 0) warp_cnt[threadIdx.x >> 5] = __popc(b);
    __syncthreads();
    if (threadIdx.x < 32) {
        uint32_t v = warp_cnt[threadIdx.x];
#pragma unroll
        for (int o = 16; o > 0; o >>= 1) v += __shfl_xor_sync(0xFFFFFFFFu, v, o);
        if (threadIdx.x == 0) block_counts[blockIdx.x] = v;
    }
}

// exclusive scan of nb block counts in place; total (clamped) -> *n_esc and the state block
__global__ void __launch_bounds__(1024)
scan_kernel(uint32_t* __restrict__ block_counts, uint32_t nb, uint32_t n, uint32_t capacity,
            uint32_t* __restrict__ n_esc, sf_dev_state* __restrict__ st, const uint32_t* __restrict__ n_dev = nullptr)
{
    sf_chain_enter();
    if (n_dev) n = min(n, *n_dev);               // flows actually scored (blocks past the count contributed zeros)
    __shared__ uint32_t warp_sum[32];
    __shared__ uint32_t carry_s;
    if (threadIdx.x == 0) carry_s = 0;
    __syncthreads();
    for (uint32_t base = 0; base < nb; base += 1024) {
        uint32_t i = base + threadIdx.x;
        uint32_t v = (i < nb) ? block_counts[i] : 0u;
        uint32_t x = v;
#pragma unroll
        for (int o = 1; o < 32; o <<= 1) { uint32_t y = __shfl_up_sync(0xFFFFFFFFu, x, o); if ((threadIdx.x & 31) >= o) x += y; }
        if ((threadIdx.x & 31) == 31) warp_sum[threadIdx.x >> 5] = x;
        __syncthreads();
        if (threadIdx.x < 32) {
            uint32_t w = warp_sum[threadIdx.x], z = w;
#pragma unroll
            for (int o = 1; o < 32; o <<= 1) { uint32_t y = __shfl_up_sync(0xFFFFFFFFu, z, o); if (threadIdx.x >= o) z += y; }
            warp_sum[threadIdx.x] = z - w;          // exclusive over warps
        }
        __syncthreads();
        uint32_t carry = carry_s;
        uint32_t excl = carry + warp_sum[threadIdx.x >> 5] + x - v;
        if (i < nb) block_counts[i] = excl;
        __syncthreads();
        if (threadIdx.x == 1023) carry_s = excl + v;
        __syncthreads();
    }
    if (threadIdx.x == 0) {
        uint32_t total = carry_s;
        if (total > capacity) { sf_dev_set_error(st, SF_ERR_CAPACITY); total = capacity; }
        if (n_esc) *n_esc = total;
        st->scan_total = total;
        atomicAdd((unsigned long long*)&st->counters.n_flows, (unsigned long long)n);
        atomicAdd((unsigned long long*)&st->counters.n_escalated, (unsigned long long)total);
        atomicAdd((unsigned long long*)&st->counters.n_fast_done, (unsigned long long)(n - total));
    }
}

// B = flows per block = the granularity of the block counts (1024 after score_kernel, 512 after a tree kernel that took
// the decisions itself)
template <int B>
__global__ void __launch_bounds__(B)
scatter_kernel(const uint8_t* __restrict__ decision, uint32_t n, const uint32_t* __restrict__ block_offsets,
               uint32_t capacity, uint32_t* __restrict__ esc_ids, const uint32_t* __restrict__ n_dev = nullptr)
{
    sf_chain_enter();
    if (n_dev) n = min(n, *n_dev);
    __shared__ uint32_t warp_off[32];
    const uint32_t f = blockIdx.x * B + threadIdx.x;
    const bool esc = (f < n) && decision[f] != 0;
    const uint32_t b = __ballot_sync(0xFFFFFFFFu, esc);
    const uint32_t lane = threadIdx.x & 31;
    if (lane == 0) warp_off[threadIdx.x >> 5] = __popc(b);
    __syncthreads();
    if (threadIdx.x < 32) {
        uint32_t w = (threadIdx.x < B / 32) ? warp_off[threadIdx.x] : 0u, z = w;
#pragma unroll
        for (int o = 1; o < 32; o <<= 1) { uint32_t y = __shfl_up_sync(0xFFFFFFFFu, z, o); if (threadIdx.x >= o) z += y; }
        warp_off[threadIdx.x] = z - w;
    }
    __syncthreads();
    if (esc) {
        uint32_t pos = block_offsets[blockIdx.x] + warp_off[threadIdx.x >> 5] + __popc(b & ((1u << lane) - 1u));
        if (pos < capacity) esc_ids[pos] = f;
    }
}

// integer piecewise-linear log2 of (a + 1): 4 * floor(log2 v) + the two bits below the leading one
__device__ __forceinline__ uint32_t ilog4(uint32_t a) {
    uint64_t v = (uint64_t)a + 1ull;
    uint32_t e = 63u - (uint32_t)__clzll((long long)v);
    uint64_t two = (e >= 2) ? (v >> (e - 2)) : (v << (2 - e));
    return 4u * e + (uint32_t)(two & 3ull);
}

__device__ __forceinline__ uint32_t pack_bf16(float lo, float hi) {
    __nv_bfloat162 v = __floats2bfloat162_rn(lo, hi);       // RNE, .x = lo (low half)
    return *reinterpret_cast<uint32_t*>(&v);
}

// W = fields per packet (16: size, L, dir, 13 header bytes; 8: size, L, dir, 5 header bytes)
// HW: the header plane starts on a 4-byte boundary, so a packet's NH header bytes are fetched as the
// aligned 32-bit words that contain them (4 loads instead of 13 for the 16-field row) and moved into
// place with funnel shifts; only the plane's last, partial word is assembled from byte loads.
template <int W, bool BF16, bool HW>
__global__ void __launch_bounds__(256)
gather_kernel(const uint32_t* __restrict__ esc_ids, const uint32_t* __restrict__ n_esc_dev,
              const uint16_t* __restrict__ size, const uint32_t* __restrict__ iat,
              const uint32_t* __restrict__ dir_bits, const uint8_t* __restrict__ hdr,
              const uint8_t* __restrict__ n_valid, uint32_t pitch, uint32_t hdr_bytes, size_t hdr_total,
              uint32_t P, uint32_t P_real, void* __restrict__ rows)
{
    constexpr int NH = W - 3;
    constexpr int NW = (NH + 6) / 4;             // words that can hold NH bytes starting at any byte of the first
    sf_chain_enter();
    const uint32_t n_esc = *n_esc_dev;
    const uint32_t lane = threadIdx.x & 31;
    const uint32_t warps = (gridDim.x * blockDim.x) >> 5;
    const uint32_t words = (pitch + 31) >> 5;
    for (uint32_t r = (blockIdx.x * blockDim.x + threadIdx.x) >> 5; r < n_esc; r += warps) {
        const uint32_t f = esc_ids[r];
        uint32_t m = P_real;
        if (n_valid) m = min(m, (uint32_t)n_valid[f]);
        const size_t row0 = (size_t)f * pitch;
        // PPL packets per lane so that a lane writes 32 contiguous bytes of bf16 (one packet of 16 fields, two of 8): a warp pass
        // then covers 1 KB of the row whatever the layout
        constexpr int PPL = (BF16 && W == 8) ? 2 : 1;
        for (uint32_t i0 = lane * PPL; i0 < P; i0 += 32 * PPL) {
#pragma unroll
          for (int q = 0; q < PPL; q++) {
            const uint32_t i = i0 + q;
            if (PPL > 1 && i >= P) break;
            float v[W];
            if (i < m) {
                v[0] = __fmul_rn(__uint2float_rn((uint32_t)size[row0 + i]), 0x1p-11f);
                v[1] = __fmul_rn(__uint2float_rn(ilog4(iat[row0 + i])), 0x1p-7f);
                v[2] = (float)((dir_bits[(size_t)f * words + (i >> 5)] >> (i & 31)) & 1u);
                if (HW) {
                    const size_t boff = (row0 + i) * hdr_bytes;
                    const size_t w0 = boff >> 2;
                    const uint32_t sh = (uint32_t)(boff & 3) * 8u;
                    uint32_t raw[NW + 1];
#pragma unroll
                    for (int j = 0; j < NW; j++) {
                        const size_t a = (w0 + j) * 4;
                        if (a + 4 <= hdr_total) {
                            raw[j] = __ldg(reinterpret_cast<const uint32_t*>(hdr) + w0 + j);
                        } else {                         // the plane's last bytes: never read past its end
                            raw[j] = 0;
                            for (uint32_t b = 0; b < 4; b++) if (a + b < hdr_total) raw[j] |= (uint32_t)hdr[a + b] << (8 * b);
                        }
                    }
                    raw[NW] = 0;
#pragma unroll
                    for (int k = 0; k < NH; k++) {
                        const uint32_t al = __funnelshift_r(raw[k / 4], raw[k / 4 + 1], sh);      // bytes k/4*4 .. +3 of the packet's header
                        v[3 + k] = __fmul_rn(__uint2float_rn((al >> (8 * (k % 4))) & 0xFFu), 0x1p-8f);
                    }
                } else {
                    const uint8_t* h = hdr + (row0 + i) * hdr_bytes;
#pragma unroll
                    for (int k = 0; k < NH; k++) v[3 + k] = __fmul_rn(__uint2float_rn((uint32_t)h[k]), 0x1p-8f);
                }
            } else {
#pragma unroll
                for (int k = 0; k < W; k++) v[k] = 0.0f;
            }
            if (BF16) {
                uint4* dst = reinterpret_cast<uint4*>(reinterpret_cast<__nv_bfloat16*>(rows) + ((size_t)r * P + i) * W);
#pragma unroll
                for (int q4 = 0; q4 < W / 8; q4++)
                    dst[q4] = make_uint4(pack_bf16(v[8 * q4], v[8 * q4 + 1]), pack_bf16(v[8 * q4 + 2], v[8 * q4 + 3]),
                                         pack_bf16(v[8 * q4 + 4], v[8 * q4 + 5]), pack_bf16(v[8 * q4 + 6], v[8 * q4 + 7]));
            } else {
                float4* dst = reinterpret_cast<float4*>(reinterpret_cast<float*>(rows) + ((size_t)r * P + i) * W);
#pragma unroll
                for (int q4 = 0; q4 < W / 4; q4++) dst[q4] = make_float4(v[4 * q4], v[4 * q4 + 1], v[4 * q4 + 2], v[4 * q4 + 3]);
            }
          }
        }
    }
}

__global__ void merge_fast_kernel(const uint8_t* __restrict__ label_fast, const uint8_t* __restrict__ decision,
                                  uint32_t n, uint8_t* __restrict__ label, uint8_t* __restrict__ stage)
{
    uint32_t f = blockIdx.x * blockDim.x + threadIdx.x;
    if (f >= n) return;
    // every flow starts with the fast answer; assigned flows are overwritten by merge_slow_kernel
    if (label) label[f] = label_fast[f];
    if (stage) stage[f] = 1;
}

__global__ void merge_slow_kernel(const uint32_t* __restrict__ esc_ids, const uint32_t* __restrict__ n_esc_dev,
                                  const uint8_t* __restrict__ label_slow, uint8_t* __restrict__ label,
                                  uint8_t* __restrict__ stage, uint8_t stage_value, sf_dev_state* count_slow_done)
{
    sf_chain_enter();
    const uint32_t n_esc = *n_esc_dev;
    if (count_slow_done && blockIdx.x == 0 && threadIdx.x == 0)
        atomicAdd((unsigned long long*)&count_slow_done->counters.n_slow_done, (unsigned long long)n_esc);
    for (uint32_t r = blockIdx.x * blockDim.x + threadIdx.x; r < n_esc; r += gridDim.x * blockDim.x) {
        uint32_t f = esc_ids[r];
        if (label) label[f] = label_slow[r];
        if (stage) stage[f] = stage_value;
    }
}

// rows of feat picked by an id list (count on the device): out[r][:] = feat[ids[r]][:]
__global__ void gather_feat_kernel(const float* __restrict__ feat, const uint32_t* __restrict__ ids,
                                   const uint32_t* __restrict__ n_dev, uint32_t F4, float4* __restrict__ out)
{
    const uint32_t e = blockIdx.x * blockDim.x + threadIdx.x;
    const uint32_t r = e / F4, c = e - r * F4;
    if (r >= *n_dev) return;
    out[e] = reinterpret_cast<const float4*>(feat)[(size_t)ids[r] * F4 + c];
}

// ids of the second list are positions in the first: out[r] = ids1[ids2_local[r]]
__global__ void compose_ids_kernel(const uint32_t* __restrict__ ids1, const uint32_t* __restrict__ ids2_local,
                                   const uint32_t* __restrict__ n_dev, uint32_t* __restrict__ out)
{
    const uint32_t r = blockIdx.x * blockDim.x + threadIdx.x;
    if (r < *n_dev) out[r] = ids1[ids2_local[r]];
}

}  // namespace

// score / label / decision only (no compaction), for at most n flows with the actual count on the device
int sf_launch_score(const sf_route_cfg* cfg, const float* fast_out, uint32_t n, uint32_t C, uint8_t* decision,
                    uint8_t* label, float* score, uint32_t* block_counts, const uint32_t* n_dev, cudaStream_t st)
{
    const uint32_t nb = (n + kScoreBlock - 1) / kScoreBlock;
    if (nb == 0) return SF_OK;
    if (cfg->rule == SF_ABSMARGIN_LT)
        score_kernel<SF_ABSMARGIN_LT><<<nb, kScoreBlock, 0, st>>>(fast_out, n, C, cfg->tau, decision, label, score, block_counts, n_dev);
    else if (cfg->rule == SF_ENTROPY_GT)
        score_kernel<SF_ENTROPY_GT><<<nb, kScoreBlock, 0, st>>>(fast_out, n, C, cfg->tau, decision, label, score, block_counts, n_dev);
    else if (cfg->rule == SF_SOFTMAX_LC_GT)
        score_kernel<SF_SOFTMAX_LC_GT><<<nb, kScoreBlock, 0, st>>>(fast_out, n, C, cfg->tau, decision, label, score, block_counts, n_dev);
    else
        score_kernel<SF_LC_GT><<<nb, kScoreBlock, 0, st>>>(fast_out, n, C, cfg->tau, decision, label, score, block_counts, n_dev);
    SF_LAUNCH_CHECK("score_kernel");
    return SF_OK;
}

namespace { __global__ void iota_kernel(uint32_t* out, uint32_t n) { uint32_t i = blockIdx.x * blockDim.x + threadIdx.x; if (i < n) out[i] = i; } }
int sf_launch_iota(uint32_t* out, uint32_t n, cudaStream_t st) {
    if (n == 0) return SF_OK;
    iota_kernel<<<(n + 255) / 256, 256, 0, st>>>(out, n);
    SF_LAUNCH_CHECK("iota_kernel");
    return SF_OK;
}

int sf_launch_gather_feat(const float* feat, const uint32_t* ids, const uint32_t* n_dev, uint32_t n_max, uint32_t F,
                          float* out, cudaStream_t st)
{
    if (n_max == 0) return SF_OK;
    const uint32_t F4 = F / 4;
    const size_t total = (size_t)n_max * F4;
    gather_feat_kernel<<<(uint32_t)((total + 255) / 256), 256, 0, st>>>(feat, ids, n_dev, F4, reinterpret_cast<float4*>(out));
    SF_LAUNCH_CHECK("gather_feat_kernel");
    return SF_OK;
}
int sf_launch_compose_ids(const uint32_t* ids1, const uint32_t* ids2_local, const uint32_t* n_dev, uint32_t n_max,
                          uint32_t* out, cudaStream_t st)
{
    if (n_max == 0) return SF_OK;
    compose_ids_kernel<<<(n_max + 255) / 256, 256, 0, st>>>(ids1, ids2_local, n_dev, out);
    SF_LAUNCH_CHECK("compose_ids_kernel");
    return SF_OK;
}

// wide rows of `capacity` flows at most (ids and count on the device) out of any planes
int sf_launch_gather(sf_ctx* ctx, const sf_route_cfg* cfg, const sf_packets* wide, const uint32_t* ids,
                     const uint32_t* n_ids_dev, uint32_t capacity, void* rows, cudaStream_t st)
{
    if (capacity == 0) return SF_OK;
    const uint32_t P = cfg->P, P_real = cfg->P_real ? cfg->P_real : cfg->P;
    uint32_t blocks = (capacity + 7) / 8;
    uint32_t max_blocks = (uint32_t)ctx->num_sms * 32;
    if (blocks > max_blocks) blocks = max_blocks;
    const size_t hdr_total = (size_t)wide->n_flows * wide->pitch_pkts * wide->hdr_bytes;
    const bool hdr_words = ((uintptr_t)wide->hdr & 3) == 0;
#define SF_GATHER2(Wv, BF) do { if (hdr_words) SF_CUDA(sf_launch_chained(gather_kernel<Wv, BF, true>, blocks, 256, 0, st, ids, n_ids_dev, wide->size, wide->iat_us, wide->dir_bits, wide->hdr, wide->n_valid, wide->pitch_pkts, wide->hdr_bytes, hdr_total, P, P_real, rows)); \
        else SF_CUDA(sf_launch_chained(gather_kernel<Wv, BF, false>, blocks, 256, 0, st, ids, n_ids_dev, wide->size, wide->iat_us, wide->dir_bits, wide->hdr, wide->n_valid, wide->pitch_pkts, wide->hdr_bytes, hdr_total, P, P_real, rows)); } while (0)
    if (cfg->wide_layout == SF_MLP16) { if (cfg->row_dtype == SF_BF16) SF_GATHER2(16, true); else SF_GATHER2(16, false); }
    else                              { if (cfg->row_dtype == SF_BF16) SF_GATHER2(8, true);  else SF_GATHER2(8, false); }
#undef SF_GATHER2
    SF_LAUNCH_CHECK("gather_kernel");
    return SF_OK;
}

size_t sf_route_scratch_bytes(uint32_t n) {
    size_t nb = ((size_t)n + SF_FOREST_BLOCK - 1) / SF_FOREST_BLOCK;               // the finer of the two block-count granularities
    return sf_align256((nb + 1) * sizeof(uint32_t)) + sf_align256((size_t)n);      // block counts + decision bytes
}

int sf_launch_route(sf_ctx* ctx, const sf_route_cfg* cfg, const float* fast_out, uint32_t n, uint32_t C,
                    const sf_packets* wide, uint32_t* esc_ids, uint32_t* n_esc, void* rows,
                    uint8_t* decision, uint8_t* label_fast, float* score, void* scratch, cudaStream_t st,
                    const uint32_t* n_dev)
{
    const uint32_t nb = (n + kScoreBlock - 1) / kScoreBlock;
    uint32_t* block_counts = reinterpret_cast<uint32_t*>(scratch);
    uint8_t* dec = decision ? decision
                            : reinterpret_cast<uint8_t*>(scratch) + sf_align256(((size_t)nb + 1) * sizeof(uint32_t));
    sf_time_begin(ctx, SF_T_SCORE, st);
    if (n > 0) {
        if (cfg->rule == SF_ABSMARGIN_LT)
            score_kernel<SF_ABSMARGIN_LT><<<nb, kScoreBlock, 0, st>>>(fast_out, n, C, cfg->tau, dec, label_fast, score, block_counts, n_dev);
        else if (cfg->rule == SF_ENTROPY_GT)
            score_kernel<SF_ENTROPY_GT><<<nb, kScoreBlock, 0, st>>>(fast_out, n, C, cfg->tau, dec, label_fast, score, block_counts, n_dev);
        else if (cfg->rule == SF_SOFTMAX_LC_GT)
            score_kernel<SF_SOFTMAX_LC_GT><<<nb, kScoreBlock, 0, st>>>(fast_out, n, C, cfg->tau, dec, label_fast, score, block_counts, n_dev);
        else
            score_kernel<SF_LC_GT><<<nb, kScoreBlock, 0, st>>>(fast_out, n, C, cfg->tau, dec, label_fast, score, block_counts, n_dev);
        SF_LAUNCH_CHECK("score_kernel");
    }
    scan_kernel<<<1, 1024, 0, st>>>(block_counts, nb, n, cfg->capacity, n_esc, ctx->d_state, n_dev);
    SF_LAUNCH_CHECK("scan_kernel");
    if (n > 0) {
        scatter_kernel<kScoreBlock><<<nb, kScoreBlock, 0, st>>>(dec, n, block_counts, cfg->capacity, esc_ids, n_dev);
        SF_LAUNCH_CHECK("scatter_kernel");
    }
    sf_time_end(ctx, SF_T_SCORE, st);
    if (wide && rows && n > 0 && cfg->capacity > 0) {
        const uint32_t P = cfg->P, P_real = cfg->P_real ? cfg->P_real : cfg->P;
        // enough warps to cover the capacity, at most a few waves of resident blocks
        uint32_t blocks = (cfg->capacity + 7) / 8;
        uint32_t max_blocks = (uint32_t)ctx->num_sms * 32;
        if (blocks > max_blocks) blocks = max_blocks;
        const uint32_t* cnt = &ctx->d_state->scan_total;
        const size_t hdr_total = (size_t)wide->n_flows * wide->pitch_pkts * wide->hdr_bytes;
        const bool hdr_words = ((uintptr_t)wide->hdr & 3) == 0;
        sf_time_begin(ctx, SF_T_GATHER, st);
#define SF_GATHER(Wv, BF) do { if (hdr_words) gather_kernel<Wv, BF, true><<<blocks, 256, 0, st>>>(esc_ids, cnt, wide->size, wide->iat_us, wide->dir_bits, wide->hdr, wide->n_valid, wide->pitch_pkts, wide->hdr_bytes, hdr_total, P, P_real, rows); \
        else gather_kernel<Wv, BF, false><<<blocks, 256, 0, st>>>(esc_ids, cnt, wide->size, wide->iat_us, wide->dir_bits, wide->hdr, wide->n_valid, wide->pitch_pkts, wide->hdr_bytes, hdr_total, P, P_real, rows); } while (0)
        if (cfg->wide_layout == SF_MLP16) { if (cfg->row_dtype == SF_BF16) SF_GATHER(16, true); else SF_GATHER(16, false); }
        else                              { if (cfg->row_dtype == SF_BF16) SF_GATHER(8, true);  else SF_GATHER(8, false); }
#undef SF_GATHER
        SF_LAUNCH_CHECK("gather_kernel");
        sf_time_end(ctx, SF_T_GATHER, st);
    }
    return SF_OK;
}

int sf_launch_route_after_fused(sf_ctx* ctx, const sf_route_cfg* cfg, uint32_t n, const sf_packets* wide, uint32_t* esc_ids,
                                uint32_t* n_esc, void* rows, const uint8_t* decision, uint32_t* block_counts, cudaStream_t st)
{
    const uint32_t nb = (n + SF_FOREST_BLOCK - 1) / SF_FOREST_BLOCK;
    sf_time_begin(ctx, SF_T_SCORE, st);
    SF_CUDA(sf_launch_chained(scan_kernel, 1, 1024, 0, st, block_counts, nb, n, cfg->capacity, n_esc, ctx->d_state, (const uint32_t*)nullptr));
    if (n > 0)
        SF_CUDA(sf_launch_chained(scatter_kernel<(int)SF_FOREST_BLOCK>, nb, SF_FOREST_BLOCK, 0, st, decision, n, (const uint32_t*)block_counts, cfg->capacity,
                                  esc_ids, (const uint32_t*)nullptr));
    sf_time_end(ctx, SF_T_SCORE, st);
    if (wide && rows && n > 0 && cfg->capacity > 0) {
        sf_time_begin(ctx, SF_T_GATHER, st);
        int rc = sf_launch_gather(ctx, cfg, wide, esc_ids, &ctx->d_state->scan_total, cfg->capacity, rows, st);
        sf_time_end(ctx, SF_T_GATHER, st);
        if (rc != SF_OK) return rc;
    }
    return SF_OK;
}

int sf_launch_merge(const uint8_t* label_fast, const uint8_t* decision, uint32_t n, const uint32_t* esc_ids,
                    const uint32_t* n_esc, uint32_t capacity, const uint8_t* label_slow,
                    uint8_t* label, uint8_t* stage, cudaStream_t st, uint8_t stage_value, bool write_fast, sf_dev_state* count_slow_done)
{
    if (n == 0) return SF_OK;
    if (write_fast)
    merge_fast_kernel<<<(n + 255) / 256, 256, 0, st>>>(label_fast, decision, n, label, stage);
    if (write_fast) SF_LAUNCH_CHECK("merge_fast_kernel");
    uint32_t blocks = (capacity + 255) / 256;
    if (blocks > 1184) blocks = 1184;
    if (blocks > 0) {
        SF_CUDA(sf_launch_chained(merge_slow_kernel, blocks, 256, 0, st, esc_ids, n_esc, label_slow, label, stage, stage_value, count_slow_done));
    }
    return SF_OK;
}

extern "C" int sf_route(sf_ctx* ctx, const sf_route_cfg* cfg, const float* fast_out, uint32_t n, uint32_t C,
                        const sf_packets* wide, uint32_t* esc_ids_out, uint32_t* n_esc_out, void* rows_out,
                        uint8_t* decision_out, uint8_t* label_fast_out, float* score_out, void* stream)
{
    if (!ctx || !cfg || !fast_out || !esc_ids_out || !n_esc_out || !cfg->tau) return SF_ERR_ARG;
    if (cfg->rule != SF_LC_GT && cfg->rule != SF_ABSMARGIN_LT && cfg->rule != SF_ENTROPY_GT && cfg->rule != SF_SOFTMAX_LC_GT) return SF_ERR_ARG;
    if (cfg->rule != SF_ABSMARGIN_LT && (C < 1 || C > 256)) return SF_ERR_ARG;
    if (rows_out) {
        if (!wide || !wide->size || !wide->iat_us || !wide->dir_bits || !wide->hdr) return SF_ERR_ARG;
        if (cfg->wide_layout != SF_MLP16 && cfg->wide_layout != SF_CNN8) return SF_ERR_ARG;
        if (cfg->row_dtype != SF_BF16 && cfg->row_dtype != SF_F32) return SF_ERR_ARG;
        uint32_t need_h = cfg->wide_layout == SF_MLP16 ? 13u : 5u;
        uint32_t P_real = cfg->P_real ? cfg->P_real : cfg->P;
        if (wide->hdr_bytes < need_h || cfg->P == 0 || P_real > cfg->P || P_real > wide->pitch_pkts) return SF_ERR_ARG;
        if (wide->n_flows < n) return SF_ERR_ARG;
        if (((uintptr_t)rows_out & 15) != 0) return SF_ERR_ARG;
    }
    SF_CUDA(cudaSetDevice(ctx->device));
    int rc = sf_ws_reserve(ctx, sf_route_scratch_bytes(n));
    if (rc != SF_OK) return rc;
    sf_ws_reset(ctx);
    void* scratch = sf_ws_alloc(ctx, sf_route_scratch_bytes(n));
    if (!scratch) return SF_ERR_ALLOC;
    sf_time_new_record(ctx);
    return sf_launch_route(ctx, cfg, fast_out, n, C, rows_out ? wide : nullptr, esc_ids_out, n_esc_out, rows_out,
                           decision_out, label_fast_out, score_out, scratch, (cudaStream_t)stream);
}

// ---- allocation-free variant of the assignment step --------------------------------
// Scratch for sf_route_noalloc: one state block, the per-block counts and one decision
// byte per flow.  It lives in the library image, so every GPU that loads the library
// holds these bytes until the process exits.
namespace {
constexpr uint32_t kNoAllocBlocks = SF_NOALLOC_MAX_FLOWS / kScoreBlock;
struct NoAllocScratch {
    sf_dev_state state;
    uint32_t block_counts[kNoAllocBlocks + 64];
    uint8_t decision[SF_NOALLOC_MAX_FLOWS];
};
}  // namespace

static __device__ __align__(256) unsigned char g_noalloc_scratch[sizeof(NoAllocScratch)];

namespace {
constexpr int kMaxDevices = 64;
NoAllocScratch* g_noalloc_ptr[kMaxDevices] = {};

__global__ void noalloc_report_kernel(const sf_dev_state* st, int32_t* status_out) {
    *status_out = st->counters.device_error;
}
}  // namespace

extern "C" int sf_route_noalloc(int device, const sf_route_cfg* cfg, const float* fast_out, uint32_t n, uint32_t C,
                                uint32_t* esc_ids_out, uint32_t* n_esc_out, uint8_t* decision_out,
                                uint8_t* label_fast_out, float* score_out, int32_t* status_out, void* stream)
{
    if (!cfg || !fast_out || !esc_ids_out || !n_esc_out || !cfg->tau) return SF_ERR_ARG;
    if (cfg->rule != SF_LC_GT && cfg->rule != SF_ABSMARGIN_LT && cfg->rule != SF_ENTROPY_GT && cfg->rule != SF_SOFTMAX_LC_GT) return SF_ERR_ARG;
    if (cfg->rule != SF_ABSMARGIN_LT && (C < 1 || C > 256)) return SF_ERR_ARG;
    if (device < 0 || device >= kMaxDevices) return SF_ERR_ARG;
    if (n > SF_NOALLOC_MAX_FLOWS) return SF_ERR_STATIC_LIMIT;
    SF_CUDA(cudaSetDevice(device));
    if (!g_noalloc_ptr[device]) {
        // In host code the array's name is only a handle; the device address has to be asked for,
        // once per device, with that device current.  Two threads that make their first call on a device
        // at the same time both store the same address here, so the unsynchronised write is harmless.
        void* p = nullptr;
        SF_CUDA(cudaGetSymbolAddress(&p, g_noalloc_scratch));
        g_noalloc_ptr[device] = reinterpret_cast<NoAllocScratch*>(p);
    }
    NoAllocScratch* sc = g_noalloc_ptr[device];
    cudaStream_t st = (cudaStream_t)stream;
    // the array keeps whatever the previous call left: the state block must start at zero
    SF_CUDA(cudaMemsetAsync(&sc->state, 0, sizeof(sf_dev_state), st));
    const uint32_t nb = (n + kScoreBlock - 1) / kScoreBlock;
    uint8_t* dec = decision_out ? decision_out : sc->decision;
    if (n > 0) {
        if (cfg->rule == SF_ABSMARGIN_LT)
            score_kernel<SF_ABSMARGIN_LT><<<nb, kScoreBlock, 0, st>>>(fast_out, n, C, cfg->tau, dec, label_fast_out, score_out, sc->block_counts);
        else if (cfg->rule == SF_ENTROPY_GT)
            score_kernel<SF_ENTROPY_GT><<<nb, kScoreBlock, 0, st>>>(fast_out, n, C, cfg->tau, dec, label_fast_out, score_out, sc->block_counts);
        else if (cfg->rule == SF_SOFTMAX_LC_GT)
            score_kernel<SF_SOFTMAX_LC_GT><<<nb, kScoreBlock, 0, st>>>(fast_out, n, C, cfg->tau, dec, label_fast_out, score_out, sc->block_counts);
        else
            score_kernel<SF_LC_GT><<<nb, kScoreBlock, 0, st>>>(fast_out, n, C, cfg->tau, dec, label_fast_out, score_out, sc->block_counts);
        SF_LAUNCH_CHECK("score_kernel");
    }
    scan_kernel<<<1, 1024, 0, st>>>(sc->block_counts, nb, n, cfg->capacity, n_esc_out, &sc->state);
    SF_LAUNCH_CHECK("scan_kernel");
    if (n > 0) {
        scatter_kernel<kScoreBlock><<<nb, kScoreBlock, 0, st>>>(dec, n, sc->block_counts, cfg->capacity, esc_ids_out);
        SF_LAUNCH_CHECK("scatter_kernel");
    }
    if (status_out) {
        noalloc_report_kernel<<<1, 1, 0, st>>>(&sc->state, status_out);
        SF_LAUNCH_CHECK("noalloc_report_kernel");
    }
    return SF_OK;
}

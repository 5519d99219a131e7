// First-packet header-bit features: the subscribed columns of the 1024 header bits of a packet
// (IPv4 60 B | TCP 60 B | UDP 8 B) as -1 (byte not present) / 0 / 1.
// A block stages 64 packet rows (8 KB, 16-byte coalesced loads), the section lengths and the
// subscription list in shared memory and writes its [64][m] tile with coalesced stores.
#include "common.cuh"

namespace {

constexpr uint32_t kRows = 64;

__global__ void __launch_bounds__(256)
header_bits_kernel(const uint8_t* __restrict__ bytes, const uint8_t* __restrict__ sec_len, uint32_t n,
                   const uint16_t* __restrict__ sub, uint32_t m, float* __restrict__ out)
{
    __shared__ __align__(16) uint8_t rows[kRows * 128];
    __shared__ uint8_t lens[kRows * 3];
    __shared__ uint16_t cols[1024];
    const uint32_t f0 = blockIdx.x * kRows;
    const uint32_t nr = min(kRows, n - f0);
    const uint4* src = reinterpret_cast<const uint4*>(bytes + (size_t)f0 * 128);
    for (uint32_t v = threadIdx.x; v < nr * 8; v += blockDim.x) reinterpret_cast<uint4*>(rows)[v] = __ldg(src + v);
    for (uint32_t v = threadIdx.x; v < nr * 3; v += blockDim.x) lens[v] = sec_len[(size_t)f0 * 3 + v];
    for (uint32_t v = threadIdx.x; v < m; v += blockDim.x) cols[v] = sub[v];
    __syncthreads();
    float* dst = out + (size_t)f0 * m;
    for (uint32_t e = threadIdx.x; e < nr * m; e += blockDim.x) {
        const uint32_t r = e / m, j = e - r * m;
        const uint32_t col = cols[j], byte = col >> 3, bit = 7u - (col & 7u);
        const uint32_t sec = byte < 60u ? 0u : (byte < 120u ? 1u : 2u);
        const uint32_t start = sec * 60u;
        float v = -1.0f;
        if (byte - start < (uint32_t)lens[r * 3 + sec]) v = (float)((rows[r * 128 + byte] >> bit) & 1u);
        dst[e] = v;
    }
}

}  // namespace

extern "C" int sf_header_bits(sf_ctx* ctx, const uint8_t* bytes, const uint8_t* sec_len, uint32_t n,
                              const uint16_t* sub, uint32_t m, float* out, void* stream)
{
    if (!ctx || !bytes || !sec_len || !sub || !out) return SF_ERR_ARG;
    if (m < 1 || m > 1024 || (((uintptr_t)bytes) & 15) != 0) return SF_ERR_ARG;
    SF_CUDA(cudaSetDevice(ctx->device));
    if (n == 0) return SF_OK;
    header_bits_kernel<<<(n + kRows - 1) / kRows, 256, 0, (cudaStream_t)stream>>>(bytes, sec_len, n, sub, m, out);
    SF_LAUNCH_CHECK("header_bits_kernel");
    return SF_OK;
}

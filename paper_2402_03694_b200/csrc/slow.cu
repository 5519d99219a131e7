// S4: slow-model handles, the fp32 MLP path (plain FFMA tiles) and dispatch to
// the bf16 tensor-core paths.
#include "common.cuh"
#include <new>
#include <stdlib.h>
#include <string.h>

namespace {

// out[r][o] = act( sum_k in[r][k] * W[o][k] + b[o] ),  r < *n_rows_dev
// (16 * RM) x 64 output tile, 16-deep K slices (the next one prefetched into registers), 256 threads with RM x 4 register
// tiles.  RM = 4: 64-row tiles; RM = 2: 32-row tiles, twice as many blocks when the batch is small.
template <bool RELU, int RM>
__global__ void __launch_bounds__(256)
dense_f32_kernel(const float* __restrict__ in, const float* __restrict__ W, const float* __restrict__ b,
                 const uint32_t* __restrict__ n_rows_dev, uint32_t K, uint32_t N, float* __restrict__ out,
                 uint32_t capacity, sf_dev_state* st)
{
    constexpr uint32_t TR = 16 * RM;               // rows per tile
    __shared__ float As[16][TR + 4];
    __shared__ float Bs[16][64 + 4];
    const uint32_t n_rows = sf_clamp_rows(*n_rows_dev, capacity, st);
    const uint32_t r0 = blockIdx.x * TR, o0 = blockIdx.y * 64;
    if (r0 >= n_rows) return;
    const uint32_t tx = threadIdx.x & 15, ty = threadIdx.x >> 4;
    float acc[RM][4];
#pragma unroll
    for (int i = 0; i < RM; i++)
#pragma unroll
        for (int j = 0; j < 4; j++) acc[i][j] = 0.0f;
    const uint32_t lr = threadIdx.x >> 2;          // 0..63: tile row loaded by this thread
    const uint32_t lk = (threadIdx.x & 3) * 4;     // 0,4,8,12
    const uint32_t ra = r0 + lr, ob = o0 + lr;
    const bool a_row = lr < TR;
    const bool vec = (K & 3u) == 0;                // rows start on 16-byte boundaries: one 16-byte load per operand and slice
    // the next K slice is fetched into registers while the current one is multiplied
    auto fetch = [&](uint32_t k0, float (&a)[4], float (&w)[4]) {
        const uint32_t k = k0 + lk;
        if (vec && k < K) {
            const float4 va = (a_row && ra < n_rows) ? __ldg(reinterpret_cast<const float4*>(in + (size_t)ra * K + k)) : make_float4(0.f, 0.f, 0.f, 0.f);
            const float4 vw = (ob < N) ? __ldg(reinterpret_cast<const float4*>(W + (size_t)ob * K + k)) : make_float4(0.f, 0.f, 0.f, 0.f);
            a[0] = va.x; a[1] = va.y; a[2] = va.z; a[3] = va.w;
            w[0] = vw.x; w[1] = vw.y; w[2] = vw.z; w[3] = vw.w;
        } else {
#pragma unroll
            for (int j = 0; j < 4; j++) {
                a[j] = (a_row && ra < n_rows && k + j < K) ? in[(size_t)ra * K + k + j] : 0.0f;
                w[j] = (ob < N && k + j < K) ? W[(size_t)ob * K + k + j] : 0.0f;
            }
        }
    };
    float pa[4], pw[4];
    fetch(0, pa, pw);
    for (uint32_t k0 = 0; k0 < K; k0 += 16) {
#pragma unroll
        for (int j = 0; j < 4; j++) { if (a_row) As[lk + j][lr] = pa[j]; Bs[lk + j][lr] = pw[j]; }
        __syncthreads();
        if (k0 + 16 < K) fetch(k0 + 16, pa, pw);
#pragma unroll
        for (int k = 0; k < 16; k++) {
            float a[RM], w[4];
#pragma unroll
            for (int i = 0; i < RM; i++) a[i] = As[k][ty * RM + i];
#pragma unroll
            for (int j = 0; j < 4; j++) w[j] = Bs[k][tx * 4 + j];
#pragma unroll
            for (int i = 0; i < RM; i++)
#pragma unroll
                for (int j = 0; j < 4; j++) acc[i][j] = fmaf(a[i], w[j], acc[i][j]);
        }
        __syncthreads();
    }
#pragma unroll
    for (int i = 0; i < RM; i++) {
        uint32_t r = r0 + ty * RM + i;
        if (r >= n_rows) continue;
#pragma unroll
        for (int j = 0; j < 4; j++) {
            uint32_t o = o0 + tx * 4 + j;
            if (o >= N) continue;
            float v = acc[i][j] + b[o];
            if (RELU) v = fmaxf(v, 0.0f);
            out[(size_t)r * N + o] = v;
        }
    }
}

__global__ void argmax_kernel(const float* __restrict__ logits, const uint32_t* __restrict__ n_rows_dev,
                              uint32_t C, uint8_t* __restrict__ label, uint32_t capacity)
{
    const uint32_t n_rows = min(*n_rows_dev, capacity);
    for (uint32_t r = blockIdx.x * blockDim.x + threadIdx.x; r < n_rows; r += gridDim.x * blockDim.x) {
        const float* p = logits + (size_t)r * C;
        uint32_t a = 0; float mx = p[0];
        for (uint32_t c = 1; c < C; c++) if (p[c] > mx) { mx = p[c]; a = c; }
        label[r] = (uint8_t)a;
    }
}

__global__ void count_slow_kernel(const uint32_t* __restrict__ n_rows_dev, uint32_t capacity, sf_dev_state* st) {
    atomicAdd((unsigned long long*)&st->counters.n_slow_done, (unsigned long long)min(*n_rows_dev, capacity));
}

void f32_to_bf16_host(const float* src, uint16_t* dst, size_t n) {
    for (size_t i = 0; i < n; i++) {
        uint32_t u; memcpy(&u, src + i, 4);
        uint32_t low = u & 0xFFFFu, up = u >> 16;
        if (low > 0x8000u || (low == 0x8000u && (up & 1u))) up++;
        dst[i] = (uint16_t)up;
    }
}

}  // namespace

size_t sf_slow_scratch_bytes(const sf_slow* s, uint32_t capacity) {
    if (s->arch == SF_SLOW_CNN) return sf_align256((size_t)capacity * s->C2 * sizeof(float)) + 256;
    uint32_t maxh = 0;
    for (uint32_t l = 1; l < s->n_layers; l++) if (s->dims[l] > maxh) maxh = s->dims[l];
    size_t esz = s->dtype == SF_BF16 ? 2 : 4;
    return 2 * sf_align256((size_t)capacity * maxh * esz) + 256;
}

int sf_launch_slow(sf_ctx* ctx, const sf_slow* s, const void* rows, const uint32_t* n_rows_dev, uint32_t capacity,
                   float* logits, uint8_t* label, void* scratch, cudaStream_t st, bool count_done)
{
    if (capacity == 0) return SF_OK;
    int rc;
    if (s->arch == SF_SLOW_CNN) {
        rc = sf_cnn_bf16_forward(ctx, s, rows, n_rows_dev, capacity, logits, label, scratch, st);
    } else if (s->dtype == SF_BF16) {
        rc = sf_mlp_bf16_forward(ctx, s, rows, n_rows_dev, capacity, logits, label, scratch, st);
    } else {
        uint32_t maxh = 0;
        for (uint32_t l = 1; l < s->n_layers; l++) if (s->dims[l] > maxh) maxh = s->dims[l];
        float* h0 = reinterpret_cast<float*>(scratch);
        float* h1 = reinterpret_cast<float*>(reinterpret_cast<char*>(scratch) + sf_align256((size_t)capacity * maxh * 4));
        const float* in = reinterpret_cast<const float*>(rows);
        sf_time_begin(ctx, SF_T_GEMM, st);
        for (uint32_t l = 0; l < s->n_layers; l++) {
            const bool last = (l + 1 == s->n_layers);
            if (last) { sf_time_end(ctx, SF_T_GEMM, st); sf_time_begin(ctx, SF_T_HEAD, st); }
            float* out = last ? logits : ((l & 1) ? h1 : h0);
            const uint32_t K = s->dims[l], N = s->dims[l + 1];
            const float* Wl = (const float*)s->d_W[l];
            // few tiles: 32-row tiles put twice as many blocks on the machine
            const bool small_tiles = (size_t)((capacity + 63) / 64) * ((N + 63) / 64) < 4u * (size_t)ctx->num_sms;
            if (small_tiles) {
                dim3 grid((capacity + 31) / 32, (N + 63) / 64);
                if (last) dense_f32_kernel<false, 2><<<grid, 256, 0, st>>>(in, Wl, s->d_b[l], n_rows_dev, K, N, out, capacity, ctx->d_state);
                else      dense_f32_kernel<true, 2><<<grid, 256, 0, st>>>(in, Wl, s->d_b[l], n_rows_dev, K, N, out, capacity, ctx->d_state);
            } else {
                dim3 grid((capacity + 63) / 64, (N + 63) / 64);
                if (last) dense_f32_kernel<false, 4><<<grid, 256, 0, st>>>(in, Wl, s->d_b[l], n_rows_dev, K, N, out, capacity, ctx->d_state);
                else      dense_f32_kernel<true, 4><<<grid, 256, 0, st>>>(in, Wl, s->d_b[l], n_rows_dev, K, N, out, capacity, ctx->d_state);
            }
            SF_LAUNCH_CHECK("dense_f32_kernel");
            in = out;
        }
        if (label) {
            uint32_t blocks = (capacity + 255) / 256; if (blocks > 1184) blocks = 1184;
            argmax_kernel<<<blocks, 256, 0, st>>>(logits, n_rows_dev, s->dims[s->n_layers], label, capacity);
            SF_LAUNCH_CHECK("argmax_kernel");
        }
        sf_time_end(ctx, SF_T_HEAD, st);
        rc = SF_OK;
    }
    if (rc != SF_OK) return rc;
    if (count_done) {                                  // the streaming path adds the count in its own last kernel
        count_slow_kernel<<<1, 1, 0, st>>>(n_rows_dev, capacity, ctx->d_state);
        SF_LAUNCH_CHECK("count_slow_kernel");
    }
    return SF_OK;
}

extern "C" int sf_mlp_create(sf_ctx* ctx, int dtype, uint32_t n_layers, const uint32_t* dims,
                             const float* const* W, const float* const* b, sf_slow** out)
{
    if (!ctx || !dims || !W || !b || !out) return SF_ERR_ARG;
    if (dtype != SF_F32 && dtype != SF_BF16) return SF_ERR_ARG;
    if (n_layers < 1 || n_layers > 8) return SF_ERR_ARG;
    for (uint32_t l = 0; l <= n_layers; l++) if (dims[l] == 0 || dims[l] > 65536) return SF_ERR_ARG;
    for (uint32_t l = 0; l < n_layers; l++) if (!W[l] || !b[l]) return SF_ERR_ARG;
    if (dims[n_layers] > 16) return SF_ERR_UNSUPPORTED;
    if (dtype == SF_BF16) {
        if (n_layers < 2) return SF_ERR_UNSUPPORTED;
        for (uint32_t l = 0; l < n_layers; l++) if (dims[l] % 64 != 0) return SF_ERR_UNSUPPORTED;
    }
    SF_CUDA(cudaSetDevice(ctx->device));
    sf_slow* s = new (std::nothrow) sf_slow();
    if (!s) return SF_ERR_ALLOC;
    memset(s, 0, sizeof(*s));
    s->ctx = ctx; s->arch = SF_SLOW_MLP; s->dtype = dtype; s->n_layers = n_layers;
    for (uint32_t l = 0; l <= n_layers; l++) s->dims[l] = dims[l];
    cudaError_t e = cudaSuccess;
    for (uint32_t l = 0; l < n_layers && e == cudaSuccess; l++) {
        size_t cnt = (size_t)dims[l] * dims[l + 1];
        e = cudaMalloc(&s->d_b[l], sizeof(float) * dims[l + 1]);
        if (e == cudaSuccess) e = cudaMemcpy(s->d_b[l], b[l], sizeof(float) * dims[l + 1], cudaMemcpyHostToDevice);
        if (e != cudaSuccess) break;
        if (dtype == SF_BF16) {
            // the last layer runs as a 128 x 16 tensor-core tile: pad its rows to 16 with zeros
            const size_t rows_pad = (l + 1 == n_layers) ? 16 : dims[l + 1];
            const size_t cnt_pad = rows_pad * dims[l];
            uint16_t* h = (uint16_t*)calloc(cnt_pad, 2);
            if (!h) { sf_slow_destroy(s); return SF_ERR_ALLOC; }
            f32_to_bf16_host(W[l], h, cnt);
            e = cudaMalloc(&s->d_W[l], cnt_pad * 2);
            if (e == cudaSuccess) e = cudaMemcpy(s->d_W[l], h, cnt_pad * 2, cudaMemcpyHostToDevice);
            free(h);
        } else {
            e = cudaMalloc(&s->d_W[l], cnt * 4);
            if (e == cudaSuccess) e = cudaMemcpy(s->d_W[l], W[l], cnt * 4, cudaMemcpyHostToDevice);
        }
    }
    if (e != cudaSuccess) { sf_slow_destroy(s); return sf_set_cuda_error(e, "sf_mlp_create"); }
    *out = s;
    return SF_OK;
}

extern "C" int sf_cnn_create(sf_ctx* ctx, int dtype, uint32_t L, uint32_t Cin, uint32_t C1, uint32_t C2, uint32_t k,
                             uint32_t n_cls, const float* w1, const float* b1, const float* w2, const float* b2,
                             const float* w3, const float* b3, sf_slow** out)
{
    if (!ctx || !w1 || !b1 || !w2 || !b2 || !w3 || !b3 || !out) return SF_ERR_ARG;
    if (dtype != SF_BF16) return SF_ERR_UNSUPPORTED;
    if (L != 128 || Cin != 8 || C1 != 64 || C2 != 128 || k != 5 || n_cls < 1 || n_cls > 16) return SF_ERR_UNSUPPORTED;
    SF_CUDA(cudaSetDevice(ctx->device));
    sf_slow* s = new (std::nothrow) sf_slow();
    if (!s) return SF_ERR_ALLOC;
    memset(s, 0, sizeof(*s));
    s->ctx = ctx; s->arch = SF_SLOW_CNN; s->dtype = dtype;
    s->L = L; s->Cin = Cin; s->C1 = C1; s->C2 = C2; s->k = k; s->n_cls = n_cls;
    int rc = sf_cnn_prepare(s, w1, b1, w2, b2, w3, b3);
    if (rc != SF_OK) { sf_slow_destroy(s); return rc; }
    *out = s;
    return SF_OK;
}

extern "C" void sf_slow_destroy(sf_slow* s) {
    if (!s) return;
    for (int l = 0; l < 8; l++) { if (s->d_W[l]) cudaFree(s->d_W[l]); if (s->d_b[l]) cudaFree(s->d_b[l]); }
    if (s->d_w1) cudaFree(s->d_w1); if (s->d_w2) cudaFree(s->d_w2); if (s->d_w3) cudaFree(s->d_w3);
    if (s->d_b1) cudaFree(s->d_b1); if (s->d_b2) cudaFree(s->d_b2); if (s->d_b3) cudaFree(s->d_b3);
    delete s;
}

extern "C" int sf_slow_infer(sf_ctx* ctx, const sf_slow* s, const void* rows, const uint32_t* n_rows_dev,
                             uint32_t capacity, float* logits_out, uint8_t* label_out, void* stream)
{
    if (!ctx || !s || !rows || !n_rows_dev || !logits_out) return SF_ERR_ARG;
    if (((uintptr_t)rows & 127) != 0) return SF_ERR_ARG;
    SF_CUDA(cudaSetDevice(ctx->device));
    size_t need = sf_slow_scratch_bytes(s, capacity);
    int rc = sf_ws_reserve(ctx, need);
    if (rc != SF_OK) return rc;
    sf_ws_reset(ctx);
    void* scratch = sf_ws_alloc(ctx, need);
    if (!scratch) return SF_ERR_ALLOC;
    sf_time_new_record(ctx);
    return sf_launch_slow(ctx, s, rows, n_rows_dev, capacity, logits_out, label_out, scratch, (cudaStream_t)stream);
}

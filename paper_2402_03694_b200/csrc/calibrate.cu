// Threshold calibration on the device (Sec. 3.2): Algorithm 1 (sort the validation scores,
// pick the quantile) and the data-parallel part of Algorithm 2 (per predicted class: sorted
// scores, quantile thresholds, counts of correct / incorrect flows above each threshold).
// The sort is a stable LSD radix sort on 64-bit keys (class << 32 | order-preserving image of
// the fp32 score), 8-bit digits, tiles of 4,096 keys; only the digits that carry information
// are passed over (4 for scores alone, 5 with classes).  The greedy max-slope selection of
// Algorithm 2 works on at most C*Q items and runs on the host.
#include "common.cuh"
#include <vector>
#include <algorithm>

namespace {

constexpr uint32_t kTile = 4096;
constexpr uint32_t kMaxPicks = 64;

__device__ __host__ __forceinline__ uint32_t f32_to_ordered(uint32_t b) { return b ^ ((b >> 31) ? 0xFFFFFFFFu : 0x80000000u); }
__device__ __host__ __forceinline__ uint32_t ordered_to_f32(uint32_t k) { return k ^ ((k >> 31) ? 0x80000000u : 0xFFFFFFFFu); }

__global__ void __launch_bounds__(256)
cal_key_kernel(const float* __restrict__ score, const uint8_t* __restrict__ label, uint32_t n, uint64_t* __restrict__ keys,
               uint32_t* __restrict__ cls_cnt)
{
    const uint32_t i = blockIdx.x * blockDim.x + threadIdx.x;
    if (i >= n) return;
    const uint32_t L = label ? label[i] : 0u;
    keys[i] = ((uint64_t)L << 32) | f32_to_ordered(__float_as_uint(score[i]));
    if (cls_cnt) atomicAdd(&cls_cnt[L], 1u);
}

__global__ void __launch_bounds__(256)
cal_hist_kernel(const uint64_t* __restrict__ keys, uint32_t n, uint32_t shift, uint32_t* __restrict__ hist, uint32_t nblk)
{
    __shared__ uint32_t h[256];
    h[threadIdx.x] = 0;
    __syncthreads();
    const uint32_t t0 = blockIdx.x * kTile;
    for (uint32_t j = threadIdx.x; j < kTile; j += 256) {
        const uint32_t i = t0 + j;
        if (i < n) atomicAdd(&h[(uint32_t)(keys[i] >> shift) & 255u], 1u);
    }
    __syncthreads();
    hist[threadIdx.x * nblk + blockIdx.x] = h[threadIdx.x];          // digit-major: one scan gives every block its bases
}

// exclusive scan of `entries` words by one block of 1024 threads, 1024 at a time with a carry
__global__ void __launch_bounds__(1024)
cal_scan_kernel(uint32_t* __restrict__ hist, uint32_t entries)
{
    __shared__ uint32_t wsum[32];
    __shared__ uint32_t carry;
    if (threadIdx.x == 0) carry = 0;
    __syncthreads();
    const uint32_t lane = threadIdx.x & 31, warp = threadIdx.x >> 5;
    for (uint32_t base = 0; base < entries; base += 1024) {
        const uint32_t i = base + threadIdx.x;
        const uint32_t v = i < entries ? hist[i] : 0u;
        uint32_t x = v;
        #pragma unroll
        for (uint32_t o = 1; o < 32; o <<= 1) { uint32_t y = __shfl_up_sync(0xFFFFFFFFu, x, o); if (lane >= o) x += y; }
        if (lane == 31) wsum[warp] = x;
        __syncthreads();
        if (warp == 0) {
            uint32_t s = wsum[lane], t = s;
            #pragma unroll
            for (uint32_t o = 1; o < 32; o <<= 1) { uint32_t y = __shfl_up_sync(0xFFFFFFFFu, t, o); if (lane >= o) t += y; }
            wsum[lane] = t - s;                                       // exclusive prefix of the warp sums
        }
        __syncthreads();
        const uint32_t c = carry;
        if (i < entries) hist[i] = c + wsum[warp] + x - v;
        __syncthreads();
        if (threadIdx.x == 1023) carry = c + wsum[31] + x;
        __syncthreads();
    }
}

// Stable scatter: the tile is taken 256 keys at a time in index order; a key's place among the
// keys of its digit = (earlier rounds) + (earlier warps of this round) + (lower lanes of its warp).
__global__ void __launch_bounds__(256)
cal_scatter_kernel(const uint64_t* __restrict__ kin, uint64_t* __restrict__ kout, uint32_t n, uint32_t shift,
                   const uint32_t* __restrict__ hist, uint32_t nblk)
{
    __shared__ uint32_t base[256];
    __shared__ uint32_t wc[8][256];
    const uint32_t tid = threadIdx.x, lane = tid & 31, warp = tid >> 5;
    base[tid] = hist[tid * nblk + blockIdx.x];
    uint32_t run = 0;                                                  // digit `tid`: keys of earlier rounds
    const uint32_t t0 = blockIdx.x * kTile;
    for (uint32_t r = 0; r < kTile / 256; r++) {
        #pragma unroll
        for (uint32_t w = 0; w < 8; w++) wc[w][tid] = 0;
        __syncthreads();
        const uint32_t i = t0 + r * 256 + tid;
        const bool valid = i < n;
        const uint64_t key = valid ? kin[i] : 0;
        const uint32_t d = valid ? ((uint32_t)(key >> shift) & 255u) : (256u + lane);   // idle lanes match nobody
        const uint32_t peers = __match_any_sync(0xFFFFFFFFu, d);
        const uint32_t below = __popc(peers & ((1u << lane) - 1u));
        if (valid && below == 0) wc[warp][d] = __popc(peers);
        __syncthreads();
        uint32_t acc = run;
        #pragma unroll
        for (uint32_t w = 0; w < 8; w++) { const uint32_t t = wc[w][tid]; wc[w][tid] = acc; acc += t; }
        run = acc;
        __syncthreads();
        if (valid) kout[base[d] + wc[warp][d] + below] = key;
        __syncthreads();
    }
}

struct Picks { uint32_t idx[kMaxPicks]; };

__global__ void cal_pick_kernel(const uint64_t* __restrict__ sorted, Picks p, uint32_t n_q, float* __restrict__ tau)
{
    const uint32_t j = threadIdx.x;
    if (j < n_q) tau[j] = __uint_as_float(ordered_to_f32((uint32_t)sorted[p.idx[j]]));
}

// thr[L][k], k = 0..Q: k = 0 the class maximum, k >= 1 the score at 1-based index ceil((Q-k)*m/Q) (at least 1)
// of the class's sorted scores.  seg[L] = start of class L in the sorted keys.
__global__ void __launch_bounds__(256)
cal_thresholds_kernel(const uint64_t* __restrict__ sorted, const uint32_t* __restrict__ cls_cnt, uint32_t C, uint32_t Q,
                      float* __restrict__ thr)
{
    __shared__ uint32_t seg[257];
    if (threadIdx.x == 0) { uint32_t a = 0; for (uint32_t L = 0; L < C; L++) { seg[L] = a; a += cls_cnt[L]; } seg[C] = a; }
    __syncthreads();
    for (uint32_t e = threadIdx.x; e < C * (Q + 1); e += blockDim.x) {
        const uint32_t L = e / (Q + 1), k = e - L * (Q + 1);
        const uint32_t m = seg[L + 1] - seg[L];
        float t = 0.0f;
        if (m) {
            uint32_t idx = k == 0 ? m : (uint32_t)(((uint64_t)(Q - k) * m + Q - 1) / Q);
            idx = idx < 1 ? 1 : idx;
            t = __uint_as_float(ordered_to_f32((uint32_t)sorted[seg[L] + idx - 1]));
        }
        thr[e] = t;
    }
}

// first[L][k][ok]: flows of predicted class L whose score exceeds thr[L][k] but not thr[L][k-1]
// (thresholds fall with k, so the set of thresholds a score exceeds is k >= k0).
__global__ void __launch_bounds__(256)
cal_count_kernel(const float* __restrict__ score, const uint8_t* __restrict__ label, const uint8_t* __restrict__ correct,
                 uint32_t n, uint32_t Q, const float* __restrict__ thr, uint32_t* __restrict__ first)
{
    const uint32_t i = blockIdx.x * blockDim.x + threadIdx.x;
    if (i >= n) return;
    const uint32_t L = label[i];
    const float u = score[i];
    const float* t = thr + (size_t)L * (Q + 1);
    uint32_t lo = 1, hi = Q + 1;                                       // first k in [1, Q] with u > t[k]; Q + 1 if none
    while (lo < hi) { const uint32_t mid = (lo + hi) >> 1; if (u > t[mid]) hi = mid; else lo = mid + 1; }
    if (lo <= Q) atomicAdd(&first[((size_t)L * (Q + 1) + lo) * 2 + (correct[i] ? 1u : 0u)], 1u);
}

// sorts keys (n of them, in `a`) on `bits` low bits; returns the buffer that holds the result
int radix_sort(uint64_t* a, uint64_t* b, uint32_t* hist, uint32_t n, uint32_t bits, cudaStream_t st, uint64_t** sorted)
{
    const uint32_t nblk = (n + kTile - 1) / kTile;
    uint64_t *in = a, *out = b;
    for (uint32_t shift = 0; shift < bits; shift += 8) {
        cal_hist_kernel<<<nblk, 256, 0, st>>>(in, n, shift, hist, nblk);
        cal_scan_kernel<<<1, 1024, 0, st>>>(hist, 256 * nblk);
        cal_scatter_kernel<<<nblk, 256, 0, st>>>(in, out, n, shift, hist, nblk);
        SF_LAUNCH_CHECK("calibration radix pass");
        std::swap(in, out);
    }
    *sorted = in;
    return SF_OK;
}

}  // namespace

extern "C" int sf_universal_thresholds_dev(sf_ctx* ctx, const float* scores, uint32_t n, const uint32_t* q_num, uint32_t q_den,
                                           uint32_t n_q, float* tau_out, void* stream)
{
    if (!ctx || !scores || !q_num || !tau_out || n == 0 || q_den == 0 || n_q == 0 || n_q > kMaxPicks) return SF_ERR_ARG;
    Picks p;
    for (uint32_t j = 0; j < n_q; j++) {
        if (q_num[j] > q_den) return SF_ERR_ARG;
        uint64_t idx = ((uint64_t)q_num[j] * n + q_den - 1) / q_den;   // ceil(q * n), 1-based
        idx = std::min<uint64_t>(std::max<uint64_t>(idx, 1), n);
        p.idx[j] = (uint32_t)(idx - 1);
    }
    SF_CUDA(cudaSetDevice(ctx->device));
    cudaStream_t st = (cudaStream_t)stream;
    const uint32_t nblk = (n + kTile - 1) / kTile;
    const size_t kb = sf_align256((size_t)n * 8), hb = sf_align256((size_t)256 * nblk * 4);
    int rc = sf_ws_reserve(ctx, 2 * kb + hb);
    if (rc != SF_OK) return rc;
    sf_ws_reset(ctx);
    uint64_t* a = (uint64_t*)sf_ws_alloc(ctx, kb);
    uint64_t* b = (uint64_t*)sf_ws_alloc(ctx, kb);
    uint32_t* hist = (uint32_t*)sf_ws_alloc(ctx, hb);
    if (!a || !b || !hist) return SF_ERR_ALLOC;
    cal_key_kernel<<<(n + 255) / 256, 256, 0, st>>>(scores, nullptr, n, a, nullptr);
    uint64_t* sorted = nullptr;
    rc = radix_sort(a, b, hist, n, 32, st, &sorted);
    if (rc != SF_OK) return rc;
    cal_pick_kernel<<<1, kMaxPicks, 0, st>>>(sorted, p, n_q, tau_out);
    SF_LAUNCH_CHECK("cal_pick_kernel");
    return SF_OK;
}

extern "C" int sf_per_class_thresholds(sf_ctx* ctx, const float* scores, const uint8_t* label, const uint8_t* correct,
                                       uint32_t n, uint32_t C, uint32_t Q, uint32_t a_num, uint32_t a_den,
                                       float* tau_host_out, uint64_t* assigned_host_out, void* stream)
{
    if (!ctx || !scores || !label || !correct || !tau_host_out) return SF_ERR_ARG;
    if (n == 0 || C == 0 || C > 256 || Q == 0 || Q > 1000 || a_den == 0 || a_num > a_den) return SF_ERR_ARG;
    SF_CUDA(cudaSetDevice(ctx->device));
    cudaStream_t st = (cudaStream_t)stream;
    const uint32_t nblk = (n + kTile - 1) / kTile;
    const size_t kb = sf_align256((size_t)n * 8), hb = sf_align256((size_t)256 * nblk * 4);
    const size_t items = (size_t)C * (Q + 1);
    const size_t cb = sf_align256(256 * 4), tb = sf_align256(items * 4), fb = sf_align256(items * 8);
    int rc = sf_ws_reserve(ctx, 2 * kb + hb + cb + tb + fb);
    if (rc != SF_OK) return rc;
    sf_ws_reset(ctx);
    uint64_t* a = (uint64_t*)sf_ws_alloc(ctx, kb);
    uint64_t* b = (uint64_t*)sf_ws_alloc(ctx, kb);
    uint32_t* hist = (uint32_t*)sf_ws_alloc(ctx, hb);
    uint32_t* cls = (uint32_t*)sf_ws_alloc(ctx, cb);
    float* thr = (float*)sf_ws_alloc(ctx, tb);
    uint32_t* first = (uint32_t*)sf_ws_alloc(ctx, fb);
    if (!a || !b || !hist || !cls || !thr || !first) return SF_ERR_ALLOC;
    SF_CUDA(cudaMemsetAsync(cls, 0, cb, st));
    SF_CUDA(cudaMemsetAsync(first, 0, fb, st));
    cal_key_kernel<<<(n + 255) / 256, 256, 0, st>>>(scores, label, n, a, cls);
    uint64_t* sorted = nullptr;
    rc = radix_sort(a, b, hist, n, 40, st, &sorted);
    if (rc != SF_OK) return rc;
    cal_thresholds_kernel<<<1, 256, 0, st>>>(sorted, cls, C, Q, thr);
    cal_count_kernel<<<(n + 255) / 256, 256, 0, st>>>(scores, label, correct, n, Q, thr, first);
    SF_LAUNCH_CHECK("calibration count kernels");
    std::vector<uint32_t> h_cls(256), h_first(items * 2);
    std::vector<float> h_thr(items);
    SF_CUDA(cudaMemcpyAsync(h_cls.data(), cls, 256 * 4, cudaMemcpyDeviceToHost, st));
    SF_CUDA(cudaMemcpyAsync(h_thr.data(), thr, items * 4, cudaMemcpyDeviceToHost, st));
    SF_CUDA(cudaMemcpyAsync(h_first.data(), first, items * 8, cudaMemcpyDeviceToHost, st));
    SF_CUDA(cudaStreamSynchronize(st));
    for (uint32_t L = C; L < 256; L++) if (h_cls[L]) return SF_ERR_ARG;        // a label outside [0, C)

    // Host: the max-slope queue over the per-class steps (at most C*Q of them).
    struct Step { float T; int64_t dI, dA; };
    std::vector<std::vector<Step>> R(C);
    float gmax = 0.0f; bool have = false;
    for (uint32_t L = 0; L < C; L++) {
        if (!h_cls[L]) continue;
        const float top = h_thr[(size_t)L * (Q + 1)];
        gmax = have ? std::max(gmax, top) : top; have = true;
        for (uint32_t k = 1; k <= Q; k++) {
            const size_t e = (size_t)L * (Q + 1) + k;
            const int64_t dI = h_first[e * 2], dA = (int64_t)h_first[e * 2] + h_first[e * 2 + 1];
            if (dA > 0) R[L].push_back({h_thr[e], dI, dA});
        }
    }
    std::vector<size_t> next(C, 0);
    for (uint32_t L = 0; L < C; L++) tau_host_out[L] = h_cls[L] ? h_thr[(size_t)L * (Q + 1)] : gmax;
    const uint64_t target = (uint64_t)a_num * n / a_den;
    uint64_t assigned = 0;
    while (assigned < target) {
        int best = -1;
        for (uint32_t L = 0; L < C; L++) {
            if (next[L] >= R[L].size()) continue;
            if (best < 0) { best = (int)L; continue; }
            const Step& s = R[L][next[L]]; const Step& t = R[best][next[best]];
            const int64_t lhs = s.dI * t.dA, rhs = t.dI * s.dA;
            if (lhs > rhs || (lhs == rhs && s.dA > t.dA)) best = (int)L;
        }
        if (best < 0) break;
        const Step& s = R[best][next[best]++];
        tau_host_out[best] = s.T;
        assigned += (uint64_t)s.dA;
    }
    if (assigned_host_out) *assigned_host_out = assigned;
    return SF_OK;
}

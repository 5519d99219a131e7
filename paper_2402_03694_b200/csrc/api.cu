// Context, error reporting, workspace, Algorithm 1 on the host, and the composite
// sf_serve_batch call that chains S1..S5 on one stream without host round trips.
#include "common.cuh"
#include <algorithm>
#include <new>
#include <stdio.h>
#include <stdlib.h>
#include <string.h>
#include <atomic>
#include <thread>
#include <vector>

static thread_local char g_cuda_err[512] = "";

int sf_set_cuda_error(cudaError_t e, const char* where) {
    snprintf(g_cuda_err, sizeof(g_cuda_err), "%s: %s (%s)", where, cudaGetErrorString(e), cudaGetErrorName(e));
    cudaGetLastError();      // clear the sticky-free error state for later calls
    return SF_ERR_CUDA;
}

extern "C" const char* sf_last_cuda_error(void) { return g_cuda_err; }

extern "C" const char* sf_version(void) { return "serveflow-b200 0.1 (sm_100a)"; }

extern "C" const char* sf_strerror(int status) {
    switch (status) {
    case SF_OK: return "ok";
    case SF_ERR_ARG: return "invalid argument";
    case SF_ERR_ALLOC: return "allocation failed";
    case SF_ERR_CUDA: return "CUDA call failed";
    case SF_ERR_CAPACITY: return "more flows assigned than the capacity of the output";
    case SF_ERR_TABLE_FULL: return "flow table full";
    case SF_ERR_UNSUPPORTED: return "unsupported shape";
    case SF_ERR_DEVICE_TIMEOUT: return "a bounded device-side wait gave up";
    case SF_ERR_STATIC_LIMIT: return "more flows than the built-in scratch of sf_route_noalloc holds (SF_NOALLOC_MAX_FLOWS)";
    }
    return "unknown status";
}

// ---- timing ----------------------------------------------------------------------
void sf_time_new_record(sf_ctx* ctx) {
    if (!ctx->timing) return;
    ctx->t_rec++;
    memset(ctx->t_used[(ctx->t_rec - 1) & 63], 0, SF_N_TIMERS);
}
void sf_time_begin(sf_ctx* ctx, int slot, cudaStream_t st) {
    if (!ctx->timing || ctx->t_rec == 0) return;
    uint32_t r = (ctx->t_rec - 1) & 63;
    if (ctx->t_used[r][slot]) return;                // a class that runs in several pieces keeps its first start
    cudaEventRecord(ctx->t_ev[r][slot][0], st);
    ctx->t_used[r][slot] = 1;
}
void sf_time_end(sf_ctx* ctx, int slot, cudaStream_t st) {
    if (!ctx->timing || ctx->t_rec == 0) return;
    uint32_t r = (ctx->t_rec - 1) & 63;
    cudaEventRecord(ctx->t_ev[r][slot][1], st);
    ctx->t_used[r][slot] = 2;
}

extern "C" int sf_ctx_set_timing(sf_ctx* ctx, int enable) {
    if (!ctx) return SF_ERR_ARG;
    SF_CUDA(cudaSetDevice(ctx->device));
    if (enable && !ctx->t_ev[0][0][0]) {
        for (int r = 0; r < 64; r++)
            for (int s = 0; s < SF_N_TIMERS; s++)
                for (int k = 0; k < 2; k++) SF_CUDA(cudaEventCreate(&ctx->t_ev[r][s][k]));
    }
    ctx->timing = enable ? 1 : 0;
    ctx->t_rec = 0;
    return SF_OK;
}

extern "C" int sf_ctx_get_timing(sf_ctx* ctx, uint32_t back, float* ms_out, void* stream) {
    if (!ctx || !ms_out || back >= 64) return SF_ERR_ARG;
    if (!ctx->timing || ctx->t_rec <= back) return SF_ERR_ARG;
    SF_CUDA(cudaSetDevice(ctx->device));
    SF_CUDA(cudaStreamSynchronize((cudaStream_t)stream));
    uint32_t r = (ctx->t_rec - 1 - back) & 63;
    for (int s = 0; s < SF_N_TIMERS; s++) {
        ms_out[s] = 0.0f;
        if (ctx->t_used[r][s] == 2) SF_CUDA(cudaEventElapsedTime(&ms_out[s], ctx->t_ev[r][s][0], ctx->t_ev[r][s][1]));
    }
    return SF_OK;
}

// ---- workspace ---------------------------------------------------------------
int sf_ws_reserve(sf_ctx* ctx, size_t bytes) {
    if (bytes <= ctx->ws_bytes) return SF_OK;
    SF_CUDA(cudaDeviceSynchronize());
    if (ctx->ws) { cudaFree(ctx->ws); ctx->ws = nullptr; ctx->ws_bytes = 0; }
    cudaError_t e = cudaMalloc(&ctx->ws, bytes);
    if (e != cudaSuccess) { sf_set_cuda_error(e, "cudaMalloc(workspace)"); return SF_ERR_ALLOC; }
    ctx->ws_bytes = bytes;
    ctx->ws_used = 0;
    return SF_OK;
}
void sf_ws_reset(sf_ctx* ctx) { ctx->ws_used = 0; }
void* sf_ws_alloc(sf_ctx* ctx, size_t bytes) {
    size_t b = sf_align256(bytes);
    if (ctx->ws_used + b > ctx->ws_bytes) return nullptr;
    void* p = ctx->ws + ctx->ws_used;
    ctx->ws_used += b;
    return p;
}

extern "C" int sf_ctx_create(sf_ctx** out, int device, size_t workspace_bytes) {
    if (!out) return SF_ERR_ARG;
    int count = 0;
    cudaError_t e = cudaGetDeviceCount(&count);
    if (e != cudaSuccess) return sf_set_cuda_error(e, "cudaGetDeviceCount");
    if (device < 0 || device >= count) return SF_ERR_ARG;
    SF_CUDA(cudaSetDevice(device));
    sf_ctx* c = new (std::nothrow) sf_ctx();
    if (!c) return SF_ERR_ALLOC;
    memset(c, 0, sizeof(*c));
    c->device = device;
    int sms = 0;
    e = cudaDeviceGetAttribute(&sms, cudaDevAttrMultiProcessorCount, device);
    c->num_sms = (e == cudaSuccess && sms > 0) ? sms : SF_NUM_SMS_DEFAULT;
    e = cudaMalloc(&c->d_state, sizeof(sf_dev_state));
    if (e == cudaSuccess) e = cudaMemset(c->d_state, 0, sizeof(sf_dev_state));
    if (e != cudaSuccess) { delete c; return sf_set_cuda_error(e, "sf_ctx_create"); }
    if (workspace_bytes) {
        int rc = sf_ws_reserve(c, sf_align256(workspace_bytes));
        if (rc != SF_OK) { cudaFree(c->d_state); delete c; return rc; }
    }
    *out = c;
    return SF_OK;
}

extern "C" void sf_ctx_destroy(sf_ctx* c) {
    if (!c) return;
    cudaSetDevice(c->device);
    if (c->ws) cudaFree(c->ws);
    if (c->stage) cudaFree(c->stage);
    if (c->stage2) cudaFree(c->stage2);
    if (c->aux) { cudaStreamDestroy(c->aux); cudaEventDestroy(c->ev_aux); cudaEventDestroy(c->ev_main); }
    if (c->pin) cudaFreeHost(c->pin);
    if (c->d_state) cudaFree(c->d_state);
    if (c->t_ev[0][0][0])
        for (int r = 0; r < 64; r++)
            for (int s = 0; s < SF_N_TIMERS; s++)
                for (int k = 0; k < 2; k++) cudaEventDestroy(c->t_ev[r][s][k]);
    delete c;
}

extern "C" int sf_ctx_poll(sf_ctx* ctx, sf_counters* host_out, int reset, void* stream) {
    if (!ctx) return SF_ERR_ARG;
    SF_CUDA(cudaSetDevice(ctx->device));
    cudaStream_t st = (cudaStream_t)stream;
    sf_counters c;
    SF_CUDA(cudaMemcpyAsync(&c, &ctx->d_state->counters, sizeof(c), cudaMemcpyDeviceToHost, st));
    if (reset) SF_CUDA(cudaMemsetAsync(&ctx->d_state->counters, 0, sizeof(sf_counters), st));
    SF_CUDA(cudaStreamSynchronize(st));
    if (host_out) *host_out = c;
    return c.device_error;
}

// ---- Algorithm 1 ---------------------------------------------------------------
extern "C" int sf_universal_thresholds(const float* scores, uint64_t n, const uint32_t* q_num, uint32_t q_den,
                                       uint32_t n_q, float* thresholds_out)
{
    if (!scores || !q_num || !thresholds_out || n == 0 || q_den == 0) return SF_ERR_ARG;
    std::vector<float> u(scores, scores + n);
    std::sort(u.begin(), u.end());
    for (uint32_t j = 0; j < n_q; j++) {
        if (q_num[j] > q_den) return SF_ERR_ARG;
        unsigned __int128 prod = (unsigned __int128)q_num[j] * n;
        uint64_t idx = (uint64_t)((prod + q_den - 1) / q_den);      // ceil(q * n), 1-based
        idx = std::min<uint64_t>(std::max<uint64_t>(idx, 1), n);
        thresholds_out[j] = u[idx - 1];
    }
    return SF_OK;
}

// ---- the composite call ----------------------------------------------------------
namespace {

struct ServePlan {
    size_t feat, fast_out, decision, label_fast, esc_ids, iota, rows, logits, label_slow, route_scratch, slow_scratch, total;
};

uint32_t slow_classes(const sf_slow* s) { return s->arch == SF_SLOW_CNN ? s->n_cls : s->dims[s->n_layers]; }
uint32_t slow_width(const sf_slow* s) { return s->arch == SF_SLOW_CNN ? s->L * s->Cin : s->dims[0]; }

ServePlan plan_serve(const sf_forest* fo, const sf_slow* s, uint32_t n, uint32_t F, const sf_route_cfg* cfg) {
    ServePlan p; size_t off = 0;
    auto take = [&](size_t bytes) { size_t o = off; off += sf_align256(bytes); return o; };
    const uint32_t Cf = fo->kind == SF_GBDT ? 1 : fo->C;
    const size_t esz = cfg->row_dtype == SF_BF16 ? 2 : 4;
    p.feat = take((size_t)n * F * 4);
    p.fast_out = take((size_t)n * Cf * 4);
    p.decision = take(n);
    p.label_fast = take(n);
    p.esc_ids = take((size_t)cfg->capacity * 4);
    p.iota = take((size_t)cfg->capacity * 4);
    p.rows = take((size_t)cfg->capacity * slow_width(s) * esz);
    p.logits = take((size_t)cfg->capacity * slow_classes(s) * 4);
    p.label_slow = take(cfg->capacity);
    p.route_scratch = take(sf_route_scratch_bytes(n));
    p.slow_scratch = take(sf_slow_scratch_bytes(s, cfg->capacity));
    p.total = off;
    return p;
}

int check_serve_args(sf_ctx* ctx, const sf_forest* fo, const sf_slow* s, const sf_packets* fast, uint32_t N, uint32_t F,
                     const sf_packets* wide, const sf_route_cfg* cfg)
{
    if (!ctx || !fo || !s || !fast || !wide || !cfg || !cfg->tau) return SF_ERR_ARG;
    if (!fast->size || !fast->iat_us || !fast->dir_bits) return SF_ERR_ARG;
    if (!wide->size || !wide->iat_us || !wide->dir_bits || !wide->hdr) return SF_ERR_ARG;
    if (N < 1 || N > 32 || N > fast->pitch_pkts) return SF_ERR_ARG;
    if (F != fo->F || F < 8 || F > 64 || F % 8) return SF_ERR_ARG;
    if (wide->n_flows < fast->n_flows) return SF_ERR_ARG;
    if ((cfg->rule == SF_LC_GT || cfg->rule == SF_ENTROPY_GT) && fo->kind != SF_RF) return SF_ERR_ARG;
    if (cfg->rule != SF_LC_GT && cfg->rule != SF_ENTROPY_GT && cfg->rule != SF_ABSMARGIN_LT && cfg->rule != SF_SOFTMAX_LC_GT) return SF_ERR_ARG;
    if (cfg->rule == SF_ABSMARGIN_LT && fo->kind != SF_GBDT) return SF_ERR_ARG;
    if (cfg->rule == SF_SOFTMAX_LC_GT && fo->kind != SF_GBDT_MC) return SF_ERR_ARG;
    const uint32_t W = cfg->wide_layout == SF_MLP16 ? 16u : 8u;
    if (cfg->wide_layout != SF_MLP16 && cfg->wide_layout != SF_CNN8) return SF_ERR_ARG;
    if ((cfg->wide_layout == SF_CNN8) != (s->arch == SF_SLOW_CNN)) return SF_ERR_ARG;
    if (cfg->P * W != slow_width(s)) return SF_ERR_ARG;
    if (cfg->row_dtype != s->dtype) return SF_ERR_ARG;
    const uint32_t P_real = cfg->P_real ? cfg->P_real : cfg->P;
    if (P_real > cfg->P || P_real > wide->pitch_pkts) return SF_ERR_ARG;
    if (wide->hdr_bytes < (cfg->wide_layout == SF_MLP16 ? 13u : 5u)) return SF_ERR_ARG;
    return SF_OK;
}

// Pull path of the host entry point: when the caller's wide planes are pinned host memory that the
// device can address, the assigned flows' rows are read straight out of it by this kernel (a warp per
// flow, 16-byte loads, every byte crosses the bus once) into compact device planes in list order -
// no host-side compaction, no round trip for the id list.
struct PullPlanes {
    const unsigned char* src[5]; unsigned char* dst[5]; uint32_t row_bytes[5];     // size, iat, dir words, header bytes, n_valid
};

__global__ void __launch_bounds__(256)
pull_rows_kernel(PullPlanes pl, const uint32_t* __restrict__ ids, const uint32_t* __restrict__ n_ids, uint32_t r_begin, uint32_t r_end)
{
    const uint32_t lane = threadIdx.x & 31;
    const uint32_t n = min(*n_ids, r_end);
    for (uint32_t r = r_begin + blockIdx.x * 8 + (threadIdx.x >> 5); r < n; r += gridDim.x * 8) {
        const size_t f = ids[r];
#pragma unroll
        for (int p = 0; p < 5; p++) {
            const uint32_t rb = pl.row_bytes[p];
            if (rb == 0) continue;
            const unsigned char* s = pl.src[p] + f * rb;
            unsigned char* d = pl.dst[p] + (size_t)r * rb;
            if ((rb & 15u) == 0 && ((uintptr_t)pl.src[p] & 15u) == 0) {
                for (uint32_t o = lane * 16; o < rb; o += 512) *reinterpret_cast<uint4*>(d + o) = *reinterpret_cast<const uint4*>(s + o);
            } else if ((rb & 3u) == 0 && ((uintptr_t)pl.src[p] & 3u) == 0) {
                for (uint32_t o = lane * 4; o < rb; o += 128) *reinterpret_cast<uint32_t*>(d + o) = *reinterpret_cast<const uint32_t*>(s + o);
            } else {
                for (uint32_t o = lane; o < rb; o += 32) d[o] = s[o];
            }
        }
    }
}

// rows of the list that fall into each chunk of R rows
__global__ void chunk_counts_kernel(const uint32_t* __restrict__ n_total, uint32_t cap, uint32_t R, uint32_t n_chunks,
                                    uint32_t* __restrict__ cnt)
{
    const uint32_t i = blockIdx.x * blockDim.x + threadIdx.x;
    if (i >= n_chunks) return;
    const uint32_t k = min(*n_total, cap), c0 = i * R;
    cnt[i] = k > c0 ? min(k - c0, R) : 0u;
}

// device-side alias of a host pointer if it is pinned and mapped, else nullptr
const void* mapped_alias(const void* host_ptr) {
    if (!host_ptr) return nullptr;
    cudaPointerAttributes a;
    if (cudaPointerGetAttributes(&a, host_ptr) != cudaSuccess) { cudaGetLastError(); return nullptr; }
    if (a.type != cudaMemoryTypeHost || !a.devicePointer) return nullptr;
    return a.devicePointer;
}

// phases: 1 = S1..S3 without the wide-row gather, 2 = gather (rows 0..n_esc-1 of `wide`, which then holds
// only the assigned flows' planes in list order) + S4 + S5 on the state phase 1 left, 3 = everything.
enum { SF_PHASE_FAST = 1, SF_PHASE_SLOW = 2, SF_PHASE_ALL = 3 };

int serve_on_device(sf_ctx* ctx, const sf_forest* fo, const sf_slow* s, const sf_packets* fast, uint32_t N, uint32_t F,
                    const sf_packets* wide, const sf_route_cfg* cfg, uint8_t* label_out, uint8_t* stage_out,
                    uint32_t* n_esc_out, cudaStream_t st, int phases = SF_PHASE_ALL)
{
    const uint32_t n = fast->n_flows;
    const ServePlan p = plan_serve(fo, s, n, F, cfg);
    int rc = sf_ws_reserve(ctx, p.total);
    if (rc != SF_OK) return rc;
    if (phases & SF_PHASE_FAST) sf_ws_reset(ctx);
    char* base = (phases & SF_PHASE_FAST) ? reinterpret_cast<char*>(sf_ws_alloc(ctx, p.total)) : ctx->ws;
    if (!base) return SF_ERR_ALLOC;
    float* feat = reinterpret_cast<float*>(base + p.feat);
    float* fast_out = reinterpret_cast<float*>(base + p.fast_out);
    uint8_t* decision = reinterpret_cast<uint8_t*>(base + p.decision);
    uint8_t* label_fast = reinterpret_cast<uint8_t*>(base + p.label_fast);
    uint32_t* esc_ids = reinterpret_cast<uint32_t*>(base + p.esc_ids);
    void* rows = base + p.rows;
    float* logits = reinterpret_cast<float*>(base + p.logits);
    uint8_t* label_slow = reinterpret_cast<uint8_t*>(base + p.label_slow);
    uint32_t* n_esc_dev = &ctx->d_state->scan_total;
    // one call for everything, a fast model and rule the tree kernel can score itself, outputs for every flow: fold the
    // assignment and the first merge into the tree kernel
    const bool fused = phases == SF_PHASE_ALL && n > 0 &&
                       ((fo->kind == SF_RF && cfg->rule == SF_LC_GT) || (fo->kind == SF_GBDT && cfg->rule == SF_ABSMARGIN_LT));

    if (phases & SF_PHASE_FAST) {
        sf_time_new_record(ctx);
        sf_time_begin(ctx, SF_T_EXTRACT, st);
        rc = sf_launch_extract(fast, N, F, feat, st);
        sf_time_end(ctx, SF_T_EXTRACT, st);
        if (rc != SF_OK) return rc;
        sf_time_begin(ctx, SF_T_FOREST, st);
        if (fused) {
            // the tree kernel takes the decisions in its epilogue (score, label, decision byte, fast label and stage 1 of every
            // flow, assigned flows per block): no score kernel, no first merge kernel
            sf_fused_route fr;
            fr.tau = cfg->tau; fr.rule = cfg->rule; fr.decision = decision; fr.label_fast = label_fast;
            fr.label_out = label_out; fr.stage_out = stage_out; fr.block_counts = reinterpret_cast<uint32_t*>(base + p.route_scratch);
            rc = sf_launch_forest(fo, feat, n, fast_out, nullptr, st, nullptr, false, &fr);
            sf_time_end(ctx, SF_T_FOREST, st);
            if (rc != SF_OK) return rc;
            rc = sf_launch_route_after_fused(ctx, cfg, n, wide, esc_ids, n_esc_out, rows, decision, fr.block_counts, st);
        } else {
            rc = sf_launch_forest(fo, feat, n, fast_out, nullptr, st);
            sf_time_end(ctx, SF_T_FOREST, st);
            if (rc != SF_OK) return rc;
            rc = sf_launch_route(ctx, cfg, fast_out, n, fo->C, (phases & SF_PHASE_SLOW) ? wide : nullptr, esc_ids, n_esc_out,
                                 rows, decision, label_fast, nullptr, base + p.route_scratch, st);
        }
        if (rc != SF_OK) return rc;
        ctx->last_feat = feat; ctx->last_fast_out = fast_out; ctx->last_esc_ids = esc_ids; ctx->last_rows = rows;
        ctx->last_logits = logits; ctx->last_label_fast = label_fast; ctx->last_label_slow = label_slow;
        if (!(phases & SF_PHASE_SLOW)) return SF_OK;
    } else {
        uint32_t* iota = reinterpret_cast<uint32_t*>(base + p.iota);
        rc = sf_launch_iota(iota, cfg->capacity, st);
        if (rc != SF_OK) return rc;
        sf_time_begin(ctx, SF_T_GATHER, st);
        rc = sf_launch_gather(ctx, cfg, wide, iota, n_esc_dev, cfg->capacity, rows, st);
        sf_time_end(ctx, SF_T_GATHER, st);
        if (rc != SF_OK) return rc;
    }
    rc = sf_launch_slow(ctx, s, rows, n_esc_dev, cfg->capacity, logits, label_slow, base + p.slow_scratch, st, !fused);
    if (rc != SF_OK) return rc;
    sf_time_begin(ctx, SF_T_MERGE, st);
    rc = sf_launch_merge(label_fast, decision, n, esc_ids, n_esc_dev, cfg->capacity, label_slow, label_out, stage_out, st, 2, !fused,
                         fused ? ctx->d_state : nullptr);
    sf_time_end(ctx, SF_T_MERGE, st);
    if (rc != SF_OK) return rc;
    ctx->last_feat = feat; ctx->last_fast_out = fast_out; ctx->last_esc_ids = esc_ids; ctx->last_rows = rows;
    ctx->last_logits = logits; ctx->last_label_fast = label_fast; ctx->last_label_slow = label_slow;
    return SF_OK;
}

// Host entry point, pull route (separate fast and slow planes, slow planes pinned and device-addressable).
// Two streams: transfers run on the context's second stream, kernels on the caller's.
//   A  the fast planes go up in chunks of whole forest waves; extract + forest of a chunk start as soon
//      as it has landed, so only the first chunk's copy and the last chunk's kernels are exposed;
//   B  route over all flows; the count comes back (4 bytes) so that only chunks with rows are launched;
//   C  the assigned flows' slow-context rows are pulled out of the pinned planes in chunks of 32,768 rows;
//      gather + slow model of a chunk run while the next chunk crosses the bus;
//   D  merge, labels back.
int serve_host_pull(sf_ctx* ctx, const sf_forest* fo, const sf_slow* s, const sf_packets* fast_h, uint32_t N, uint32_t F,
                    const sf_packets* wide_h, const void* const m_wide[5], const sf_route_cfg* cfg_h, char* sb2,
                    const size_t a_fast[4], size_t a_tau, size_t a_lab, size_t a_stg, size_t a_ne, uint32_t n_tau,
                    uint8_t* label_h, uint8_t* stage_h, uint32_t* n_esc_h, cudaStream_t st)
{
    const uint32_t n = fast_h->n_flows, Pf = fast_h->pitch_pkts, wf = (Pf + 31) / 32;
    const uint32_t Pw = wide_h->pitch_pkts, Hb = wide_h->hdr_bytes, words = (Pw + 31) / 32;
    if (!ctx->aux) {
        SF_CUDA(cudaStreamCreateWithFlags(&ctx->aux, cudaStreamNonBlocking));
        SF_CUDA(cudaEventCreateWithFlags(&ctx->ev_aux, cudaEventDisableTiming));
        SF_CUDA(cudaEventCreateWithFlags(&ctx->ev_main, cudaEventDisableTiming));
    }
    cudaStream_t sx = ctx->aux;
    sf_route_cfg cd = *cfg_h;
    cd.tau = (const float*)(sb2 + a_tau);
    const ServePlan p = plan_serve(fo, s, n, F, &cd);
    int rc = sf_ws_reserve(ctx, p.total);
    if (rc != SF_OK) return rc;
    sf_ws_reset(ctx);
    char* base = reinterpret_cast<char*>(sf_ws_alloc(ctx, p.total));
    if (!base) return SF_ERR_ALLOC;
    float* feat = (float*)(base + p.feat); float* fast_out = (float*)(base + p.fast_out);
    uint8_t* decision = (uint8_t*)(base + p.decision); uint8_t* label_fast = (uint8_t*)(base + p.label_fast);
    uint32_t* esc_ids = (uint32_t*)(base + p.esc_ids); uint32_t* iota = (uint32_t*)(base + p.iota);
    char* rows = base + p.rows; float* logits = (float*)(base + p.logits); uint8_t* label_slow = (uint8_t*)(base + p.label_slow);
    uint32_t* n_esc_dev = &ctx->d_state->scan_total;
    const uint32_t Cf = fo->kind == SF_GBDT ? 1 : fo->C;
    sf_time_new_record(ctx);

    // A: uploads on sx, kernels on st
    SF_CUDA(cudaMemcpyAsync(sb2 + a_tau, cfg_h->tau, (size_t)n_tau * 4, cudaMemcpyHostToDevice, st));
    SF_CUDA(cudaEventRecord(ctx->ev_main, st));
    SF_CUDA(cudaStreamWaitEvent(sx, ctx->ev_main, 0));            // the staging buffers are free once earlier work on st is done
    const uint32_t FC = (uint32_t)ctx->num_sms * 512u * 2u;       // two full waves of the forest kernel
    for (uint32_t f0 = 0; f0 < n; f0 += FC) {
        const uint32_t m = std::min(FC, n - f0);
        SF_CUDA(cudaMemcpyAsync(sb2 + a_fast[0] + (size_t)f0 * Pf * 2, (const char*)fast_h->size + (size_t)f0 * Pf * 2, (size_t)m * Pf * 2, cudaMemcpyHostToDevice, sx));
        SF_CUDA(cudaMemcpyAsync(sb2 + a_fast[1] + (size_t)f0 * Pf * 4, (const char*)fast_h->iat_us + (size_t)f0 * Pf * 4, (size_t)m * Pf * 4, cudaMemcpyHostToDevice, sx));
        SF_CUDA(cudaMemcpyAsync(sb2 + a_fast[2] + (size_t)f0 * wf * 4, (const char*)fast_h->dir_bits + (size_t)f0 * wf * 4, (size_t)m * wf * 4, cudaMemcpyHostToDevice, sx));
        if (fast_h->n_valid)
            SF_CUDA(cudaMemcpyAsync(sb2 + a_fast[3] + f0, fast_h->n_valid + f0, m, cudaMemcpyHostToDevice, sx));
        SF_CUDA(cudaEventRecord(ctx->ev_aux, sx));
        SF_CUDA(cudaStreamWaitEvent(st, ctx->ev_aux, 0));
        sf_packets fc = *fast_h;
        fc.size = (const uint16_t*)(sb2 + a_fast[0]) + (size_t)f0 * Pf; fc.iat_us = (const uint32_t*)(sb2 + a_fast[1]) + (size_t)f0 * Pf;
        fc.dir_bits = (const uint32_t*)(sb2 + a_fast[2]) + (size_t)f0 * wf; fc.hdr = nullptr;
        fc.n_valid = fast_h->n_valid ? (const uint8_t*)(sb2 + a_fast[3]) + f0 : nullptr;
        fc.n_flows = m;
        sf_time_begin(ctx, SF_T_EXTRACT, st);
        rc = sf_launch_extract(&fc, N, F, feat + (size_t)f0 * F, st);
        sf_time_end(ctx, SF_T_EXTRACT, st);
        if (rc != SF_OK) return rc;
        sf_time_begin(ctx, SF_T_FOREST, st);
        rc = sf_launch_forest(fo, feat + (size_t)f0 * F, m, fast_out + (size_t)f0 * Cf, nullptr, st);
        sf_time_end(ctx, SF_T_FOREST, st);
        if (rc != SF_OK) return rc;
    }
    // B: assignment over all flows; the count comes back
    rc = sf_launch_route(ctx, &cd, fast_out, n, fo->C, nullptr, esc_ids, (uint32_t*)(sb2 + a_ne), nullptr, decision, label_fast,
                         nullptr, base + p.route_scratch, st);
    if (rc != SF_OK) return rc;
    uint32_t k = 0;
    SF_CUDA(cudaMemcpyAsync(&k, sb2 + a_ne, 4, cudaMemcpyDeviceToHost, st));
    SF_CUDA(cudaStreamSynchronize(st));
    // C: pull, gather and slow model chunk by chunk
    const size_t r_sz = (size_t)Pw * 2, r_ia = (size_t)Pw * 4, r_dr = (size_t)words * 4, r_hd = (size_t)Pw * Hb;
    const size_t esz = cd.row_dtype == SF_BF16 ? 2 : 4, D = slow_width(s), Cs = slow_classes(s);
    if (k) {
        const uint32_t R = std::min<uint32_t>(32768u, cd.capacity), n_chunks = (k + R - 1) / R;
        const size_t c_sz = 0, c_ia = sf_align256(c_sz + k * r_sz), c_dr = sf_align256(c_ia + k * r_ia),
                     c_hd = sf_align256(c_dr + k * r_dr), c_nv = sf_align256(c_hd + k * r_hd),
                     c_cnt = sf_align256(c_nv + (wide_h->n_valid ? k : 0)), c_total = c_cnt + sf_align256((size_t)n_chunks * 4) + 256;
        if (c_total > ctx->stage2_bytes) {
            SF_CUDA(cudaDeviceSynchronize());
            if (ctx->stage2) { cudaFree(ctx->stage2); ctx->stage2 = nullptr; }
            ctx->stage2_bytes = 0;
            const size_t want = c_total + c_total / 4;
            cudaError_t e = cudaMalloc(&ctx->stage2, want);
            if (e != cudaSuccess) { sf_set_cuda_error(e, "cudaMalloc(pulled rows)"); return SF_ERR_ALLOC; }
            ctx->stage2_bytes = want;
        }
        char* dv = ctx->stage2;
        uint32_t* cnt = (uint32_t*)(dv + c_cnt);
        PullPlanes pl;
        const size_t c_off[5] = {c_sz, c_ia, c_dr, c_hd, c_nv};
        const uint32_t rb[5] = {(uint32_t)r_sz, (uint32_t)r_ia, (uint32_t)r_dr, (uint32_t)r_hd, wide_h->n_valid ? 1u : 0u};
        for (int q = 0; q < 5; q++) { pl.src[q] = (const unsigned char*)m_wide[q]; pl.dst[q] = (unsigned char*)dv + c_off[q]; pl.row_bytes[q] = rb[q]; }
        chunk_counts_kernel<<<(n_chunks + 255) / 256, 256, 0, st>>>(n_esc_dev, cd.capacity, R, n_chunks, cnt);
        SF_LAUNCH_CHECK("chunk_counts_kernel");
        rc = sf_launch_iota(iota, R, st);
        if (rc != SF_OK) return rc;
        SF_CUDA(cudaEventRecord(ctx->ev_main, st));
        SF_CUDA(cudaStreamWaitEvent(sx, ctx->ev_main, 0));
        sf_time_begin(ctx, SF_T_PULL, sx);
        for (uint32_t c = 0; c < n_chunks; c++) {
            const uint32_t r0 = c * R, r1 = std::min(k, r0 + R);
            const uint32_t grid = std::min<uint32_t>((r1 - r0 + 7) / 8, (uint32_t)ctx->num_sms * 4u);
            pull_rows_kernel<<<grid, 256, 0, sx>>>(pl, esc_ids, n_esc_dev, r0, r1);
            SF_LAUNCH_CHECK("pull_rows_kernel");
            if (c + 1 == n_chunks) sf_time_end(ctx, SF_T_PULL, sx);
            SF_CUDA(cudaEventRecord(ctx->ev_aux, sx));
            SF_CUDA(cudaStreamWaitEvent(st, ctx->ev_aux, 0));
            sf_packets wc = *wide_h;
            wc.size = (const uint16_t*)(dv + c_sz + r0 * r_sz); wc.iat_us = (const uint32_t*)(dv + c_ia + r0 * r_ia);
            wc.dir_bits = (const uint32_t*)(dv + c_dr + r0 * r_dr); wc.hdr = (const uint8_t*)(dv + c_hd + r0 * r_hd);
            wc.n_valid = wide_h->n_valid ? (const uint8_t*)(dv + c_nv + r0) : nullptr;
            wc.n_flows = r1 - r0;
            sf_time_begin(ctx, SF_T_GATHER, st);
            rc = sf_launch_gather(ctx, &cd, &wc, iota, cnt + c, R, rows + (size_t)r0 * D * esz, st);
            sf_time_end(ctx, SF_T_GATHER, st);
            if (rc != SF_OK) return rc;
            rc = sf_launch_slow(ctx, s, rows + (size_t)r0 * D * esz, cnt + c, R, logits + (size_t)r0 * Cs, label_slow + r0,
                                base + p.slow_scratch, st);
            if (rc != SF_OK) return rc;
        }
    }
    // D: merge and results
    sf_time_begin(ctx, SF_T_MERGE, st);
    rc = sf_launch_merge(label_fast, decision, n, esc_ids, n_esc_dev, cd.capacity, label_slow, (uint8_t*)(sb2 + a_lab),
                         (uint8_t*)(sb2 + a_stg), st);
    sf_time_end(ctx, SF_T_MERGE, st);
    if (rc != SF_OK) return rc;
    ctx->last_feat = feat; ctx->last_fast_out = fast_out; ctx->last_esc_ids = esc_ids; ctx->last_rows = rows;
    ctx->last_logits = logits; ctx->last_label_fast = label_fast; ctx->last_label_slow = label_slow;
    SF_CUDA(cudaMemcpyAsync(label_h, sb2 + a_lab, n, cudaMemcpyDeviceToHost, st));
    SF_CUDA(cudaMemcpyAsync(stage_h, sb2 + a_stg, n, cudaMemcpyDeviceToHost, st));
    SF_CUDA(cudaStreamSynchronize(st));
    if (n_esc_h) *n_esc_h = k;
    return SF_OK;
}

}  // namespace

extern "C" int sf_serve_batch(sf_ctx* ctx, const sf_forest* fo, const sf_slow* s, const sf_packets* fast, uint32_t N,
                              uint32_t F, const sf_packets* wide, const sf_route_cfg* cfg, uint8_t* label_out,
                              uint8_t* stage_out, uint32_t* n_esc_out, void* stream)
{
    int rc = check_serve_args(ctx, fo, s, fast, N, F, wide, cfg);
    if (rc != SF_OK) return rc;
    if (!label_out || !stage_out) return SF_ERR_ARG;
    SF_CUDA(cudaSetDevice(ctx->device));
    return serve_on_device(ctx, fo, s, fast, N, F, wide, cfg, label_out, stage_out, n_esc_out, (cudaStream_t)stream);
}

extern "C" int sf_serve_batch3(sf_ctx* ctx, const sf_forest* f1, const sf_forest* f2, const sf_slow* s, const sf_packets* fast,
                               uint32_t N, uint32_t F, const sf_packets* wide, const sf_route_cfg* cfg1,
                               const sf_route_cfg* cfg2, uint8_t* label_out, uint8_t* stage_out, uint32_t* n_esc_out,
                               void* stream)
{
    if (!f1 || !cfg1 || !cfg1->tau) return SF_ERR_ARG;
    int rc = check_serve_args(ctx, f2, s, fast, N, F, wide, cfg2);
    if (rc != SF_OK) return rc;
    if (!label_out || !stage_out) return SF_ERR_ARG;
    if (f1->kind != SF_RF || f1->F != F || cfg1->rule != SF_LC_GT) return SF_ERR_ARG;
    if (cfg2->rule != SF_LC_GT && cfg2->rule != SF_SOFTMAX_LC_GT) return SF_ERR_ARG;      // fast model: forest or multi-class boosted trees
    SF_CUDA(cudaSetDevice(ctx->device));
    cudaStream_t st = (cudaStream_t)stream;
    const uint32_t n = fast->n_flows, cap = cfg2->capacity;
    const size_t esz = cfg2->row_dtype == SF_BF16 ? 2 : 4;
    size_t off = 0;
    auto take = [&](size_t bytes) { size_t o = off; off += sf_align256(bytes); return o; };
    const size_t o_feat = take((size_t)n * F * 4), o_p1 = take((size_t)n * f1->C * 4), o_dec1 = take(n), o_lab1 = take(n),
                 o_ids1 = take((size_t)n * 4), o_feat2 = take((size_t)n * F * 4), o_p2 = take((size_t)n * f2->C * 4),
                 o_dec2 = take(n), o_lab2 = take(n), o_ids2l = take((size_t)cap * 4), o_ids2 = take((size_t)cap * 4),
                 o_rows = take((size_t)cap * slow_width(s) * esz), o_logits = take((size_t)cap * slow_classes(s) * 4),
                 o_labs = take(cap), o_rs1 = take(sf_route_scratch_bytes(n)), o_rs2 = take(sf_route_scratch_bytes(n)),
                 o_slow = take(sf_slow_scratch_bytes(s, cap)), o_cnt = take(64);
    rc = sf_ws_reserve(ctx, off);
    if (rc != SF_OK) return rc;
    sf_ws_reset(ctx);
    char* w = reinterpret_cast<char*>(sf_ws_alloc(ctx, off));
    if (!w) return SF_ERR_ALLOC;
    float* feat = (float*)(w + o_feat); float* feat2 = (float*)(w + o_feat2);
    float* p1 = (float*)(w + o_p1); float* p2 = (float*)(w + o_p2);
    uint32_t* ids1 = (uint32_t*)(w + o_ids1); uint32_t* ids2l = (uint32_t*)(w + o_ids2l); uint32_t* ids2 = (uint32_t*)(w + o_ids2);
    uint32_t* cnt = n_esc_out ? n_esc_out : (uint32_t*)(w + o_cnt);          // [0] after the fastest model, [1] after the fast one
    sf_time_new_record(ctx);
    sf_time_begin(ctx, SF_T_EXTRACT, st);
    rc = sf_launch_extract(fast, N, F, feat, st);
    sf_time_end(ctx, SF_T_EXTRACT, st);
    if (rc != SF_OK) return rc;
    sf_time_begin(ctx, SF_T_FOREST, st);
    rc = sf_launch_forest(f1, feat, n, p1, nullptr, st);
    if (rc != SF_OK) return rc;
    // tier 1 -> 2: every flow the fastest model is unsure of (capacity n: the list cannot overflow)
    sf_route_cfg c1 = *cfg1;
    c1.capacity = n;
    rc = sf_launch_route(ctx, &c1, p1, n, f1->C, nullptr, ids1, &cnt[0], nullptr, (uint8_t*)(w + o_dec1), (uint8_t*)(w + o_lab1),
                         nullptr, w + o_rs1, st);
    if (rc != SF_OK) return rc;
    rc = sf_launch_gather_feat(feat, ids1, &cnt[0], n, F, feat2, st);
    if (rc != SF_OK) return rc;
    rc = sf_launch_forest(f2, feat2, n, p2, nullptr, st, &cnt[0]);
    sf_time_end(ctx, SF_T_FOREST, st);
    if (rc != SF_OK) return rc;
    // tier 2 -> 3: positions in the first list, then the flow ids themselves
    rc = sf_launch_route(ctx, cfg2, p2, n, f2->C, nullptr, ids2l, &cnt[1], nullptr, (uint8_t*)(w + o_dec2), (uint8_t*)(w + o_lab2),
                         nullptr, w + o_rs2, st, &cnt[0]);
    if (rc != SF_OK) return rc;
    rc = sf_launch_compose_ids(ids1, ids2l, &cnt[1], cap, ids2, st);
    if (rc != SF_OK) return rc;
    sf_time_begin(ctx, SF_T_GATHER, st);
    rc = sf_launch_gather(ctx, cfg2, wide, ids2, &cnt[1], cap, w + o_rows, st);
    sf_time_end(ctx, SF_T_GATHER, st);
    if (rc != SF_OK) return rc;
    rc = sf_launch_slow(ctx, s, w + o_rows, &cnt[1], cap, (float*)(w + o_logits), (uint8_t*)(w + o_labs), w + o_slow, st);
    if (rc != SF_OK) return rc;
    sf_time_begin(ctx, SF_T_MERGE, st);
    rc = sf_launch_merge((uint8_t*)(w + o_lab1), nullptr, n, ids1, &cnt[0], n, (uint8_t*)(w + o_lab2), label_out, stage_out, st, 2, true);
    if (rc == SF_OK)
        rc = sf_launch_merge(nullptr, nullptr, n, ids2, &cnt[1], cap, (uint8_t*)(w + o_labs), label_out, stage_out, st, 3, false);
    sf_time_end(ctx, SF_T_MERGE, st);
    if (rc != SF_OK) return rc;
    ctx->last_feat = feat; ctx->last_fast_out = p2; ctx->last_esc_ids = ids2; ctx->last_rows = w + o_rows;
    ctx->last_logits = (float*)(w + o_logits); ctx->last_label_fast = (uint8_t*)(w + o_lab1); ctx->last_label_slow = (uint8_t*)(w + o_labs);
    return SF_OK;
}

extern "C" int sf_serve_batch_host(sf_ctx* ctx, const sf_forest* fo, const sf_slow* s, const sf_packets* fast_h,
                                   uint32_t N, uint32_t F, const sf_packets* wide_h, const sf_route_cfg* cfg_h,
                                   uint8_t* label_h, uint8_t* stage_h, uint32_t* n_esc_h, void* stream)
{
    int rc = check_serve_args(ctx, fo, s, fast_h, N, F, wide_h, cfg_h);
    if (rc != SF_OK) return rc;
    if (!label_h || !stage_h) return SF_ERR_ARG;
    SF_CUDA(cudaSetDevice(ctx->device));
    cudaStream_t st = (cudaStream_t)stream;
    const uint32_t n = fast_h->n_flows;
    const bool shared = fast_h->size == wide_h->size && fast_h->iat_us == wide_h->iat_us &&
                        fast_h->dir_bits == wide_h->dir_bits && fast_h->pitch_pkts == wide_h->pitch_pkts;
    if (!shared) {
        // Two-phase host path: only the fast planes of all flows cross the bus first; after S1..S3 the
        // assigned ids come back, worker threads compact those flows' wide rows into pinned memory and
        // copy them over chunk by chunk (the gather of one chunk overlaps the copy of the previous one),
        // and only then S4/S5 run.  The slow model sees more packets only of the flows assigned to it.
        const uint32_t Pw = wide_h->pitch_pkts, Hb = wide_h->hdr_bytes, words = (Pw + 31) / 32;
        const size_t fsz = (size_t)n * fast_h->pitch_pkts * 2, fia = (size_t)n * fast_h->pitch_pkts * 4,
                     fdr = (size_t)n * ((fast_h->pitch_pkts + 31) / 32) * 4, fnv = fast_h->n_valid ? (size_t)n : 0;
        const uint32_t n_tau2 = cfg_h->rule == SF_ABSMARGIN_LT ? 1 : fo->C;
        size_t off2 = 0;
        auto take2 = [&](size_t bytes) { size_t o = off2; off2 += sf_align256(bytes); return o; };
        const size_t a_fs = take2(fsz), a_fi = take2(fia), a_fd = take2(fdr), a_fv = take2(fnv), a_tau = take2(n_tau2 * 4),
                     a_lab = take2(n), a_stg = take2(n), a_ne = take2(4);
        if (off2 > ctx->stage_bytes) {
            SF_CUDA(cudaDeviceSynchronize());
            if (ctx->stage) { cudaFree(ctx->stage); ctx->stage = nullptr; ctx->stage_bytes = 0; }
            cudaError_t e = cudaMalloc(&ctx->stage, off2);
            if (e != cudaSuccess) { sf_set_cuda_error(e, "cudaMalloc(staging)"); return SF_ERR_ALLOC; }
            ctx->stage_bytes = off2;
        }
        char* sb2 = ctx->stage;
        {
            const void* m_wide[5] = {mapped_alias(wide_h->size), mapped_alias(wide_h->iat_us), mapped_alias(wide_h->dir_bits),
                                     mapped_alias(wide_h->hdr), wide_h->n_valid ? mapped_alias(wide_h->n_valid) : nullptr};
            if (m_wide[0] && m_wide[1] && m_wide[2] && m_wide[3] && (!wide_h->n_valid || m_wide[4])) {
                const size_t a_fast[4] = {a_fs, a_fi, a_fd, a_fv};
                return serve_host_pull(ctx, fo, s, fast_h, N, F, wide_h, m_wide, cfg_h, sb2, a_fast, a_tau, a_lab, a_stg, a_ne,
                                       n_tau2, label_h, stage_h, n_esc_h, st);
            }
        }
        SF_CUDA(cudaMemcpyAsync(sb2 + a_fs, fast_h->size, fsz, cudaMemcpyHostToDevice, st));
        SF_CUDA(cudaMemcpyAsync(sb2 + a_fi, fast_h->iat_us, fia, cudaMemcpyHostToDevice, st));
        SF_CUDA(cudaMemcpyAsync(sb2 + a_fd, fast_h->dir_bits, fdr, cudaMemcpyHostToDevice, st));
        if (fnv) SF_CUDA(cudaMemcpyAsync(sb2 + a_fv, fast_h->n_valid, fnv, cudaMemcpyHostToDevice, st));
        SF_CUDA(cudaMemcpyAsync(sb2 + a_tau, cfg_h->tau, (size_t)n_tau2 * 4, cudaMemcpyHostToDevice, st));
        sf_packets fd2 = *fast_h;
        fd2.size = (const uint16_t*)(sb2 + a_fs); fd2.iat_us = (const uint32_t*)(sb2 + a_fi);
        fd2.dir_bits = (const uint32_t*)(sb2 + a_fd); fd2.hdr = nullptr;
        fd2.n_valid = fnv ? (const uint8_t*)(sb2 + a_fv) : nullptr;
        sf_route_cfg cd2 = *cfg_h;
        cd2.tau = (const float*)(sb2 + a_tau);
        const size_t r_sz = (size_t)Pw * 2, r_ia = (size_t)Pw * 4, r_dr = (size_t)words * 4, r_hd = (size_t)Pw * Hb;
        rc = serve_on_device(ctx, fo, s, &fd2, N, F, wide_h, &cd2, (uint8_t*)(sb2 + a_lab), (uint8_t*)(sb2 + a_stg),
                             (uint32_t*)(sb2 + a_ne), st, SF_PHASE_FAST);
        if (rc != SF_OK) return rc;
        uint32_t k = 0;
        SF_CUDA(cudaMemcpyAsync(&k, sb2 + a_ne, 4, cudaMemcpyDeviceToHost, st));
        SF_CUDA(cudaStreamSynchronize(st));
        std::vector<uint32_t> ids(k);
        if (k) SF_CUDA(cudaMemcpy(ids.data(), ctx->last_esc_ids, (size_t)k * 4, cudaMemcpyDeviceToHost));
        // compact planes of the k assigned flows: [k][Pw] sizes, [k][Pw] iats, [k][words] dir words, [k][Pw][Hb] header bytes, [k] n_valid
        const size_t c_sz = 0, c_ia = sf_align256(c_sz + k * r_sz), c_dr = sf_align256(c_ia + k * r_ia),
                     c_hd = sf_align256(c_dr + k * r_dr), c_nv = sf_align256(c_hd + k * r_hd),
                     c_total = sf_align256(c_nv + (wide_h->n_valid ? k : 0)) + 256;
        if (c_total > ctx->stage2_bytes || c_total > ctx->pin_bytes) {
            SF_CUDA(cudaDeviceSynchronize());
            const size_t want = c_total + c_total / 4;
            cudaError_t e = cudaSuccess;
            if (c_total > ctx->stage2_bytes) {
                if (ctx->stage2) { cudaFree(ctx->stage2); ctx->stage2 = nullptr; }
                ctx->stage2_bytes = 0;
                e = cudaMalloc(&ctx->stage2, want);
                if (e == cudaSuccess) ctx->stage2_bytes = want;
            }
            if (e == cudaSuccess && c_total > ctx->pin_bytes) {
                if (ctx->pin) { cudaFreeHost(ctx->pin); ctx->pin = nullptr; }
                ctx->pin_bytes = 0;
                e = cudaMallocHost(&ctx->pin, want);
                if (e == cudaSuccess) ctx->pin_bytes = want;
            }
            if (e != cudaSuccess) { sf_set_cuda_error(e, "cudaMalloc(compact staging)"); return SF_ERR_ALLOC; }
        }
        char* pin = ctx->pin; char* dv = ctx->stage2;
        const uint32_t chunk = 4096, n_chunks = (k + chunk - 1) / chunk;
        std::atomic<uint32_t> next(0);
        std::atomic<int> failed(0);
        auto worker = [&]() {
            if (cudaSetDevice(ctx->device) != cudaSuccess) { failed = 1; return; }
            for (;;) {
                const uint32_t c = next.fetch_add(1);
                if (c >= n_chunks) break;
                const uint32_t r0 = c * chunk, r1 = std::min(k, r0 + chunk);
                for (uint32_t r = r0; r < r1; r++) {
                    const size_t f = ids[r];
                    memcpy(pin + c_sz + r * r_sz, (const char*)wide_h->size + f * r_sz, r_sz);
                    memcpy(pin + c_ia + r * r_ia, (const char*)wide_h->iat_us + f * r_ia, r_ia);
                    memcpy(pin + c_dr + r * r_dr, (const char*)wide_h->dir_bits + f * r_dr, r_dr);
                    memcpy(pin + c_hd + r * r_hd, (const char*)wide_h->hdr + f * r_hd, r_hd);
                    if (wide_h->n_valid) pin[c_nv + r] = (char)wide_h->n_valid[f];
                }
                const size_t m = r1 - r0;
                cudaError_t e = cudaMemcpyAsync(dv + c_sz + r0 * r_sz, pin + c_sz + r0 * r_sz, m * r_sz, cudaMemcpyHostToDevice, st);
                if (e == cudaSuccess) e = cudaMemcpyAsync(dv + c_ia + r0 * r_ia, pin + c_ia + r0 * r_ia, m * r_ia, cudaMemcpyHostToDevice, st);
                if (e == cudaSuccess) e = cudaMemcpyAsync(dv + c_dr + r0 * r_dr, pin + c_dr + r0 * r_dr, m * r_dr, cudaMemcpyHostToDevice, st);
                if (e == cudaSuccess) e = cudaMemcpyAsync(dv + c_hd + r0 * r_hd, pin + c_hd + r0 * r_hd, m * r_hd, cudaMemcpyHostToDevice, st);
                if (e == cudaSuccess && wide_h->n_valid) e = cudaMemcpyAsync(dv + c_nv + r0, pin + c_nv + r0, m, cudaMemcpyHostToDevice, st);
                if (e != cudaSuccess) failed = 1;
            }
        };
        {
            uint32_t n_thr = std::thread::hardware_concurrency();
            n_thr = std::max(1u, std::min(std::min(n_thr, 16u), n_chunks));
            std::vector<std::thread> pool;
            for (uint32_t i = 1; i < n_thr; i++) pool.emplace_back(worker);
            worker();
            for (auto& th : pool) th.join();
        }
        if (failed) return sf_set_cuda_error(cudaGetLastError(), "compact copy");
        sf_packets wd2 = *wide_h;
        wd2.size = (const uint16_t*)(dv + c_sz); wd2.iat_us = (const uint32_t*)(dv + c_ia);
        wd2.dir_bits = (const uint32_t*)(dv + c_dr); wd2.hdr = (const uint8_t*)(dv + c_hd);
        wd2.n_valid = wide_h->n_valid ? (const uint8_t*)(dv + c_nv) : nullptr;
        wd2.n_flows = k;
        rc = serve_on_device(ctx, fo, s, &fd2, N, F, &wd2, &cd2, (uint8_t*)(sb2 + a_lab), (uint8_t*)(sb2 + a_stg),
                             (uint32_t*)(sb2 + a_ne), st, SF_PHASE_SLOW);
        if (rc != SF_OK) return rc;
        SF_CUDA(cudaMemcpyAsync(label_h, sb2 + a_lab, n, cudaMemcpyDeviceToHost, st));
        SF_CUDA(cudaMemcpyAsync(stage_h, sb2 + a_stg, n, cudaMemcpyDeviceToHost, st));
        if (n_esc_h) *n_esc_h = k;
        SF_CUDA(cudaStreamSynchronize(st));
        return SF_OK;
    }
    auto plane_bytes = [](const sf_packets* p, size_t& s_sz, size_t& s_iat, size_t& s_dir, size_t& s_hdr, size_t& s_nv) {
        s_sz = (size_t)p->n_flows * p->pitch_pkts * 2;
        s_iat = (size_t)p->n_flows * p->pitch_pkts * 4;
        s_dir = (size_t)p->n_flows * ((p->pitch_pkts + 31) / 32) * 4;
        s_hdr = p->hdr ? (size_t)p->n_flows * p->pitch_pkts * p->hdr_bytes : 0;
        s_nv = p->n_valid ? (size_t)p->n_flows : 0;
    };
    size_t off = 0;
    auto take = [&](size_t bytes) { size_t o = off; off += sf_align256(bytes); return o; };
    size_t fs, fi, fd, fh, fv, ws_, wi, wd, wh, wv;
    plane_bytes(fast_h, fs, fi, fd, fh, fv);
    plane_bytes(wide_h, ws_, wi, wd, wh, wv);
    size_t o_fs = 0, o_fi = 0, o_fd = 0, o_fv = 0;
    if (!shared) { o_fs = take(fs); o_fi = take(fi); o_fd = take(fd); }
    o_fv = take(fv);
    size_t o_ws = take(ws_), o_wi = take(wi), o_wd = take(wd), o_wh = take(wh), o_wv = take(wv);
    const uint32_t n_tau = cfg_h->rule == SF_ABSMARGIN_LT ? 1 : fo->C;
    size_t o_tau = take(n_tau * 4), o_label = take(n), o_stage = take(n), o_nesc = take(4);
    if (off > ctx->stage_bytes) {
        SF_CUDA(cudaDeviceSynchronize());
        if (ctx->stage) { cudaFree(ctx->stage); ctx->stage = nullptr; ctx->stage_bytes = 0; }
        cudaError_t e = cudaMalloc(&ctx->stage, off);
        if (e != cudaSuccess) { sf_set_cuda_error(e, "cudaMalloc(staging)"); return SF_ERR_ALLOC; }
        ctx->stage_bytes = off;
    }
    char* sb = ctx->stage;
#define SF_H2D(dst_off, src, bytes) do { if ((bytes) > 0) SF_CUDA(cudaMemcpyAsync(sb + (dst_off), (src), (bytes), cudaMemcpyHostToDevice, st)); } while (0)
    SF_H2D(o_ws, wide_h->size, ws_); SF_H2D(o_wi, wide_h->iat_us, wi); SF_H2D(o_wd, wide_h->dir_bits, wd);
    SF_H2D(o_wh, wide_h->hdr, wh); SF_H2D(o_wv, wide_h->n_valid, wv);
    if (!shared) { SF_H2D(o_fs, fast_h->size, fs); SF_H2D(o_fi, fast_h->iat_us, fi); SF_H2D(o_fd, fast_h->dir_bits, fd); }
    SF_H2D(o_fv, fast_h->n_valid, fv);
    SF_H2D(o_tau, cfg_h->tau, (size_t)n_tau * 4);
#undef SF_H2D
    sf_packets wide_d = *wide_h, fast_d = *fast_h;
    wide_d.size = (const uint16_t*)(sb + o_ws); wide_d.iat_us = (const uint32_t*)(sb + o_wi);
    wide_d.dir_bits = (const uint32_t*)(sb + o_wd); wide_d.hdr = (const uint8_t*)(sb + o_wh);
    wide_d.n_valid = wide_h->n_valid ? (const uint8_t*)(sb + o_wv) : nullptr;
    if (shared) { fast_d.size = wide_d.size; fast_d.iat_us = wide_d.iat_us; fast_d.dir_bits = wide_d.dir_bits; }
    else { fast_d.size = (const uint16_t*)(sb + o_fs); fast_d.iat_us = (const uint32_t*)(sb + o_fi); fast_d.dir_bits = (const uint32_t*)(sb + o_fd); }
    fast_d.hdr = nullptr;
    fast_d.n_valid = fast_h->n_valid ? (const uint8_t*)(sb + o_fv) : nullptr;
    sf_route_cfg cfg_d = *cfg_h;
    cfg_d.tau = (const float*)(sb + o_tau);
    rc = serve_on_device(ctx, fo, s, &fast_d, N, F, &wide_d, &cfg_d, (uint8_t*)(sb + o_label), (uint8_t*)(sb + o_stage),
                         (uint32_t*)(sb + o_nesc), st);
    if (rc != SF_OK) return rc;
    SF_CUDA(cudaMemcpyAsync(label_h, sb + o_label, n, cudaMemcpyDeviceToHost, st));
    SF_CUDA(cudaMemcpyAsync(stage_h, sb + o_stage, n, cudaMemcpyDeviceToHost, st));
    if (n_esc_h) SF_CUDA(cudaMemcpyAsync(n_esc_h, sb + o_nesc, 4, cudaMemcpyDeviceToHost, st));
    SF_CUDA(cudaStreamSynchronize(st));
    return SF_OK;
}

extern "C" int sf_serve_batch_intermediates(sf_ctx* ctx, const float** feat, const float** fast_out,
                                            const uint32_t** esc_ids, const void** rows, const float** logits,
                                            const uint8_t** label_fast, const uint8_t** label_slow)
{
    if (!ctx || !ctx->last_feat) return SF_ERR_ARG;
    if (feat) *feat = ctx->last_feat;
    if (fast_out) *fast_out = ctx->last_fast_out;
    if (esc_ids) *esc_ids = ctx->last_esc_ids;
    if (rows) *rows = ctx->last_rows;
    if (logits) *logits = ctx->last_logits;
    if (label_fast) *label_fast = ctx->last_label_fast;
    if (label_slow) *label_slow = ctx->last_label_slow;
    return SF_OK;
}

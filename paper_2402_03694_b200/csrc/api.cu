// Context, error reporting, workspace, Algorithm 1 on the host, and the composite
// sf_serve_batch call that chains S1..S5 on one stream without host round trips.
#include "common.cuh"
#include <algorithm>
#include <new>
#include <stdio.h>
#include <stdlib.h>
#include <string.h>
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
    size_t feat, fast_out, decision, label_fast, esc_ids, rows, logits, label_slow, route_scratch, slow_scratch, total;
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
    if (cfg->rule == SF_LC_GT && fo->kind != SF_RF) return SF_ERR_ARG;
    if (cfg->rule == SF_ABSMARGIN_LT && fo->kind != SF_GBDT) return SF_ERR_ARG;
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

int serve_on_device(sf_ctx* ctx, const sf_forest* fo, const sf_slow* s, const sf_packets* fast, uint32_t N, uint32_t F,
                    const sf_packets* wide, const sf_route_cfg* cfg, uint8_t* label_out, uint8_t* stage_out,
                    uint32_t* n_esc_out, cudaStream_t st)
{
    const uint32_t n = fast->n_flows;
    const ServePlan p = plan_serve(fo, s, n, F, cfg);
    int rc = sf_ws_reserve(ctx, p.total);
    if (rc != SF_OK) return rc;
    sf_ws_reset(ctx);
    char* base = reinterpret_cast<char*>(sf_ws_alloc(ctx, p.total));
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

    sf_time_new_record(ctx);
    sf_time_begin(ctx, SF_T_EXTRACT, st);
    rc = sf_launch_extract(fast, N, F, feat, st);
    sf_time_end(ctx, SF_T_EXTRACT, st);
    if (rc != SF_OK) return rc;
    sf_time_begin(ctx, SF_T_FOREST, st);
    rc = sf_launch_forest(fo, feat, n, fast_out, nullptr, st);
    sf_time_end(ctx, SF_T_FOREST, st);
    if (rc != SF_OK) return rc;
    rc = sf_launch_route(ctx, cfg, fast_out, n, fo->C, wide, esc_ids, n_esc_out, rows, decision, label_fast, nullptr,
                         base + p.route_scratch, st);
    if (rc != SF_OK) return rc;
    rc = sf_launch_slow(ctx, s, rows, n_esc_dev, cfg->capacity, logits, label_slow, base + p.slow_scratch, st);
    if (rc != SF_OK) return rc;
    sf_time_begin(ctx, SF_T_MERGE, st);
    rc = sf_launch_merge(label_fast, decision, n, esc_ids, n_esc_dev, cfg->capacity, label_slow, label_out, stage_out, st);
    sf_time_end(ctx, SF_T_MERGE, st);
    if (rc != SF_OK) return rc;
    ctx->last_feat = feat; ctx->last_fast_out = fast_out; ctx->last_esc_ids = esc_ids; ctx->last_rows = rows;
    ctx->last_logits = logits; ctx->last_label_fast = label_fast; ctx->last_label_slow = label_slow;
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
    const uint32_t n_tau = cfg_h->rule == SF_LC_GT ? fo->C : 1;
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

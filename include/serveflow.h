/*
 * serveflow.h - C ABI of the B200 (sm_100a) fast-slow flow-serving library.
 *
 * The library runs the data-parallel hot path of the fast-slow serving
 * architecture of "ServeFlow: A Fast-Slow Model Architecture for Network Traffic
 * Analysis": every flow is first answered by a cheap model on its first few
 * packets; an uncertainty score decides which flows are assigned to a slow model
 * that sees more packets of the same flow (Sec. 3.1, Fig. 4; Sec. 3.2).
 *
 * Conventions
 *  - Every call returns an int status: SF_OK (0) or a negative SF_ERR_* code;
 *    sf_strerror() names it.  Nothing aborts or throws across this boundary.
 *  - Unless a parameter says "host", data pointers are DEVICE pointers owned by
 *    the caller, read-only unless named *_out.  Outputs documented as nullable
 *    are skipped when NULL.
 *  - Calls enqueue work on the caller's stream (a cudaStream_t passed as void*,
 *    NULL = the default stream) and do not synchronise, except where stated.
 *  - A context serves ONE stream at a time.  Every compute call on a context uses the
 *    context's single device workspace (grown, when a call needs more, by a synchronising
 *    free + allocate) and its device-side count of assigned flows, so calls on one context
 *    must be ordered on one stream, or by events, and must not be issued from two threads
 *    at once; calls that overlap on the GPU race on the intermediates.  The pointers that
 *    sf_serve_batch_intermediates returns are valid until the next compute call on that
 *    context.  Use one context per stream for concurrent work.
 *  - Handles (sf_ctx, sf_forest, sf_slow, sf_table) are owned by the library,
 *    built from HOST arrays that are copied and re-laid-out inside, and released
 *    by the matching *_destroy.  A handle belongs to the device of its context.
 *  - Arguments are validated on the host before anything is launched.  Device-side
 *    conditions (capacity overflow, a full hash table, a wait that ran out) are
 *    recorded in a device error word that sf_ctx_poll() reads; no kernel traps.
 *  - There is no CPU fallback: without a CUDA device every compute call fails.
 */
#ifndef SERVEFLOW_H
#define SERVEFLOW_H

#include <stddef.h>
#include <stdint.h>

#ifdef __cplusplus
extern "C" {
#endif

#define SF_OK                  0
#define SF_ERR_ARG            -1   /* NULL where not allowed, size out of range, misaligned pointer */
#define SF_ERR_ALLOC          -2   /* device or host allocation failed */
#define SF_ERR_CUDA           -3   /* a CUDA runtime/driver call failed (sf_last_cuda_error) */
#define SF_ERR_CAPACITY       -4   /* more flows were assigned than `capacity`; the list was clamped */
#define SF_ERR_TABLE_FULL     -5   /* a key found no slot within the probe limit; its packet was dropped */
#define SF_ERR_UNSUPPORTED    -6   /* shape outside what the kernels implement */
#define SF_ERR_DEVICE_TIMEOUT -7   /* a bounded device-side wait gave up */
#define SF_ERR_STATIC_LIMIT   -8   /* sf_route_noalloc: more flows than its built-in scratch holds */

/* enums passed as int */
#define SF_RF           0          /* random forest: mean of leaf class-probability vectors */
#define SF_GBDT         1          /* boosted trees, binary logistic: sum of leaf scalars (margin) */
#define SF_GBDT_MC      2          /* boosted trees, multi-class: tree t belongs to class t mod C (one tree per class and
                                      boosting round, the layout of the libraries Sec. 4.4 names); C margins per flow */
#define SF_LC_GT        0          /* assign iff 1 - max_c prob[c] > tau[argmax]  (Sec. 3.2, least confidence) */
#define SF_ABSMARGIN_LT 1          /* assign iff |margin| < tau[0]  (|p-0.5| < 0.2  <=>  |margin| < ln(7/3)) */
#define SF_ENTROPY_GT   2          /* assign iff -sum_c prob[c] ln prob[c] > tau[argmax]  (Sec. 3.2, entropy; fp32 logf:
                                      scores agree with a double-precision evaluation to about 1e-6, not bit for bit) */
#define SF_SOFTMAX_LC_GT 3         /* input = C margins (SF_GBDT_MC): assign iff 1 - max softmax(margin) > tau[argmax], i.e.
                                      1 - 1/sum_j exp(m_j - m_max) (Sec. 3.2's least confidence; fp32 expf, tolerance as above) */
#define SF_MLP16        0          /* wide row = P packets x 16 fields */
#define SF_CNN8         1          /* wide row = P positions x 8 channels (channels last) */
#define SF_F32          0
#define SF_BF16         1

/* |margin| threshold equivalent to |sigmoid(margin) - 0.5| < 0.2: fp32(ln(0.7/0.3)) */
#define SF_TAU_MARGIN_DEFAULT 0x1.b1d106p-1f

typedef struct sf_ctx sf_ctx;
typedef struct sf_forest sf_forest;
typedef struct sf_slow sf_slow;
typedef struct sf_table sf_table;

const char* sf_strerror(int status);
/* Text of the last CUDA error seen by this thread's last failing call (host string, never NULL). */
const char* sf_last_cuda_error(void);
/* Library version and the SM architecture it was compiled for ("sm_100a"). */
const char* sf_version(void);

/* ---- context ------------------------------------------------------------ */
/* Creates a context on `device`: a device workspace of `workspace_bytes` (scan
 * scratch, intermediates of sf_serve_batch; grown with a synchronising
 * reallocation if a later call needs more), device counters and the error word.
 * Fails with SF_ERR_CUDA when no device is present. */
int  sf_ctx_create(sf_ctx** out, int device, size_t workspace_bytes);
void sf_ctx_destroy(sf_ctx* ctx);

typedef struct {
    uint64_t n_flows;                  /* flows seen by sf_route / sf_serve_batch / the table */
    uint64_t n_fast_done;              /* answered by the fast model */
    uint64_t n_escalated;              /* assigned to the slow model */
    uint64_t n_slow_done;              /* answered by the slow model */
    uint64_t n_missed;                 /* dropped: table full */
    uint64_t n_dropped_after_decision; /* packets of flows that already have their answer */
    int32_t  device_error;             /* first SF_ERR_* recorded on the device, or 0 */
    int32_t  reserved;
} sf_counters;
/* Synchronises `stream`, copies the counters to host memory and returns
 * device_error (SF_OK if none).  `reset` != 0 clears counters and error word. */
int  sf_ctx_poll(sf_ctx* ctx, sf_counters* host_out, int reset, void* stream);

/* Per-kernel timing (off by default).  When enabled, every compute call records
 * CUDA events on its stream around each kernel class and keeps the last 64 calls'
 * records.  sf_ctx_get_timing synchronises `stream` and writes SF_N_TIMERS
 * elapsed times in milliseconds (0 for classes the call did not run) of the call
 * made `back` calls ago (0 = the most recent) to host memory. */
#define SF_T_EXTRACT 0   /* S1 feature kernel */
#define SF_T_FOREST  1   /* S2 tree-ensemble kernel */
#define SF_T_SCORE   2   /* S3 score + scan + scatter kernels */
#define SF_T_GATHER  3   /* S3 wide-row gather kernel */
#define SF_T_GEMM    4   /* S4 hidden layers (tensor-core GEMMs, the fp32 dense kernels, or the fused CNN kernel) */
#define SF_T_HEAD    5   /* S4 last layer + argmax */
#define SF_T_MERGE   6   /* S5 merge kernels */
#define SF_T_TABLE   7   /* streaming table kernels */
#define SF_T_PULL    8   /* host entry point: kernel that fetches the assigned flows' rows from pinned host memory */
#define SF_N_TIMERS  9
int  sf_ctx_set_timing(sf_ctx* ctx, int enable);
int  sf_ctx_get_timing(sf_ctx* ctx, uint32_t back, float* ms_host_out, void* stream);

/* ---- packet planes -------------------------------------------------------- */
/* Header planes of n_flows flows with a row pitch of pitch_pkts packets:
 *   size     uint16[n][pitch]          packet length in bytes
 *   iat_us   uint32[n][pitch]          inter-arrival time before the packet, microseconds
 *   dir_bits uint32[n][ceil(pitch/32)] bit (i%32) of word (i/32) = direction of packet i
 *   hdr      uint8 [n][pitch][hdr_bytes]  raw header bytes (only the wide rows use them; may be NULL otherwise)
 *   n_valid  uint8 [n] or NULL         packets actually present (NULL = all)
 * Rows must be 16-byte aligned: pitch*2 and pitch*4 multiples of 16 or the planes
 * are read with narrower loads (any pitch is accepted; base pointers must be
 * aligned to 16 bytes). */
typedef struct {
    const uint16_t* size;
    const uint32_t* iat_us;
    const uint32_t* dir_bits;
    const uint8_t*  hdr;
    const uint8_t*  n_valid;
    uint32_t n_flows, pitch_pkts, hdr_bytes;
} sf_packets;

/* ---- S1: feature extraction ----------------------------------------------- */
/* The pipeline's "feature computation" step (Sec. 1, Fig. 1) for a batch.  For
 * each flow, F = 8*G statistics of the first min(N, n_valid) packets, feature
 * 8g+k: group g = quantity x subset (g0 size/all, g1 iat/all, g2 size/fwd,
 * g3 size/bwd, g4 iat/fwd, g5 iat/bwd, g6 size/turn, g7 iat/turn; fwd = dir bit 0,
 * turn = direction differs from the previous packet), slot k = cnt, sum, min, max,
 * mean, var (population), first, last.  Sums are exact integers (128-bit for the
 * variance numerator) converted to fp32 once, round-to-nearest-even; mean =
 * fp32(sum)/fp32(cnt); var = fp32(cnt*S2 - S1^2)/fp32(cnt^2); empty subset = zeros.
 * feat_out: fp32[n_flows][F] row-major.  N in 1..32, N <= pitch, F in {8,16,..,64}. */
int  sf_extract_features(sf_ctx* ctx, const sf_packets* pk, uint32_t N, uint32_t F,
                         float* feat_out, void* stream);

/* First-packet header-bit features (Sec. 4.1 and 4.4: 1024 header bits per packet from the
 * IPv4, TCP and UDP headers, with a subscription to a subset of the columns).  bytes:
 * uint8[n][128] = IPv4 header bytes 0..59 | TCP header bytes 0..59 | UDP header bytes 0..7
 * (16-byte aligned); sec_len: uint8[n][3] = bytes present in each section; sub: uint16[m]
 * (device), column indices 0..1023, m <= 1024.  Column i is bit (7 - i%8) of byte i/8;
 * out fp32[n][m]: -1 if that byte is not present, else 0 or 1.  With m <= 64 the rows can go
 * straight into sf_fast_infer as the features of a first-packet model. */
int  sf_header_bits(sf_ctx* ctx, const uint8_t* bytes, const uint8_t* sec_len, uint32_t n,
                    const uint16_t* sub, uint32_t m, float* out, void* stream);

/* ---- S2: fast model (tree ensemble) ---------------------------------------- */
/* Builds an ensemble of T complete binary trees of depth `depth` (heap order:
 * children of node i are 2i+1, 2i+2) from HOST arrays fid uint16[T][2^d-1],
 * thr fp32[T][2^d-1], leaf fp32[T][2^d][C] (SF_RF) or fp32[T][2^d] (SF_GBDT, C
 * ignored and treated as 2 classes; SF_GBDT_MC, T a multiple of C).  depth 1..12,
 * F <= 64, C <= 16.  SF_GBDT_MC needs a whole boosting round (C trees of 12*2^d bytes)
 * within one shared-memory chunk, else sf_fast_infer returns SF_ERR_UNSUPPORTED. */
int  sf_forest_create(sf_ctx* ctx, int kind, uint32_t T, uint32_t depth, uint32_t F, uint32_t C,
                      const uint16_t* fid_host, const float* thr_host, const float* leaf_host,
                      sf_forest** out);
void sf_forest_destroy(sf_forest* forest);
/* The fast model of the cascade (Sec. 3.1) on n feature rows fp32[n][F].  At a
 * node a flow goes LEFT iff x[fid] <= thr.  SF_RF: prob[c] = (sum over trees
 * t = 0..T-1, in that order, fp32) of leaf[t][l_t][c], divided by fp32(T) ->
 * out fp32[n][C].  SF_GBDT: margin = sum of leaf[t][l_t] in tree order ->
 * out fp32[n].  SF_GBDT_MC: margin[c] = sum over the trees t = c, c+C, c+2C, ... in that
 * order -> out fp32[n][C].  leaf_idx_out (nullable): uint16[n][T]. */
int  sf_fast_infer(sf_ctx* ctx, const sf_forest* forest, const float* feat, uint32_t n,
                   float* prob_or_margin_out, uint16_t* leaf_idx_out, void* stream);

/* ---- S3: uncertainty score, threshold, compaction, wide rows --------------- */
typedef struct {
    int rule;               /* SF_LC_GT | SF_ABSMARGIN_LT | SF_ENTROPY_GT | SF_SOFTMAX_LC_GT */
    const float* tau;       /* device: fp32[C] per predicted class (all equal = universal threshold) for
                               SF_LC_GT; fp32[1] for SF_ABSMARGIN_LT */
    int wide_layout;        /* SF_MLP16 | SF_CNN8 */
    int row_dtype;          /* SF_BF16 | SF_F32 */
    uint32_t P;             /* packets per wide row (row width D = 16*P or 8*P) */
    uint32_t P_real;        /* packets taken from the planes; positions P_real..P-1 are zero (0 = P) */
    uint32_t capacity;      /* rows available in esc_ids_out / rows_out */
} sf_route_cfg;
/* Flow assignment (Sec. 3.2): score = LC(x) = 1 - max_y P(y|x) (or |margin|),
 * fast label = argmax (lowest index on ties; margin > 0 for SF_GBDT), a flow is
 * assigned to the slow model iff the score passes the threshold (strict
 * comparison).  Assigned flow ids are written in ascending order to
 * esc_ids_out[0..n_esc) and their count to *n_esc_out (device).  If `wide` and
 * rows_out are given, each assigned flow's wide row is gathered and converted:
 * per packet size*2^-11, L(iat)*2^-7 (L = integer piecewise-linear log2 of iat+1,
 * 0..128), direction 0/1, header bytes*2^-8 (13 for SF_MLP16, 5 for SF_CNN8),
 * rounded to bf16 (RNE) or kept fp32.  If more than `capacity` flows qualify the
 * count saturates at capacity and the error word gets SF_ERR_CAPACITY.
 * Nullable: rows_out (with wide), decision_out uint8[n], label_fast_out uint8[n],
 * score_out fp32[n]. */
int  sf_route(sf_ctx* ctx, const sf_route_cfg* cfg, const float* prob_or_margin, uint32_t n, uint32_t C,
              const sf_packets* wide, uint32_t* esc_ids_out, uint32_t* n_esc_out, void* rows_out,
              uint8_t* decision_out, uint8_t* label_fast_out, float* score_out, void* stream);

/* Assignment without any allocation.  (The paper has no counterpart to this call: it
 * exists for the way some programs have to use a GPU library.)
 *
 * Who needs it: code that runs where device memory may not be allocated or freed - a
 * serving loop whose memory was handed out once at start-up and is now fixed, a plug-in
 * running inside another framework's memory pool, a real-time thread that must not take
 * the driver's allocator lock.  Such callers cannot create an sf_ctx (that allocates),
 * so this call takes no context.
 *
 * It does what sf_route does up to the list of assigned flows - score, fast label,
 * strict threshold, ascending ids, count, under any of sf_route's four rules - and
 * gathers no wide rows.  The per-block
 * counts and, when decision_out is NULL, the per-flow decisions go to a fixed array
 * built into the library image (about 4 MB; every GPU that loads the library keeps it
 * until the process ends), so n may be at most SF_NOALLOC_MAX_FLOWS; a larger n is
 * refused with SF_ERR_STATIC_LIMIT before anything is launched.  The call performs no
 * cudaMalloc/cudaFree and calls nothing that allocates.
 *
 * All outputs are device pointers of the caller: esc_ids_out uint32[cfg->capacity],
 * n_esc_out uint32[1]; nullable: decision_out uint8[n], label_fast_out uint8[n],
 * score_out fp32[n], status_out int32[1] (0, or SF_ERR_CAPACITY when more flows
 * qualified than cfg->capacity; the count then saturates as in sf_route).
 * cfg->wide_layout, row_dtype, P and P_real are ignored.
 *
 * The first call on a device looks up the array's device address (a one-time set-up
 * with that device current); make that first call before starting any stream capture.
 * First calls made by several threads at once are harmless (each stores the same address).
 * All calls on a device share the one array and it keeps the previous call's contents
 * (the call clears the part that must start at zero), so two calls whose GPU work
 * overlaps - different streams, or different threads - race; run them one after the
 * other on a stream, or order them with events. */
#define SF_NOALLOC_MAX_FLOWS 4194304u
int  sf_route_noalloc(int device, const sf_route_cfg* cfg, const float* prob_or_margin, uint32_t n, uint32_t C,
                      uint32_t* esc_ids_out, uint32_t* n_esc_out, uint8_t* decision_out, uint8_t* label_fast_out,
                      float* score_out, int32_t* status_out, void* stream);

/* Algorithm 1 (universal uncertainty thresholds) on HOST data: sorts a copy of
 * the n validation scores ascending and returns, for each quantile
 * q = q_num[j]/q_den, the score at 1-based index ceil(q*n).  Host-only helper. */
int  sf_universal_thresholds(const float* scores_host, uint64_t n, const uint32_t* q_num_host,
                             uint32_t q_den, uint32_t n_q, float* thresholds_host_out);

/* Algorithm 1 on DEVICE scores (float32[n], no NaNs): a stable radix sort of the scores on the
 * device, then the same 1-based pick ceil(q*n) per quantile; tau_out is a DEVICE float32[n_q]
 * (n_q <= 64), so it can be handed to sf_route_cfg.tau without a host round trip.  q_num is a
 * host array.  Uses the context's workspace (may grow it, synchronising); asynchronous on
 * `stream` otherwise.  Scores compare as IEEE values with -0 before +0. */
int  sf_universal_thresholds_dev(sf_ctx* ctx, const float* scores, uint32_t n, const uint32_t* q_num_host,
                                 uint32_t q_den, uint32_t n_q, float* tau_out, void* stream);

/* Algorithm 2 (slope-based per-class uncertainty thresholds, Sec. 3.2) on a validation batch
 * that lives on the device: scores float32[n], label uint8[n] = the fast model's predicted
 * class (< C <= 256), correct uint8[n] = 1 where that prediction was right.  Reading of the
 * outline the paper gives: per predicted class the candidate thresholds are the quantiles
 * (Q-k)/Q, k = 1..Q (Q <= 1000), of that class's scores by Algorithm 1's pick; a step's slope
 * is (newly assigned incorrect flows) / (newly assigned flows), steps that assign nothing
 * new are dropped; thresholds start at each class's maximum and, while fewer than
 * floor(a_num/a_den * n) validation flows are assigned, the steepest next step over all
 * classes is taken (fractions compared exactly; ties: the larger step, then the lower
 * class).  A class with no validation flow gets the global maximum score.
 * The device sorts (class, score) keys, picks the thresholds and counts the flows between
 * them; the selection over the <= C*Q steps runs on the host.  tau_host_out: float32[C];
 * assigned_host_out (nullable): validation flows with score > tau[label].  Synchronises
 * `stream`. */
int  sf_per_class_thresholds(sf_ctx* ctx, const float* scores, const uint8_t* label, const uint8_t* correct,
                             uint32_t n, uint32_t C, uint32_t Q, uint32_t a_num, uint32_t a_den,
                             float* tau_host_out, uint64_t* assigned_host_out, void* stream);

/* ---- S4: slow model -------------------------------------------------------- */
/* MLP h_{k+1} = ReLU(W_k h_k + b_k), logits = W_L h_L + b_L.  dims_host has
 * n_layers+1 entries; W_host[k] is fp32 [dims[k+1]][dims[k]] (HOST), b_host[k]
 * fp32[dims[k+1]].  SF_BF16: weights and hidden activations are bf16 (RNE),
 * products accumulate in fp32 on the tensor cores, biases and logits fp32; needs
 * hidden widths that are multiples of 64 and dims[0] a multiple of 64.  SF_F32:
 * plain fp32.  The last layer may have any width up to 16 classes. */
int  sf_mlp_create(sf_ctx* ctx, int dtype, uint32_t n_layers, const uint32_t* dims_host,
                   const float* const* W_host, const float* const* b_host, sf_slow** out);
/* 1-D CNN over L positions x Cin channels (channels last): conv(k) Cin->C1 + ReLU,
 * conv(k) C1->C2 + ReLU (stride 1, zero "same" padding), mean over positions,
 * linear C2->n_cls.  w1 [C1][k][Cin], w2 [C2][k][C1], w3 [n_cls][C2] (HOST, fp32).
 * Implemented shape: L=128, Cin=8, C1=64, C2=128, k=5, n_cls<=16, SF_BF16. */
int  sf_cnn_create(sf_ctx* ctx, int dtype, uint32_t L, uint32_t Cin, uint32_t C1, uint32_t C2, uint32_t k,
                   uint32_t n_cls, const float* w1_host, const float* b1_host, const float* w2_host,
                   const float* b2_host, const float* w3_host, const float* b3_host, sf_slow** out);
void sf_slow_destroy(sf_slow* slow);
/* The slow model of the cascade (Sec. 3.1) on the first *n_rows_dev rows (a DEVICE
 * count, read by the kernels: no host round trip) of rows[capacity][D] (bf16 or
 * fp32 as the model's dtype).  logits_out fp32[capacity][n_cls]; label_out
 * uint8[capacity] (nullable) = argmax, lowest index on ties.  Rows at or beyond
 * the count are not written.  A count above `capacity` is treated as `capacity`
 * (nothing is read or written beyond the buffers) and SF_ERR_CAPACITY is recorded in
 * the error word. */
int  sf_slow_infer(sf_ctx* ctx, const sf_slow* slow, const void* rows, const uint32_t* n_rows_dev,
                   uint32_t capacity, float* logits_out, uint8_t* label_out, void* stream);

/* ---- S1..S5: the whole cascade on one batch -------------------------------- */
/* Features of fast_ctx (first N packets) -> fast model -> assignment -> wide rows
 * of slow_ctx -> slow model -> merge: label_out[f] = slow label if assigned else
 * fast label; stage_out[f] = 1 (fast) or 2 (slow); *n_esc_out (device, nullable)
 * = number assigned.  Intermediates live in the context's workspace.  fast_ctx
 * and slow_ctx may be the same planes.  Results equal the staged calls'. */
int  sf_serve_batch(sf_ctx* ctx, const sf_forest* forest, const sf_slow* slow, const sf_packets* fast_ctx,
                    uint32_t N, uint32_t F, const sf_packets* slow_ctx, const sf_route_cfg* cfg,
                    uint8_t* label_out, uint8_t* stage_out, uint32_t* n_esc_out, void* stream);
/* Same, but every plane pointer of fast_ctx / slow_ctx, cfg->tau, label_out,
 * stage_out and n_esc_out are HOST pointers, and the call returns after
 * synchronising the stream.  With separate fast and slow planes only what the
 * method needs crosses the bus: the fast planes of all flows go up, S1..S3 run,
 * and then only the ASSIGNED flows' slow-context rows follow.  If the slow planes
 * are pinned host memory that the device can address (cudaHostAlloc /
 * cudaHostRegister), a kernel reads those rows straight out of them with no work on
 * the host; otherwise the id list comes back, host threads compact the rows into the
 * context's pinned buffer and they are copied up in chunks.  With shared planes
 * everything is copied to device staging buffers first. */
int  sf_serve_batch_host(sf_ctx* ctx, const sf_forest* forest, const sf_slow* slow, const sf_packets* fast_ctx_host,
                         uint32_t N, uint32_t F, const sf_packets* slow_ctx_host, const sf_route_cfg* cfg_host_tau,
                         uint8_t* label_host_out, uint8_t* stage_host_out, uint32_t* n_esc_host_out, void* stream);
/* Three-tier cascade (Sec. 3.1: the fastest model answers what it is sure of, the fast model
 * looks at the rest using the SAME features, the slow model at what is still uncertain, with
 * more packets; Sec. 3.2: thresholds per predicted class).  The fastest model is an SF_RF
 * ensemble (typically a single tree), the fast model SF_RF with SF_LC_GT or SF_GBDT_MC with
 * SF_SOFTMAX_LC_GT, both over the same F features.
 * cfg_fastest: only rule (SF_LC_GT) and tau (fp32[C of fastest]) are used; cfg_fast: as in
 * sf_serve_batch.  stage_out: 1, 2 or 3.  n_esc_out (device, nullable): uint32[2] = flows
 * passed on by the fastest model, flows assigned to the slow model.  The context counters
 * count routing decisions: n_flows grows by n plus the first count. */
int  sf_serve_batch3(sf_ctx* ctx, const sf_forest* fastest, const sf_forest* fast, const sf_slow* slow,
                     const sf_packets* fast_ctx, uint32_t N, uint32_t F, const sf_packets* slow_ctx,
                     const sf_route_cfg* cfg_fastest, const sf_route_cfg* cfg_fast, uint8_t* label_out,
                     uint8_t* stage_out, uint32_t* n_esc_out, void* stream);
/* Pointers into the workspace to the intermediates of the last sf_serve_batch on
 * this context (for inspection and tests): any out pointer may be NULL. */
int  sf_serve_batch_intermediates(sf_ctx* ctx, const float** feat, const float** fast_out, const uint32_t** esc_ids,
                                  const void** rows, const float** logits, const uint8_t** label_fast,
                                  const uint8_t** label_slow);

/* ---- streaming: device-resident per-flow state table ----------------------- */
/* One batch of interleaved packets, struct of arrays (device).  More than 65,536 packets in one call are
 * ingested as consecutive pieces of 65,536 (the table ends as if each piece had come in its own call). */
typedef struct {
    const uint32_t* src; const uint32_t* dst;     /* addresses */
    const uint16_t* sport; const uint16_t* dport; /* ports */
    const uint8_t*  proto;
    const uint8_t*  dir;                          /* 0/1 */
    const uint16_t* size;
    const uint32_t* iat_us;
    const uint8_t*  hdr;                          /* uint8[n][13] */
    uint32_t n;
} sf_pkt_batch;
typedef struct {
    uint32_t n_new_flows;        /* keys first seen in this batch */
    uint32_t n_fast_fired;       /* flows that reached fast_pkts packets and were scored */
    uint32_t n_fast_done;        /* ... of which answered by the fast model */
    uint32_t n_escalated;        /* ... of which assigned to the slow model */
    uint32_t n_slow_fired;       /* assigned flows that reached slow_pkts packets and were answered */
    uint32_t n_dropped_after_decision;
    uint32_t n_missed;           /* packets dropped because no slot was found */
    uint32_t reserved;
} sf_batch_result;
typedef struct { uint32_t src, dst; uint16_t sport, dport; uint8_t proto; uint8_t pad[3]; } sf_key;
typedef struct {
    uint8_t found;      /* key present */
    uint8_t stage;      /* 0 collecting, 1 answered by the fast model, 2 assigned and waiting, 3 answered by the slow model */
    uint8_t label_fast, label_slow;
    uint32_t n_pkts;    /* packets recorded */
    float score;
} sf_flow_result;
/* The queues of Sec. 3.1 / 4.1 (first-packet features, later packets joined by
 * flow id, escalations) replaced by one device hash table keyed by the 5-tuple:
 * 2^log2_slots slots, linear probing with a bounded probe count; every flow keeps
 * its first fast_pkts packets; flows assigned to the slow model get one of
 * `slow_slabs` slabs holding slow_pkts packets.  fast_pkts in 1..32, fast_pkts < slow_pkts
 * <= 128 (the slow model must see more packets than the fast one, else SF_ERR_ARG). */
int  sf_table_create(sf_ctx* ctx, uint32_t log2_slots, uint32_t fast_pkts, uint32_t slow_pkts,
                     uint32_t slow_slabs, sf_table** out);
void sf_table_destroy(sf_table* table);
/* Ingests one batch in arrival order: look up / insert each key, append the packet
 * to its flow's context, run S1-S3 (F features of the first fast_pkts packets) for
 * flows that just reached fast_pkts packets, and S4 for assigned flows that just
 * reached slow_pkts packets (wide row = slow_pkts real packets zero-padded to
 * cfg->P).  *result_dev (device) receives the batch's counts. */
int  sf_table_ingest(sf_ctx* ctx, sf_table* table, const sf_pkt_batch* batch, const sf_forest* forest,
                     uint32_t F, const sf_slow* slow, const sf_route_cfg* cfg, sf_batch_result* result_dev,
                     void* stream);
/* Same, for a batch in HOST memory (pinned memory makes the copies asynchronous): every plane pointer of
 * batch_host is a host pointer; the planes are copied to a device staging buffer of the context on
 * `stream`, the batch is ingested, the counts are copied to *result_host_out (host) and the stream is
 * synchronised.  cfg->tau stays a DEVICE pointer (thresholds belong to the model, not to the batch). */
int  sf_table_ingest_host(sf_ctx* ctx, sf_table* table, const sf_pkt_batch* batch_host, const sf_forest* forest,
                          uint32_t F, const sf_slow* slow, const sf_route_cfg* cfg, sf_batch_result* result_host_out,
                          void* stream);
int  sf_table_lookup(sf_ctx* ctx, const sf_table* table, const sf_key* keys_dev, uint32_t n,
                     sf_flow_result* out_dev, void* stream);
/* Pipelined ingest (off by default; the paper's server likewise keeps packet collection and inference in separate consumers,
 * Sec. 4.1).  With it on, sf_table_ingest enqueues the look-up and the sort of the batch on the caller's stream and everything
 * from the context update on (S1-S4, table updates, the counts in *result_dev) on a stream of the table's own, so that the next
 * batch's look-up and sort overlap this batch's model work.  Results are the same as without it.  What changes for the caller:
 * *result_dev, the context's counters and the table's state are complete on the caller's stream only after sf_table_flush
 * (sf_table_lookup, sf_table_sweep and sf_table_ingest_host flush by themselves); a batch's input planes and its result_dev
 * must stay untouched until then; every call on the table uses the same stream; the context serves this table only while
 * batches are in flight (its workspace is the model phase's scratch).  Turning it on allocates a second set of per-batch
 * scratch (about 2 MB + 4 bytes per slot) and synchronises the device; turning it off waits for the table's stream. */
int  sf_table_set_pipelined(sf_ctx* ctx, sf_table* table, int on);
/* Makes `stream` wait for the model work of every batch ingested so far (no-op unless pipelined). */
int  sf_table_flush(sf_ctx* ctx, sf_table* table, void* stream);

/* Table lifecycle.  Sec. 3.1 and 4.1: data that waits without a match is discarded after a
 * timeout; the QoE task of Sec. 5.1 needs a monitored flow to be inferred again and again.
 * sf_table_set_time: the time stamp (caller's unit, 32 bits, may wrap) that the packets of
 * the following sf_table_ingest calls carry; a flow remembers the stamp of its last batch.
 * sf_table_sweep: one pass over all slots on `stream`: a flow with now - last_seen >
 * idle_timeout (unsigned 32-bit difference) is discarded whatever its stage - its slot can be
 * claimed by a later flow, its slow-context slab returns to the pool, its key, if it comes
 * back, is a new flow; with rearm != 0 every remaining flow that has its answer (stage 1 or
 * 3) starts a new window (packet count 0, stage 0; the old labels stay readable until the
 * next answer).  result_dev (device) is overwritten with the counts.  Slabs are also returned
 * when the slow model has answered.  Do not overlap a sweep with an ingest on another stream. */
typedef struct {
    uint32_t n_expired_pending;    /* discarded before the fast model ran */
    uint32_t n_expired_assigned;   /* discarded while waiting for their slow context */
    uint32_t n_expired_done;       /* discarded after their answer */
    uint32_t n_rearmed;
    uint32_t n_live;               /* flows in the table after the sweep */
    uint32_t pad[3];
} sf_sweep_result;
int  sf_table_set_time(sf_table* table, uint32_t now);
int  sf_table_sweep(sf_ctx* ctx, sf_table* table, uint32_t now, uint32_t idle_timeout, int rearm,
                    sf_sweep_result* result_dev, void* stream);

#ifdef __cplusplus
}
#endif
#endif /* SERVEFLOW_H */

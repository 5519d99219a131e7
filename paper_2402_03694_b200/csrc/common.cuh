// Internal declarations shared by the translation units of libserveflow.
#pragma once
#include <cuda_runtime.h>
#include <cuda_bf16.h>
#include <stdint.h>
#include <stddef.h>
#include "../../include/serveflow.h"

#define SF_NUM_SMS_DEFAULT 148

// Device-visible block: counters first (mirrors sf_counters), then scratch words.
struct sf_dev_state {
    sf_counters counters;
    uint32_t    scan_total;      // number of assigned flows found by the last route
    uint32_t    blocks_done;     // blocks of the running few-rows layer that have stored their columns (the last one puts it back to zero)
    uint32_t    pad[14];
};

struct sf_ctx {
    int device;
    int num_sms;
    // general workspace (bump-allocated per call)
    char*  ws;
    size_t ws_bytes;
    size_t ws_used;
    // fixed small state
    sf_dev_state* d_state;
    // staging for the host-pointer entry point
    char*  stage;
    size_t stage_bytes;
    char*  stage2;               // compact wide planes of the assigned flows (device) and their pinned host mirror
    char*  pin;
    size_t stage2_bytes;
    size_t pin_bytes;
    cudaStream_t aux;            // second stream of the host entry point (transfers that overlap the kernels)
    cudaEvent_t ev_aux, ev_main;
    // optional per-kernel-class timing: ring of event pairs
    int timing;
    uint32_t t_rec;                               // records started so far
    cudaEvent_t t_ev[64][SF_N_TIMERS][2];
    uint8_t t_used[64][SF_N_TIMERS];
    // intermediates of the last sf_serve_batch
    const float* last_feat; const float* last_fast_out; const uint32_t* last_esc_ids;
    const void* last_rows; const float* last_logits; const uint8_t* last_label_fast;
    const uint8_t* last_label_slow;
};

// nodes 1, 2, 3 (1-based heap) of up to 1024 trees: {threshold bits, byte offset of the feature's row}; a kernel argument
#define SF_FOREST_TOP_TREES 1024
struct sf_forest_top { uint2 n[SF_FOREST_TOP_TREES][3]; };

struct sf_forest {
    sf_ctx* ctx;
    int kind;
    uint32_t T, depth, F, C;
    // per-tree image of tree_stride bytes: 2^depth node entries of 8 bytes {thr bits, byte offset of the
    // feature's row in the kernel's shared-memory tile}, 1-based heap (entry 0 unused), then (GBDT) 2^depth leaf scalars
    unsigned char* d_image;
    unsigned char* d_image_small;      // same trees with feature offsets for the 128-flow tile of the small-batch kernels (random forests only)
    uint32_t tree_stride;
    // leaves: RF fp32[T][2^d][C]; GBDT fp32[T][2^d]
    float* d_leaf;
    cudaTextureObject_t leaf_tex;      // RF with C % 4 == 0: the same table as a linear texture of 16-byte texels (0 = none)
    struct sf_forest_top* h_top;       // host copy of every tree's nodes 1..3, handed to the tree kernel as an argument
    bool top_ok;                       // the kernel variant that reads them is usable (binary boosted trees, T <= 1024, depth >= 2)
};

enum { SF_SLOW_MLP = 0, SF_SLOW_CNN = 1 };

struct sf_slow {
    sf_ctx* ctx;
    int arch;                 // SF_SLOW_MLP | SF_SLOW_CNN
    int dtype;                // SF_F32 | SF_BF16
    uint32_t n_layers;
    uint32_t dims[9];
    void*  d_W[8];            // bf16 or fp32 [out][in]
    float* d_b[8];
    // CNN
    uint32_t L, Cin, C1, C2, k, n_cls;
    void* d_w1; void* d_w2; void* d_w3;      // re-laid-out bf16 operands
    float* d_b1; float* d_b2; float* d_b3;
    float h_cnn_b1[64];                      // conv1 bias, handed to the fused kernel as a launch parameter
};

// ---- helpers ---------------------------------------------------------------
int  sf_set_cuda_error(cudaError_t e, const char* where);      // records text, returns SF_ERR_CUDA
#define SF_CUDA(call) do { cudaError_t e__ = (call); if (e__ != cudaSuccess) return sf_set_cuda_error(e__, #call); } while (0)
#define SF_LAUNCH_CHECK(name) do { cudaError_t e__ = cudaGetLastError(); if (e__ != cudaSuccess) return sf_set_cuda_error(e__, name); } while (0)

// ---- chained launches ---------------------------------------------------------
// A kernel launched with sf_launch_chained may be scheduled while the previous kernel of the stream is still draining (programmatic
// stream serialisation): its blocks are set up early and the gap between two short dependent kernels shrinks.  Such a kernel's FIRST
// statement, before any return and any access to global memory, must be sf_chain_enter(): it lets the kernel after it be set up
// early in turn, then waits until every earlier kernel of the stream has completed and its writes are visible.  Launched the plain
// way the same kernel runs unchanged (both instructions are no-ops then).
#ifdef __CUDACC__
__device__ __forceinline__ void sf_chain_release() { asm volatile("griddepcontrol.launch_dependents;" ::: "memory"); }
__device__ __forceinline__ void sf_chain_wait() { asm volatile("griddepcontrol.wait;" ::: "memory"); }
__device__ __forceinline__ void sf_chain_enter() { sf_chain_release(); sf_chain_wait(); }
// (A kernel may instead call sf_chain_release() first and sf_chain_wait() later, in every thread that goes on to touch global
// memory other than constant model data: what it does in between - barrier set-up, loading weights - overlaps its predecessor.)
template <typename... KArgs, typename... Args>
inline cudaError_t sf_launch_chained(void (*kernel)(KArgs...), dim3 grid, dim3 block, size_t smem, cudaStream_t st, Args... args) {
    cudaLaunchConfig_t lc = {};
    lc.gridDim = grid; lc.blockDim = block; lc.dynamicSmemBytes = smem; lc.stream = st;
    cudaLaunchAttribute at[1];
    at[0].id = cudaLaunchAttributeProgrammaticStreamSerialization;
    at[0].val.programmaticStreamSerializationAllowed = 1;
    lc.attrs = at; lc.numAttrs = 1;
    return cudaLaunchKernelEx(&lc, kernel, args...);
}
#endif

// timing: sf_time_new_record at the start of a public compute call, begin/end around kernels
void sf_time_new_record(sf_ctx* ctx);
void sf_time_begin(sf_ctx* ctx, int slot, cudaStream_t st);
void sf_time_end(sf_ctx* ctx, int slot, cudaStream_t st);

// workspace: reset at the start of a composite call, then bump-allocate (256-byte aligned)
int   sf_ws_reserve(sf_ctx* ctx, size_t bytes);     // ensure capacity (may reallocate, synchronising)
void  sf_ws_reset(sf_ctx* ctx);
void* sf_ws_alloc(sf_ctx* ctx, size_t bytes);       // NULL if the reservation was too small
static inline size_t sf_align256(size_t b) { return (b + 255) & ~(size_t)255; }

// Assignment folded into the tree kernel's epilogue (the composite call on large batches): with tau set, every live flow's
// fast label, decision byte, final label (= fast label) and stage (= 1) are written by the tree kernel, and
// block_counts[b] = assigned flows among flows [b * SF_FOREST_BLOCK, (b + 1) * SF_FOREST_BLOCK).
#define SF_FOREST_BLOCK 512u
struct sf_fused_route {
    const float* tau;             // nullptr: not fused
    int rule;                     // SF_LC_GT (random forest) or SF_ABSMARGIN_LT (binary boosted trees)
    uint8_t* decision; uint8_t* label_fast; uint8_t* label_out; uint8_t* stage_out;
    uint32_t* block_counts;
};

// ---- internal launchers (each validates nothing; callers did) ---------------
int sf_launch_extract(const sf_packets* pk, uint32_t N, uint32_t F, float* feat, cudaStream_t st,
                      const uint32_t* n_dev = nullptr,    // n_dev: optional device-side flow count (<= pk->n_flows)
                      const uint32_t* row_ids = nullptr); // row_ids: optional, flow f's packets are row row_ids[f] of the planes
int sf_launch_forest(const sf_forest* fo, const float* feat, uint32_t n, float* out, uint16_t* leaf_idx, cudaStream_t st,
                     const uint32_t* n_dev = nullptr, bool small_tiles = false,    // small_tiles + leaf_idx (used as scratch): few flows per launch, trees spread over the grid
                     const sf_fused_route* fused = nullptr);                       // fused: see sf_fused_route (SF_RF / SF_GBDT, whole batch, n_dev unused)
// what is left of the assignment after a tree kernel that took the decisions: scan of its block counts, ascending ids, gather
int sf_launch_route_after_fused(sf_ctx* ctx, const sf_route_cfg* cfg, uint32_t n, const sf_packets* wide, uint32_t* esc_ids,
                                uint32_t* n_esc, void* rows, const uint8_t* decision, uint32_t* block_counts, cudaStream_t st);
// route scratch: block_counts uint32[ceil(n/1024)+1], decision bytes if the caller gave none
size_t sf_route_scratch_bytes(uint32_t n);
int sf_launch_route(sf_ctx* ctx, const sf_route_cfg* cfg, const float* fast_out, uint32_t n, uint32_t C,
                    const sf_packets* wide, uint32_t* esc_ids, uint32_t* n_esc, void* rows,
                    uint8_t* decision, uint8_t* label_fast, float* score, void* scratch, cudaStream_t st,
                    const uint32_t* n_dev = nullptr);       // n_dev: optional device-side count of scored flows (<= n)
int sf_launch_score(const sf_route_cfg* cfg, const float* fast_out, uint32_t n, uint32_t C, uint8_t* decision,
                    uint8_t* label, float* score, uint32_t* block_counts, const uint32_t* n_dev, cudaStream_t st);
int sf_launch_iota(uint32_t* out, uint32_t n, cudaStream_t st);      // out[i] = i
int sf_launch_gather(sf_ctx* ctx, const sf_route_cfg* cfg, const sf_packets* wide, const uint32_t* ids,
                     const uint32_t* n_ids_dev, uint32_t capacity, void* rows, cudaStream_t st);
size_t sf_slow_scratch_bytes(const sf_slow* s, uint32_t capacity);
int sf_launch_slow(sf_ctx* ctx, const sf_slow* s, const void* rows, const uint32_t* n_rows_dev, uint32_t capacity,
                   float* logits, uint8_t* label, void* scratch, cudaStream_t st, bool count_done = true);
int sf_launch_merge(const uint8_t* label_fast, const uint8_t* decision, uint32_t n, const uint32_t* esc_ids,
                    const uint32_t* n_esc, uint32_t capacity, const uint8_t* label_slow,
                    uint8_t* label, uint8_t* stage, cudaStream_t st, uint8_t stage_value = 2, bool write_fast = true,
                    sf_dev_state* count_slow_done = nullptr);       // count_slow_done: also add the list's length to n_slow_done
int sf_launch_gather_feat(const float* feat, const uint32_t* ids, const uint32_t* n_dev, uint32_t n_max, uint32_t F,
                          float* out, cudaStream_t st);
int sf_launch_compose_ids(const uint32_t* ids1, const uint32_t* ids2_local, const uint32_t* n_dev, uint32_t n_max,
                          uint32_t* out, cudaStream_t st);

// small batches of a random forest in two steps (forest.cu): leaf indices only; the caller adds the leaf vectors itself
int sf_launch_forest_leaf_index(const sf_forest* fo, const float* feat, uint32_t n, uint16_t* leaf_idx, cudaStream_t st,
                                const uint32_t* n_dev);

// the same with the features computed inside the kernel from the flows' packets (rows row_ids[0..n) of pk, first N packets);
// SF_ERR_UNSUPPORTED when the planes are not laid out for it (the caller then runs the two kernels)
int sf_launch_forest_leaf_index_packets(const sf_forest* fo, const sf_packets* pk, uint32_t N, const uint32_t* row_ids, uint32_t n,
                                        uint16_t* leaf_idx, cudaStream_t st, const uint32_t* n_dev);

// bf16 tensor-core layers (gemm_tc.cu)
int sf_mlp_bf16_forward(sf_ctx* ctx, const sf_slow* s, const void* rows, const uint32_t* n_rows_dev, uint32_t capacity,
                        float* logits, uint8_t* label, void* scratch, cudaStream_t st);
int sf_cnn_bf16_forward(sf_ctx* ctx, const sf_slow* s, const void* rows, const uint32_t* n_rows_dev, uint32_t capacity,
                        float* logits, uint8_t* label, void* scratch, cudaStream_t st);
int sf_cnn_prepare(sf_slow* s, const float* w1, const float* b1, const float* w2, const float* b2,
                   const float* w3, const float* b3);

// record a device-side condition once (first error wins)
__device__ __forceinline__ void sf_dev_set_error(sf_dev_state* st, int code) {
    atomicCAS(&st->counters.device_error, 0, code);
}

// A row count that lives in device memory is the caller's word: the slow-model kernels take at most
// `capacity` rows (what the buffers hold) and record SF_ERR_CAPACITY when the word said more.
__device__ __forceinline__ uint32_t sf_clamp_rows(uint32_t n_rows, uint32_t capacity, sf_dev_state* st) {
    if (n_rows <= capacity) return n_rows;
    if (st && blockIdx.x == 0 && blockIdx.y == 0 && threadIdx.x == 0) sf_dev_set_error(st, SF_ERR_CAPACITY);
    return capacity;
}

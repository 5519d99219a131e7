// S2: tree-ensemble inference (the cascade's fast model).
//
// One thread per flow; a block owns a tile of flows whose feature rows sit in
// shared memory transposed ([feature][flow], so a lane's read of x[fid] hits bank
// = lane whatever fid is).  The ensemble streams through shared memory in chunks
// of whole trees (8-byte nodes {thr, fid}, 1-based heap), double-buffered with
// cp.async so the next chunk loads while the block walks the current one.  A
// thread adds its leaf payloads in tree order t = 0..T-1, which fixes the fp32
// summation order; random-forest leaf vectors are gathered from L2 one tree ahead
// of their use so the gather latency hides behind the next tree's walk.
#include "common.cuh"
#include <new>
#include <stdlib.h>
#include <string.h>

namespace {

constexpr int kChunkBytes = 32 * 1024;     // one depth-12 tree of 8-byte nodes

__device__ __forceinline__ void cp_async16(void* smem, const void* gmem) {
    uint32_t s = (uint32_t)__cvta_generic_to_shared(smem);
    asm volatile("cp.async.cg.shared.global [%0], [%1], 16;\n" ::"r"(s), "l"(gmem) : "memory");
}
__device__ __forceinline__ void cp_async_commit() { asm volatile("cp.async.commit_group;\n" ::: "memory"); }
template <int N>
__device__ __forceinline__ void cp_async_wait() { asm volatile("cp.async.wait_group %0;\n" ::"n"(N) : "memory"); }

__device__ __forceinline__ uint32_t walk_tree(const uint2* __restrict__ nodes, const float* __restrict__ xcol,
                                              uint32_t B, uint32_t depth) {
    uint32_t i = 1;
    for (uint32_t l = 0; l < depth; l++) {
        uint2 nd = nodes[i];
        float x = xcol[nd.y * B];
        i = 2 * i + ((x <= __uint_as_float(nd.x)) ? 0u : 1u);
    }
    return i - (1u << depth);
}

// KIND: SF_RF (leaf = C-vector of class probabilities) or SF_GBDT (leaf = scalar, C = 1).
template <int KIND, int C>
__global__ void forest_kernel(const float* __restrict__ feat, uint32_t n, uint32_t F,
                              const uint2* __restrict__ nodes, const float* __restrict__ leaf,
                              uint32_t T, uint32_t depth, uint32_t trees_per_chunk,
                              float* __restrict__ out, uint16_t* __restrict__ leaf_idx)
{
    extern __shared__ __align__(16) unsigned char smem_raw[];
    const uint32_t B = blockDim.x;
    uint2* buf0 = reinterpret_cast<uint2*>(smem_raw);
    uint2* buf1 = reinterpret_cast<uint2*>(smem_raw + kChunkBytes);
    float* xs = reinterpret_cast<float*>(smem_raw + 2 * kChunkBytes);       // [F][B]
    const uint32_t f0 = blockIdx.x * B;
    const uint32_t f = f0 + threadIdx.x;
    const bool live = f < n;
    const uint32_t tree_nodes = 1u << depth;                 // entries per tree (entry 0 unused)
    const uint32_t n_chunks = (T + trees_per_chunk - 1) / trees_per_chunk;

    auto issue_chunk = [&](uint32_t ck, uint2* dst) {
        uint32_t t0 = ck * trees_per_chunk;
        uint32_t nt = min(trees_per_chunk, T - t0);
        uint32_t vecs = nt * tree_nodes / 2;                 // 16-byte units
        const uint4* src = reinterpret_cast<const uint4*>(nodes + (size_t)t0 * tree_nodes);
        uint4* d4 = reinterpret_cast<uint4*>(dst);
        for (uint32_t v = threadIdx.x; v < vecs; v += B) cp_async16(d4 + v, src + v);
        cp_async_commit();
    };

    issue_chunk(0, buf0);
    // feature tile, transposed
    if (live) {
        const float* row = feat + (size_t)f * F;
        if ((F & 3) == 0) {
            for (uint32_t j = 0; j < F; j += 4) {
                float4 v = __ldg(reinterpret_cast<const float4*>(row + j));
                xs[(j + 0) * B + threadIdx.x] = v.x; xs[(j + 1) * B + threadIdx.x] = v.y;
                xs[(j + 2) * B + threadIdx.x] = v.z; xs[(j + 3) * B + threadIdx.x] = v.w;
            }
        } else {
            for (uint32_t j = 0; j < F; j++) xs[j * B + threadIdx.x] = row[j];
        }
    } else {
        for (uint32_t j = 0; j < F; j++) xs[j * B + threadIdx.x] = 0.0f;
    }

    float acc[C];
    float pend[C];
#pragma unroll
    for (int c = 0; c < C; c++) { acc[c] = 0.0f; pend[c] = 0.0f; }
    bool have_pend = false;
    const float* xcol = xs + threadIdx.x;

    for (uint32_t ck = 0; ck < n_chunks; ck++) {
        uint2* cur = (ck & 1) ? buf1 : buf0;
        if (ck + 1 < n_chunks) { issue_chunk(ck + 1, (ck & 1) ? buf0 : buf1); cp_async_wait<1>(); }
        else cp_async_wait<0>();
        __syncthreads();
        const uint32_t t0 = ck * trees_per_chunk;
        const uint32_t nt = min(trees_per_chunk, T - t0);
        for (uint32_t tt = 0; tt < nt; tt++) {
            const uint32_t t = t0 + tt;
            const uint32_t l = walk_tree(cur + (size_t)tt * tree_nodes, xcol, B, depth);
            if (leaf_idx && live) leaf_idx[(size_t)f * T + t] = (uint16_t)l;
            if (KIND == SF_GBDT) {
                acc[0] = __fadd_rn(acc[0], __ldg(leaf + (size_t)t * tree_nodes + l));
            } else {
                // add the previous tree's vector (already in flight), then fetch this one
                if (have_pend) {
#pragma unroll
                    for (int c = 0; c < C; c++) acc[c] = __fadd_rn(acc[c], pend[c]);
                }
                const float* lv = leaf + ((size_t)t * tree_nodes + l) * C;
                if ((C & 3) == 0) {
#pragma unroll
                    for (int c = 0; c < C; c += 4) {
                        float4 v = __ldg(reinterpret_cast<const float4*>(lv + c));
                        pend[c] = v.x; pend[c + 1] = v.y; pend[c + 2] = v.z; pend[c + 3] = v.w;
                    }
                } else {
#pragma unroll
                    for (int c = 0; c < C; c++) pend[c] = __ldg(lv + c);
                }
                have_pend = true;
            }
        }
        __syncthreads();          // everyone is done with `cur` before it is refilled
    }
    if (!live) return;
    if (KIND == SF_GBDT) {
        out[f] = acc[0];
    } else {
        const float fT = __uint2float_rn(T);
#pragma unroll
        for (int c = 0; c < C; c++) {
            float a = have_pend ? __fadd_rn(acc[c], pend[c]) : acc[c];
            out[(size_t)f * C + c] = __fdiv_rn(a, fT);
        }
    }
}

template <int KIND, int C>
int launch(const sf_forest* fo, const float* feat, uint32_t n, float* out, uint16_t* leaf_idx, cudaStream_t st) {
    const uint32_t tree_bytes = (1u << fo->depth) * 8u;
    const uint32_t tpc = kChunkBytes / tree_bytes;                 // >= 1 for depth <= 12
    // block of 512 flows while the feature tile fits, else 256
    uint32_t B = 512;
    size_t smem = 2 * (size_t)kChunkBytes + (size_t)fo->F * B * sizeof(float);
    if (smem > 200 * 1024) { B = 256; smem = 2 * (size_t)kChunkBytes + (size_t)fo->F * B * sizeof(float); }
    auto k = forest_kernel<KIND, C>;
    SF_CUDA(cudaFuncSetAttribute(k, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)smem));
    const uint32_t grid = (n + B - 1) / B;
    k<<<grid, B, smem, st>>>(feat, n, fo->F, fo->d_nodes, fo->d_leaf, fo->T, fo->depth, tpc, out, leaf_idx);
    SF_LAUNCH_CHECK("forest_kernel");
    return SF_OK;
}

}  // namespace

int sf_launch_forest(const sf_forest* fo, const float* feat, uint32_t n, float* out, uint16_t* leaf_idx, cudaStream_t st) {
    if (n == 0) return SF_OK;
    if (fo->kind == SF_GBDT) return launch<SF_GBDT, 1>(fo, feat, n, out, leaf_idx, st);
    switch (fo->C) {
    case 1:  return launch<SF_RF, 1>(fo, feat, n, out, leaf_idx, st);
    case 2:  return launch<SF_RF, 2>(fo, feat, n, out, leaf_idx, st);
    case 3:  return launch<SF_RF, 3>(fo, feat, n, out, leaf_idx, st);
    case 4:  return launch<SF_RF, 4>(fo, feat, n, out, leaf_idx, st);
    case 5:  return launch<SF_RF, 5>(fo, feat, n, out, leaf_idx, st);
    case 6:  return launch<SF_RF, 6>(fo, feat, n, out, leaf_idx, st);
    case 7:  return launch<SF_RF, 7>(fo, feat, n, out, leaf_idx, st);
    case 8:  return launch<SF_RF, 8>(fo, feat, n, out, leaf_idx, st);
    case 9:  return launch<SF_RF, 9>(fo, feat, n, out, leaf_idx, st);
    case 10: return launch<SF_RF, 10>(fo, feat, n, out, leaf_idx, st);
    case 11: return launch<SF_RF, 11>(fo, feat, n, out, leaf_idx, st);
    case 12: return launch<SF_RF, 12>(fo, feat, n, out, leaf_idx, st);
    case 13: return launch<SF_RF, 13>(fo, feat, n, out, leaf_idx, st);
    case 14: return launch<SF_RF, 14>(fo, feat, n, out, leaf_idx, st);
    case 15: return launch<SF_RF, 15>(fo, feat, n, out, leaf_idx, st);
    case 16: return launch<SF_RF, 16>(fo, feat, n, out, leaf_idx, st);
    }
    return SF_ERR_UNSUPPORTED;
}

extern "C" int sf_forest_create(sf_ctx* ctx, int kind, uint32_t T, uint32_t depth, uint32_t F, uint32_t C,
                                const uint16_t* fid, const float* thr, const float* leaf, sf_forest** out)
{
    if (!ctx || !fid || !thr || !leaf || !out) return SF_ERR_ARG;
    if (kind != SF_RF && kind != SF_GBDT) return SF_ERR_ARG;
    if (T < 1 || depth < 1 || depth > 12 || F < 1 || F > 64) return SF_ERR_ARG;
    if (kind == SF_RF && (C < 1 || C > 16)) return SF_ERR_ARG;
    SF_CUDA(cudaSetDevice(ctx->device));
    const uint32_t n_int = (1u << depth) - 1u, n_ent = 1u << depth;
    for (size_t i = 0; i < (size_t)T * n_int; i++) if (fid[i] >= F) return SF_ERR_ARG;
    sf_forest* fo = new (std::nothrow) sf_forest();
    if (!fo) return SF_ERR_ALLOC;
    fo->ctx = ctx; fo->kind = kind; fo->T = T; fo->depth = depth; fo->F = F; fo->C = (kind == SF_GBDT) ? 1 : C;
    fo->d_nodes = nullptr; fo->d_leaf = nullptr;
    // 1-based heap: host node i (0-based, children 2i+1 / 2i+2) becomes entry i+1 (children 2j, 2j+1)
    uint2* h = (uint2*)malloc(sizeof(uint2) * (size_t)T * n_ent);
    if (!h) { delete fo; return SF_ERR_ALLOC; }
    for (uint32_t t = 0; t < T; t++) {
        h[(size_t)t * n_ent] = make_uint2(0u, 0u);
        for (uint32_t i = 0; i < n_int; i++) {
            uint32_t bits; float v = thr[(size_t)t * n_int + i];
            memcpy(&bits, &v, 4);
            h[(size_t)t * n_ent + i + 1] = make_uint2(bits, (uint32_t)fid[(size_t)t * n_int + i]);
        }
    }
    size_t leaf_count = (size_t)T * n_ent * fo->C;
    cudaError_t e = cudaMalloc(&fo->d_nodes, sizeof(uint2) * (size_t)T * n_ent);
    if (e == cudaSuccess) e = cudaMalloc(&fo->d_leaf, sizeof(float) * leaf_count);
    if (e == cudaSuccess) e = cudaMemcpy(fo->d_nodes, h, sizeof(uint2) * (size_t)T * n_ent, cudaMemcpyHostToDevice);
    if (e == cudaSuccess) e = cudaMemcpy(fo->d_leaf, leaf, sizeof(float) * leaf_count, cudaMemcpyHostToDevice);
    free(h);
    if (e != cudaSuccess) { sf_forest_destroy(fo); return sf_set_cuda_error(e, "sf_forest_create"); }
    *out = fo;
    return SF_OK;
}

extern "C" void sf_forest_destroy(sf_forest* fo) {
    if (!fo) return;
    if (fo->d_nodes) cudaFree(fo->d_nodes);
    if (fo->d_leaf) cudaFree(fo->d_leaf);
    delete fo;
}

extern "C" int sf_fast_infer(sf_ctx* ctx, const sf_forest* fo, const float* feat, uint32_t n,
                             float* out, uint16_t* leaf_idx_out, void* stream)
{
    if (!ctx || !fo || !feat || !out) return SF_ERR_ARG;
    if (((uintptr_t)feat & 15) != 0) return SF_ERR_ARG;
    SF_CUDA(cudaSetDevice(ctx->device));
    sf_time_new_record(ctx);
    sf_time_begin(ctx, SF_T_FOREST, (cudaStream_t)stream);
    int rc = sf_launch_forest(fo, feat, n, out, leaf_idx_out, (cudaStream_t)stream);
    sf_time_end(ctx, SF_T_FOREST, (cudaStream_t)stream);
    return rc;
}

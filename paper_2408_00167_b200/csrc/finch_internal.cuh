// Internal declarations shared by the translation units of libfinch (not part of the public ABI).
#pragma once

#include <cuda_bf16.h>
#include <cuda_runtime.h>
#include <stdint.h>

#include "finch.h"

namespace finch {

// Device-side view of a finch_tensor (strides in elements, head_dim contiguous).
struct TensorView {
    const char *ptr;
    int64_t stride_layer, stride_head, stride_tok;
};

struct BatchView {
    int batch;
    const int *q_off, *chunk_off, *cache_off, *cache_len, *budget;
    int total_q, total_chunk, total_cache;
    int max_q, max_cache, max_chunk, max_budget;
    const float *self_lse;  // optional extra softmax-denominator term per prompt row (natural log), or null
    const int *row_limit;   // optional visible-candidate count per query row [total_q], or null
    int row_norm;           // scale a row's weights by the fraction of the candidates it sees
};

struct ModelView {
    int L, Hq, Hkv, d;
    int G;           // selection groups per layer
    int hpg;         // query heads per selection group
    int g;           // query heads per KV head
    int kvpg;        // KV heads per selection group
    float scale;     // logit scale (natural units)
    int elem_bytes;  // 2 (bf16) or 4 (f32)
    float rope_theta;  // rotary base for re-positioning kept keys, 0 = plain copies
    int rope_pairing;  // 0: pairs (t, t + d/2), 1: pairs (2t, 2t + 1)
    // (cos, sin) of n * theta^(-2t/d) for n = 0 .. rope_rows - 1 and t = 0 .. d/2 - 1, [rope_rows][d/2]; device
    // memory owned by the context, computed in double on the host when the context is created
    const float2 *rope_table;
    int rope_rows;
};

struct Ctx {
    finch_config cfg;
    ModelView model;
    int *d_status;  // device status word (nullptr for a validation-only context)
    bool dry;       // validation-only context: nothing is ever enqueued
    int sm_count;
    mutable uint64_t launches;  // kernels enqueued through this context
    // finch_step_host only: a second stream carries the chunk's V rows to the device while the scoring kernels,
    // which do not read them, already run; events tie it to the caller's stream on both sides
    cudaStream_t copy_stream;
    cudaEvent_t ev_entry, ev_v_ready, ev_selected;
};

inline TensorView view_of(const finch_tensor *t) {
    return TensorView{(const char *)t->ptr, t->stride_layer, t->stride_head, t->stride_tok};
}
inline BatchView view_of(const finch_batch *b) {
    return BatchView{b->batch,       b->q_off,       b->chunk_off, b->cache_off, b->cache_len, b->budget,    b->total_q,
                     b->total_chunk, b->total_cache, b->max_q,     b->max_cache, b->max_chunk, b->max_budget,
                     b->prompt_self_lse, b->row_limit, b->row_norm};
}

constexpr float kLog2e = 1.4426950408889634f;
constexpr float kLn2 = 0.6931471805599453f;

// What every kernel needs to know about one unit = (layer, selection group, request).
struct UnitInfo {
    int l, G, b;
    int n_q, c, m, N;
    int q0, cache0, chunk0, cap;
    bool ok;
};

__device__ __forceinline__ UnitInfo unit_info(const ModelView &mv, const BatchView &bv, int unit, int b) {
    UnitInfo u;
    u.l = unit / mv.G;
    u.G = unit % mv.G;
    u.b = b;
    u.q0 = bv.q_off[b];
    u.n_q = bv.q_off[b + 1] - u.q0;
    u.cache0 = bv.cache_off[b];
    u.cap = bv.cache_off[b + 1] - u.cache0;
    u.chunk0 = bv.chunk_off[b];
    u.c = bv.cache_len[b];
    u.m = bv.chunk_off[b + 1] - u.chunk0;
    u.N = u.c + u.m;
    // lengths within the host bounds, and every region inside its packed tensor (the offsets come from device memory)
    u.ok = u.n_q >= 0 && u.n_q <= bv.max_q && u.c >= 0 && u.c <= bv.max_cache && u.m >= 0 && u.m <= bv.max_chunk &&
           u.c <= u.cap && u.q0 >= 0 && u.q0 <= bv.total_q - u.n_q && u.cache0 >= 0 && u.cap >= 0 &&
           u.cache0 <= bv.total_cache - u.cap && u.chunk0 >= 0 && u.chunk0 <= bv.total_chunk - u.m;
    return u;
}

// ---- programmatic dependent launch: the kernels of a step form a chain on one stream.  Launched with the
// programmatic-serialization attribute, a kernel may be scheduled while its predecessor is still running; it then
// executes everything that does not touch global memory (barrier set-up, tensor-memory allocation), and blocks
// in dependency_wait() until the predecessor has completed and its writes are visible.  Every kernel of the chain
// calls dependency_wait() unconditionally, before its first global access and before any early return, so that
// completion of a kernel always implies completion of everything before it.  Only kernels whose whole grid is
// resident at once call dependents_may_launch(): CTAs of the next kernel that arrive early and park in their wait
// would otherwise hold registers and thread slots that later waves of the running kernel need.
__device__ __forceinline__ void dependency_wait() { asm volatile("griddepcontrol.wait;" ::: "memory"); }
__device__ __forceinline__ void dependents_may_launch() { asm volatile("griddepcontrol.launch_dependents;" ::: "memory"); }

template <typename... Params, typename... Args>
cudaError_t launch_chained(void (*kernel)(Params...), dim3 grid, dim3 block, size_t smem, cudaStream_t stream,
                           Args &&...args) {
    cudaLaunchConfig_t cfg = {};
    cfg.gridDim = grid;
    cfg.blockDim = block;
    cfg.dynamicSmemBytes = smem;
    cfg.stream = stream;
    cudaLaunchAttribute attr[1];
    attr[0].id = cudaLaunchAttributeProgrammaticStreamSerialization;
    attr[0].val.programmaticStreamSerializationAllowed = 1;
    cfg.attrs = attr;
    cfg.numAttrs = 1;
    return cudaLaunchKernelEx(&cfg, kernel, Params(args)...);
}

// ---- launchers implemented in the kernel files; each returns the cudaError_t of its launches ----

// warp-level dot-product scoring (any dtype, any prompt length).  row_stats [L][Hq][total_q] is scratch that holds
// (max base-2 logit, 1 / sum of exp2) per prompt row; row_lse (nullable) is the caller-visible natural-log copy.
cudaError_t launch_score_simt(const Ctx &ctx, const TensorView &q, const TensorView &cache_k, const TensorView &chunk_k,
                              const BatchView &bv, float *scores, float2 *row_stats, float *row_lse,
                              cudaStream_t stream);

// tensor-core scoring (bf16, head_dim 64 or 128, either group mode).  The scratch
// holds one float2 per prompt row and key split; up to kScoreMaxSplits splits are used when it is large enough.
constexpr int kScoreMaxSplits = 8;
bool score_tc_supported(const Ctx &ctx);
size_t score_tc_scratch_min(const Ctx &ctx, const BatchView &bv);  // least scratch (float2) of the two-launch path
cudaError_t launch_score_tc(const Ctx &ctx, const TensorView &q, const TensorView &cache_k, const TensorView &chunk_k,
                            const BatchView &bv, float *scores, float2 *partial, size_t partial_capacity,
                            float *row_lse, cudaStream_t stream);

// both sweeps in one persistent kernel (single-request batches without a row mask whose query tiles fit the shared
// memory): score_fused_scratch gives the float2 entries of scratch it needs, 0 when it does not take the batch
size_t score_fused_scratch(const Ctx &ctx, const BatchView &bv);
int score_fused_window(const Ctx &ctx, const BatchView &bv);  // key tiles per window; 0: the batch goes elsewhere
cudaError_t launch_score_fused(const Ctx &ctx, const TensorView &q, const TensorView &cache_k, const TensorView &chunk_k,
                               const BatchView &bv, float *scores, float2 *scratch, size_t scratch_capacity,
                               float *row_lse, cudaStream_t stream);

// scoring dispatch shared by finch_score, finch_score_static and finch_step; `scratch` holds scratch_capacity
// float2 entries, at least one per prompt row (n_layers * n_q_heads * total_q)
cudaError_t run_score(const Ctx &ctx, const TensorView &q, const TensorView &cache_k, const TensorView &chunk_k,
                      const BatchView &bv, float *scores, float2 *scratch, size_t scratch_capacity, float *row_lse,
                      cudaStream_t stream);

cudaError_t launch_select(const Ctx &ctx, const float *scores, const BatchView &bv, int *kept_idx, int *out_len,
                          cudaStream_t stream);

cudaError_t launch_compact(const Ctx &ctx, const int *kept_idx, const int *out_len, const TensorView &cache_k,
                           const TensorView &cache_v, const int *cache_pos, const TensorView &chunk_k,
                           const TensorView &chunk_v, const int *chunk_pos, const BatchView &bv, const TensorView &out_k,
                           const TensorView &out_v, int *out_pos, cudaStream_t stream);

}  // namespace finch

// Host side of the C ABI: context, argument validation, workspace layout and kernel dispatch.
#include <limits.h>
#include <math.h>
#include <new>
#include <string.h>

#include <atomic>
#include <vector>

#include "finch_internal.cuh"

using namespace finch;

struct finch_ctx : public Ctx {};

namespace {

constexpr size_t kAlign = 256;
inline size_t align_up(size_t x) { return (x + kAlign - 1) / kAlign * kAlign; }

inline bool aligned16(const void *p) { return ((uintptr_t)p & 15u) == 0; }

finch_status check_tensor(const finch_ctx *ctx, const finch_tensor *t, bool allow_null_ptr) {
    if (!t) return FINCH_ERR_INVALID_ARG;
    if (!t->ptr) return allow_null_ptr ? FINCH_OK : FINCH_ERR_INVALID_ARG;
    const int64_t e = ctx->model.elem_bytes;
    if (!aligned16(t->ptr) || (t->stride_layer * e) % 16 || (t->stride_head * e) % 16 || (t->stride_tok * e) % 16)
        return FINCH_ERR_BAD_LAYOUT;
    if (t->stride_tok < ctx->model.d || t->stride_head < 0 || t->stride_layer < 0) return FINCH_ERR_INVALID_ARG;
    return FINCH_OK;
}

finch_status check_batch(const finch_ctx *ctx, const finch_batch *b) {
    if (!ctx || !b) return FINCH_ERR_INVALID_ARG;
    if (b->batch < 0 || b->batch > ctx->cfg.max_batch) return FINCH_ERR_INVALID_ARG;
    if (b->total_q < 0 || b->total_chunk < 0 || b->total_cache < 0) return FINCH_ERR_INVALID_ARG;
    if (b->max_q < 0 || b->max_cache < 0 || b->max_chunk < 0 || b->max_budget < 0) return FINCH_ERR_INVALID_ARG;
    if (b->max_q > ctx->cfg.max_prompt) return FINCH_ERR_INVALID_ARG;
    if ((int64_t)b->max_cache + b->max_chunk > ctx->cfg.max_candidates) return FINCH_ERR_INVALID_ARG;
    if (b->max_q > b->total_q || b->max_chunk > b->total_chunk || b->max_cache > b->total_cache ||
        b->max_budget > b->total_cache)
        return FINCH_ERR_INVALID_ARG;
    if (b->batch > 0 && (!b->q_off || !b->chunk_off || !b->cache_off || !b->cache_len || !b->budget))
        return FINCH_ERR_INVALID_ARG;
    return FINCH_OK;
}

struct WsLayout {
    size_t lse_off, lse_bytes;        // scoring scratch: row statistics per key split and group, partial scores
    size_t scores_off, scores_bytes;  // scores inside finch_step when the caller gives none
    size_t total;
};

WsLayout ws_layout(const finch_ctx *ctx, const finch_batch *b) {
    WsLayout w{};
    const ModelView &mv = ctx->model;
    w.lse_off = 0;
    const size_t n_kv_scores = (size_t)mv.L * mv.Hkv * ((size_t)b->total_cache + b->total_chunk);
    w.lse_bytes = (size_t)mv.L * mv.Hq * (size_t)b->total_q * sizeof(float2) * (kScoreMaxSplits * 4 + 1) +
                  (4 * n_kv_scores + 2) * sizeof(float) +  // row statistics, partial scores per KV head,
                  ((size_t)b->batch + 1) * 8 + 4096;       // and the item plan of a multi-request batch
    const size_t fused = score_fused_scratch(*ctx, view_of(b)) * sizeof(float2);  // the one-kernel path's layout
    w.lse_bytes = align_up(w.lse_bytes > fused ? w.lse_bytes : fused);
    w.scores_off = w.lse_off + w.lse_bytes;
    w.scores_bytes = align_up((size_t)mv.L * mv.G * ((size_t)b->total_cache + b->total_chunk) * sizeof(float));
    w.total = w.scores_off + w.scores_bytes;
    if (w.total == 0) w.total = kAlign;
    return w;
}

finch_status cuda_status(cudaError_t e) { return e == cudaSuccess ? FINCH_OK : FINCH_ERR_CUDA; }

// Do two [layers][heads][tokens][head_dim] views share a byte?  Their byte extents are compared; extents that
// intersect are still disjoint when both views have the same strides, whole rows as their head and layer strides,
// and base pointers that differ by a shift which keeps every row of one between the rows of the other (K and V
// interleaved in one buffer).  Anything else that intersects counts as an overlap.
bool views_overlap(const finch_ctx *ctx, const finch_tensor *a, int64_t a_tokens, const finch_tensor *b,
                   int64_t b_tokens) {
    if (!a || !b || !a->ptr || !b->ptr || a_tokens <= 0 || b_tokens <= 0) return false;
    const ModelView &mv = ctx->model;
    const int64_t e = mv.elem_bytes, row = (int64_t)mv.d * e;
    auto extent = [&](const finch_tensor *t, int64_t tokens) {
        return ((int64_t)(mv.L - 1) * t->stride_layer + (int64_t)(mv.Hkv - 1) * t->stride_head +
                (tokens - 1) * t->stride_tok) * e + row;
    };
    const uintptr_t a0 = (uintptr_t)a->ptr, b0 = (uintptr_t)b->ptr;
    const uintptr_t a1 = a0 + (uintptr_t)extent(a, a_tokens), b1 = b0 + (uintptr_t)extent(b, b_tokens);
    if (a1 <= b0 || b1 <= a0) return false;
    const int64_t pitch = a->stride_tok * e;
    if (a->stride_tok == b->stride_tok && a->stride_head == b->stride_head && a->stride_layer == b->stride_layer &&
        a->stride_head % a->stride_tok == 0 && a->stride_layer % a->stride_tok == 0 && pitch >= 2 * row) {
        const int64_t shift = (int64_t)((a0 > b0 ? a0 - b0 : b0 - a0) % (uintptr_t)pitch);
        if (shift >= row && shift <= pitch - row) return false;  // rows of one lie in the gaps of the other
    }
    return true;
}

finch_status validate_score(const finch_ctx *ctx, const finch_tensor *q, const finch_tensor *cache_k,
                            const finch_tensor *chunk_k, const finch_batch *batch) {
    finch_status s = check_batch(ctx, batch);
    if (s) return s;
    if ((s = check_tensor(ctx, q, batch->total_q == 0))) return s;
    if ((s = check_tensor(ctx, cache_k, batch->total_cache == 0))) return s;
    if ((s = check_tensor(ctx, chunk_k, batch->total_chunk == 0))) return s;
    if (batch->max_q == 0 && batch->batch > 0) return FINCH_ERR_INVALID_ARG;  // scoring needs prompt rows
    return FINCH_OK;
}

finch_status validate_compact(const finch_ctx *ctx, const int32_t *kept_idx, const int32_t *out_len,
                              const finch_tensor *cache_k, const finch_tensor *cache_v, const int32_t *cache_pos,
                              const finch_tensor *chunk_k, const finch_tensor *chunk_v, const int32_t *chunk_pos,
                              const finch_batch *batch, const finch_tensor *out_k, const finch_tensor *out_v,
                              const int32_t *out_pos) {
    finch_status s = check_batch(ctx, batch);
    if (s) return s;
    const bool no_cache = batch->total_cache == 0, no_chunk = batch->total_chunk == 0;
    if ((s = check_tensor(ctx, cache_k, no_cache))) return s;
    if ((s = check_tensor(ctx, cache_v, no_cache))) return s;
    if ((s = check_tensor(ctx, chunk_k, no_chunk))) return s;
    if ((s = check_tensor(ctx, chunk_v, no_chunk))) return s;
    if ((s = check_tensor(ctx, out_k, no_cache))) return s;
    if ((s = check_tensor(ctx, out_v, no_cache))) return s;
    if (!no_cache && (!out_pos || !kept_idx)) return FINCH_ERR_INVALID_ARG;
    if (!no_chunk && !chunk_pos) return FINCH_ERR_INVALID_ARG;
    if (batch->max_cache > 0 && !cache_pos) return FINCH_ERR_INVALID_ARG;
    if (batch->batch > 0 && !out_len) return FINCH_ERR_INVALID_ARG;
    // the gather runs in parallel: an output row that shares bytes with any input row, or with the other output,
    // would race
    const finch_tensor *outs[2] = {out_k, out_v};
    const finch_tensor *ins[4] = {cache_k, cache_v, chunk_k, chunk_v};
    const int64_t in_tokens[4] = {batch->total_cache, batch->total_cache, batch->total_chunk, batch->total_chunk};
    for (auto o : outs)
        for (int i = 0; i < 4; ++i)
            if (views_overlap(ctx, o, batch->total_cache, ins[i], in_tokens[i])) return FINCH_ERR_INVALID_ARG;
    if (views_overlap(ctx, out_k, batch->total_cache, out_v, batch->total_cache)) return FINCH_ERR_INVALID_ARG;
    return FINCH_OK;
}

}  // namespace

namespace finch {

// Tensor cores take every request when the context allows them (bf16, head_dim 64 or 128, either group mode);
// warp-level dot products take everything else, and also a batch whose tensors the TMA unit cannot describe.
cudaError_t run_score(const Ctx &ctx, const TensorView &q, const TensorView &cache_k, const TensorView &chunk_k,
                      const BatchView &bv, float *scores, float2 *scratch, size_t scratch_capacity, float *row_lse,
                      cudaStream_t stream) {
    if (score_tc_supported(ctx)) {
        cudaError_t e = launch_score_fused(ctx, q, cache_k, chunk_k, bv, scores, scratch, scratch_capacity, row_lse, stream);
        if (e != cudaErrorNotSupported) return e;
        e =
            launch_score_tc(ctx, q, cache_k, chunk_k, bv, scores, scratch, scratch_capacity, row_lse, stream);
        if (e != cudaErrorNotSupported) return e;
    }
    return launch_score_simt(ctx, q, cache_k, chunk_k, bv, scores, scratch, row_lse, stream);
}

}  // namespace finch

extern "C" {

const char *finch_status_string(finch_status s) {
    switch (s) {
        case FINCH_OK: return "ok";
        case FINCH_ERR_INVALID_ARG: return "invalid argument";
        case FINCH_ERR_UNSUPPORTED: return "unsupported device or shape";
        case FINCH_ERR_BAD_LAYOUT: return "pointer or stride not 16-byte aligned";
        case FINCH_ERR_WORKSPACE_TOO_SMALL: return "workspace too small";
        case FINCH_ERR_OOM: return "out of memory";
        case FINCH_ERR_CUDA: return "CUDA error";
        case FINCH_ERR_DEVICE_STATUS: return "device status word is non-zero";
    }
    return "unknown status";
}

finch_status finch_ctx_create(const finch_config *cfg, finch_ctx **out) {
    if (!cfg || !out) return FINCH_ERR_INVALID_ARG;
    if (cfg->n_layers <= 0 || cfg->n_q_heads <= 0 || cfg->n_kv_heads <= 0 || cfg->head_dim <= 0)
        return FINCH_ERR_INVALID_ARG;
    if (cfg->n_q_heads % cfg->n_kv_heads) return FINCH_ERR_INVALID_ARG;
    if (cfg->dtype != FINCH_F32 && cfg->dtype != FINCH_BF16) return FINCH_ERR_INVALID_ARG;
    if (cfg->group_mode != FINCH_GROUP_PER_KV_HEAD && cfg->group_mode != FINCH_GROUP_PER_LAYER)
        return FINCH_ERR_INVALID_ARG;
    if (cfg->max_batch <= 0 || cfg->max_prompt <= 0 || cfg->max_candidates <= 0) return FINCH_ERR_INVALID_ARG;
    if (!(cfg->scale >= 0.f) || isinf(cfg->scale)) return FINCH_ERR_INVALID_ARG;
    if (cfg->head_dim % 32 || cfg->head_dim > 256) return FINCH_ERR_UNSUPPORTED;
    if (!(cfg->rope_theta >= 0.f) || isinf(cfg->rope_theta) || (cfg->rope_theta > 0.f && cfg->rope_theta < 1.f))
        return FINCH_ERR_INVALID_ARG;
    if (cfg->rope_pairing != 0 && cfg->rope_pairing != 1) return FINCH_ERR_INVALID_ARG;
    if ((int64_t)cfg->n_layers * cfg->n_kv_heads > 65535 || cfg->max_batch > 65535) return FINCH_ERR_UNSUPPORTED;

    finch_ctx *ctx = new (std::nothrow) finch_ctx();
    if (!ctx) return FINCH_ERR_OOM;
    ctx->cfg = *cfg;
    ModelView &mv = ctx->model;
    mv.L = cfg->n_layers;
    mv.Hq = cfg->n_q_heads;
    mv.Hkv = cfg->n_kv_heads;
    mv.d = cfg->head_dim;
    mv.G = cfg->group_mode == FINCH_GROUP_PER_KV_HEAD ? cfg->n_kv_heads : 1;
    mv.hpg = mv.Hq / mv.G;
    mv.g = mv.Hq / mv.Hkv;
    mv.kvpg = mv.Hkv / mv.G;
    mv.scale = cfg->scale > 0.f ? cfg->scale : 1.0f / sqrtf((float)cfg->head_dim);
    mv.elem_bytes = cfg->dtype == FINCH_F32 ? 4 : 2;
    mv.rope_theta = cfg->rope_theta;
    mv.rope_pairing = cfg->rope_pairing;
    mv.rope_table = nullptr;
    mv.rope_rows = 0;
    ctx->d_status = nullptr;
    ctx->dry = cfg->device < 0;
    ctx->sm_count = 0;
    ctx->copy_stream = nullptr;
    ctx->ev_entry = ctx->ev_v_ready = ctx->ev_selected = nullptr;
    ctx->launches = 0;
    if (!ctx->dry) {
        int n_dev = 0;
        cudaDeviceProp prop;
        if (cudaGetDeviceCount(&n_dev) != cudaSuccess || cfg->device >= n_dev ||
            cudaGetDeviceProperties(&prop, cfg->device) != cudaSuccess || prop.major != 10) {
            (void)cudaGetLastError();
            delete ctx;
            return FINCH_ERR_UNSUPPORTED;
        }
        ctx->sm_count = prop.multiProcessorCount;
        // the context's device is made current only while its resources are created; the caller's comes back after
        int caller_device = -1;
        if (cudaGetDevice(&caller_device) != cudaSuccess) caller_device = -1;
        struct Restore {
            int dev;
            ~Restore() {
                if (dev >= 0) (void)cudaSetDevice(dev);
            }
        } restore{caller_device == cfg->device ? -1 : caller_device};
        if (cudaSetDevice(cfg->device) != cudaSuccess || cudaMalloc(&ctx->d_status, sizeof(int)) != cudaSuccess) {
            (void)cudaGetLastError();
            delete ctx;
            return FINCH_ERR_OOM;
        }
        if (cudaMemset(ctx->d_status, 0, sizeof(int)) != cudaSuccess ||
            cudaStreamCreateWithFlags(&ctx->copy_stream, cudaStreamNonBlocking) != cudaSuccess ||
            cudaEventCreateWithFlags(&ctx->ev_entry, cudaEventDisableTiming) != cudaSuccess ||
            cudaEventCreateWithFlags(&ctx->ev_v_ready, cudaEventDisableTiming) != cudaSuccess ||
            cudaEventCreateWithFlags(&ctx->ev_selected, cudaEventDisableTiming) != cudaSuccess) {
            (void)cudaGetLastError();
            finch_ctx_destroy(ctx);
            return FINCH_ERR_CUDA;
        }
        if (cfg->rope_theta > 0.f) {
            // a kept key moves by fewer positions than there are candidates: one table row per distance
            const int rows = cfg->max_candidates + 1, half = cfg->head_dim / 2;
            std::vector<float2> table((size_t)rows * half);
            for (int t = 0; t < half; ++t) {
                const double inv_freq = pow((double)cfg->rope_theta, -2.0 * t / cfg->head_dim);
                for (int n = 0; n < rows; ++n)
                    table[(size_t)n * half + t] = make_float2((float)cos(n * inv_freq), (float)sin(n * inv_freq));
            }
            float2 *dev = nullptr;
            if (cudaMalloc(&dev, table.size() * sizeof(float2)) != cudaSuccess ||
                cudaMemcpy(dev, table.data(), table.size() * sizeof(float2), cudaMemcpyHostToDevice) != cudaSuccess) {
                (void)cudaGetLastError();
                if (dev) cudaFree(dev);
                finch_ctx_destroy(ctx);
                return FINCH_ERR_OOM;
            }
            mv.rope_table = dev;
            mv.rope_rows = rows;
        }
    }
    *out = ctx;
    return FINCH_OK;
}

void finch_ctx_destroy(finch_ctx *ctx) {
    if (!ctx) return;
    if (ctx->ev_entry) cudaEventDestroy(ctx->ev_entry);
    if (ctx->ev_v_ready) cudaEventDestroy(ctx->ev_v_ready);
    if (ctx->ev_selected) cudaEventDestroy(ctx->ev_selected);
    if (ctx->copy_stream) cudaStreamDestroy(ctx->copy_stream);
    if (ctx->model.rope_table) cudaFree(const_cast<float2 *>(ctx->model.rope_table));
    if (ctx->d_status) cudaFree(ctx->d_status);
    delete ctx;
}

finch_status finch_workspace_bytes(const finch_ctx *ctx, const finch_batch *batch, size_t *out) {
    if (!out) return FINCH_ERR_INVALID_ARG;
    finch_status s = check_batch(ctx, batch);
    if (s) return s;
    *out = ws_layout(ctx, batch).total;
    return FINCH_OK;
}

finch_status finch_score(finch_ctx *ctx, const finch_tensor *prompt_q, const finch_tensor *cache_k,
                         const finch_tensor *chunk_k, const finch_batch *batch, float *scores, float *row_lse, void *ws,
                         size_t ws_bytes, void *cuda_stream) {
    finch_status s = validate_score(ctx, prompt_q, cache_k, chunk_k, batch);
    if (s) return s;
    const WsLayout w = ws_layout(ctx, batch);
    if (!scores && (size_t)batch->total_cache + batch->total_chunk > 0) return FINCH_ERR_INVALID_ARG;
    if (!ws) return FINCH_ERR_INVALID_ARG;
    if (!aligned16(ws)) return FINCH_ERR_BAD_LAYOUT;
    if (ws_bytes < w.lse_off + w.lse_bytes) return FINCH_ERR_WORKSPACE_TOO_SMALL;
    float2 *row_stats = (float2 *)((char *)ws + w.lse_off);
    if (ctx->dry) return FINCH_ERR_UNSUPPORTED;
    return cuda_status(run_score(*ctx, view_of(prompt_q), view_of(cache_k), view_of(chunk_k), view_of(batch), scores,
                                 row_stats, w.lse_bytes / sizeof(float2), row_lse, (cudaStream_t)cuda_stream));
}

finch_status finch_select(finch_ctx *ctx, const float *scores, const finch_batch *batch, int32_t *kept_idx,
                          int32_t *out_len, void *ws, size_t ws_bytes, void *cuda_stream) {
    (void)ws;
    (void)ws_bytes;
    finch_status s = check_batch(ctx, batch);
    if (s) return s;
    if (batch->batch > 0 && !out_len) return FINCH_ERR_INVALID_ARG;
    if ((size_t)batch->total_cache + batch->total_chunk > 0 && !scores) return FINCH_ERR_INVALID_ARG;
    if (batch->total_cache > 0 && !kept_idx) return FINCH_ERR_INVALID_ARG;
    if (ctx->dry) return FINCH_ERR_UNSUPPORTED;
    return cuda_status(launch_select(*ctx, scores, view_of(batch), kept_idx, out_len, (cudaStream_t)cuda_stream));
}

finch_status finch_compact(finch_ctx *ctx, const int32_t *kept_idx, const int32_t *out_len, const finch_tensor *cache_k,
                           const finch_tensor *cache_v, const int32_t *cache_pos, const finch_tensor *chunk_k,
                           const finch_tensor *chunk_v, const int32_t *chunk_pos, const finch_batch *batch,
                           const finch_tensor *out_k, const finch_tensor *out_v, int32_t *out_pos, void *cuda_stream) {
    finch_status s = validate_compact(ctx, kept_idx, out_len, cache_k, cache_v, cache_pos, chunk_k, chunk_v, chunk_pos,
                                      batch, out_k, out_v, out_pos);
    if (s) return s;
    if (ctx->dry) return FINCH_ERR_UNSUPPORTED;
    return cuda_status(launch_compact(*ctx, kept_idx, out_len, view_of(cache_k), view_of(cache_v), cache_pos,
                                      view_of(chunk_k), view_of(chunk_v), chunk_pos, view_of(batch), view_of(out_k),
                                      view_of(out_v), out_pos, (cudaStream_t)cuda_stream));
}

finch_status finch_step(finch_ctx *ctx, const finch_tensor *prompt_q, const finch_tensor *cache_k,
                        const finch_tensor *cache_v, const int32_t *cache_pos, const finch_tensor *chunk_k,
                        const finch_tensor *chunk_v, const int32_t *chunk_pos, const finch_batch *batch,
                        const finch_tensor *out_k, const finch_tensor *out_v, int32_t *out_pos, int32_t *kept_idx,
                        int32_t *out_len, float *scores, void *ws, size_t ws_bytes, void *cuda_stream) {
    finch_status s = validate_score(ctx, prompt_q, cache_k, chunk_k, batch);
    if (s) return s;
    if ((s = validate_compact(ctx, kept_idx, out_len, cache_k, cache_v, cache_pos, chunk_k, chunk_v, chunk_pos, batch,
                              out_k, out_v, out_pos)))
        return s;
    if (!ws) return FINCH_ERR_INVALID_ARG;
    if (!aligned16(ws)) return FINCH_ERR_BAD_LAYOUT;
    const WsLayout w = ws_layout(ctx, batch);
    if (ws_bytes < (scores ? w.lse_off + w.lse_bytes : w.total)) return FINCH_ERR_WORKSPACE_TOO_SMALL;
    float2 *row_stats = (float2 *)((char *)ws + w.lse_off);
    if (!scores) scores = (float *)((char *)ws + w.scores_off);
    if (ctx->dry) return FINCH_ERR_UNSUPPORTED;
    cudaStream_t stream = (cudaStream_t)cuda_stream;
    const BatchView bv = view_of(batch);
    cudaError_t e = run_score(*ctx, view_of(prompt_q), view_of(cache_k), view_of(chunk_k), bv, scores, row_stats,
                              w.lse_bytes / sizeof(float2), nullptr, stream);
    if (e == cudaSuccess) e = launch_select(*ctx, scores, bv, kept_idx, out_len, stream);
    if (e == cudaSuccess)
        e = launch_compact(*ctx, kept_idx, out_len, view_of(cache_k), view_of(cache_v), cache_pos, view_of(chunk_k),
                           view_of(chunk_v), chunk_pos, bv, view_of(out_k), view_of(out_v), out_pos, stream);
    return cuda_status(e);
}

// finch_step with this step's new inputs in HOST memory: copies prompt_q, chunk_k, chunk_v and chunk_pos into the
// caller's device staging tensors, runs the step, copies kept_idx and out_len back and waits for the stream.
finch_status finch_step_host(finch_ctx *ctx, const void *host_prompt_q, const void *host_chunk_k,
                             const void *host_chunk_v, const int32_t *host_chunk_pos, const finch_tensor *stage_q,
                             const finch_tensor *stage_chunk_k, const finch_tensor *stage_chunk_v,
                             int32_t *stage_chunk_pos, const finch_tensor *cache_k, const finch_tensor *cache_v,
                             const int32_t *cache_pos, const finch_batch *batch, const finch_tensor *out_k,
                             const finch_tensor *out_v, int32_t *out_pos, int32_t *kept_idx, int32_t *out_len,
                             int32_t *host_kept_idx, int32_t *host_out_len, void *ws, size_t ws_bytes,
                             void *cuda_stream) {
    finch_status s = check_batch(ctx, batch);
    if (s) return s;
    if (!stage_q || !stage_chunk_k || !stage_chunk_v) return FINCH_ERR_INVALID_ARG;
    const ModelView &mv = ctx->model;
    auto dense = [&](const finch_tensor *t, int heads, int64_t tokens) {
        return t->stride_tok == mv.d && t->stride_head == tokens * mv.d && t->stride_layer == (int64_t)heads * tokens * mv.d;
    };
    if (!dense(stage_q, mv.Hq, batch->total_q) || !dense(stage_chunk_k, mv.Hkv, batch->total_chunk) ||
        !dense(stage_chunk_v, mv.Hkv, batch->total_chunk))
        return FINCH_ERR_BAD_LAYOUT;  // the staging tensors receive dense host arrays
    if (batch->total_q > 0 && !host_prompt_q) return FINCH_ERR_INVALID_ARG;
    if (batch->total_chunk > 0 && (!host_chunk_k || !host_chunk_v || !host_chunk_pos || !stage_chunk_pos))
        return FINCH_ERR_INVALID_ARG;
    if (batch->batch > 0 && !host_out_len) return FINCH_ERR_INVALID_ARG;
    if (batch->total_cache > 0 && !host_kept_idx) return FINCH_ERR_INVALID_ARG;
    // validate the step itself before anything is enqueued (a validation-only context stops here)
    if ((s = validate_score(ctx, stage_q, cache_k, stage_chunk_k, batch))) return s;
    if ((s = validate_compact(ctx, kept_idx, out_len, cache_k, cache_v, cache_pos, stage_chunk_k, stage_chunk_v,
                              stage_chunk_pos, batch, out_k, out_v, out_pos)))
        return s;
    if (!ws) return FINCH_ERR_INVALID_ARG;
    if (!aligned16(ws)) return FINCH_ERR_BAD_LAYOUT;
    if (ws_bytes < ws_layout(ctx, batch).total) return FINCH_ERR_WORKSPACE_TOO_SMALL;
    if (ctx->dry) return FINCH_ERR_UNSUPPORTED;
    cudaStream_t stream = (cudaStream_t)cuda_stream, side = ctx->copy_stream;
    const size_t e = mv.elem_bytes;
    const size_t q_bytes = (size_t)mv.L * mv.Hq * batch->total_q * mv.d * e;
    const size_t c_bytes = (size_t)mv.L * mv.Hkv * batch->total_chunk * mv.d * e;
    const WsLayout w = ws_layout(ctx, batch);
    float2 *row_stats = (float2 *)((char *)ws + w.lse_off);
    float *scores = (float *)((char *)ws + w.scores_off);
    const BatchView bv = view_of(batch);
    // The scoring kernels read Q and the chunk's K; only the compaction reads the chunk's V.  V therefore travels
    // on the side stream, behind everything already enqueued on the caller's stream (an earlier step's compaction
    // may still be reading the staging tensor), and the compaction waits for it.  The kept indices go back to the
    // host on the side stream too, while the compaction runs.
    auto ok = [](cudaError_t ce) { return ce == cudaSuccess; };
    bool good = ok(cudaEventRecord(ctx->ev_entry, stream)) && ok(cudaStreamWaitEvent(side, ctx->ev_entry, 0));
    if (good && q_bytes) good = ok(cudaMemcpyAsync(stage_q->ptr, host_prompt_q, q_bytes, cudaMemcpyHostToDevice, stream));
    if (good && c_bytes)
        good = ok(cudaMemcpyAsync(stage_chunk_k->ptr, host_chunk_k, c_bytes, cudaMemcpyHostToDevice, stream));
    if (good && batch->total_chunk)
        good = ok(cudaMemcpyAsync(stage_chunk_pos, host_chunk_pos, (size_t)batch->total_chunk * 4,
                                  cudaMemcpyHostToDevice, stream));
    if (good && c_bytes)
        good = ok(cudaMemcpyAsync(stage_chunk_v->ptr, host_chunk_v, c_bytes, cudaMemcpyHostToDevice, side));
    good = good && ok(cudaEventRecord(ctx->ev_v_ready, side));
    if (good)
        good = ok(run_score(*ctx, view_of(stage_q), view_of(cache_k), view_of(stage_chunk_k), bv, scores, row_stats,
                            w.lse_bytes / sizeof(float2), nullptr, stream));
    if (good) good = ok(launch_select(*ctx, scores, bv, kept_idx, out_len, stream));
    good = good && ok(cudaEventRecord(ctx->ev_selected, stream)) && ok(cudaStreamWaitEvent(side, ctx->ev_selected, 0));
    const size_t kept_bytes = (size_t)mv.L * mv.G * batch->total_cache * 4;
    if (good && kept_bytes) good = ok(cudaMemcpyAsync(host_kept_idx, kept_idx, kept_bytes, cudaMemcpyDeviceToHost, side));
    if (good && batch->batch)
        good = ok(cudaMemcpyAsync(host_out_len, out_len, (size_t)batch->batch * 4, cudaMemcpyDeviceToHost, side));
    good = good && ok(cudaStreamWaitEvent(stream, ctx->ev_v_ready, 0));
    if (good)
        good = ok(launch_compact(*ctx, kept_idx, out_len, view_of(cache_k), view_of(cache_v), cache_pos,
                                 view_of(stage_chunk_k), view_of(stage_chunk_v), stage_chunk_pos, bv, view_of(out_k),
                                 view_of(out_v), out_pos, stream));
    // both streams are drained before returning, also after a failure, so that nothing of this call is still in
    // flight when the caller reuses its buffers
    const bool drained = ok(cudaStreamSynchronize(side)) & ok(cudaStreamSynchronize(stream));
    if (!good || !drained) {
        (void)cudaGetLastError();
        return FINCH_ERR_CUDA;
    }
    return FINCH_OK;
}

finch_status finch_launch_count(const finch_ctx *ctx, uint64_t *out) {
    if (!ctx || !out) return FINCH_ERR_INVALID_ARG;
    *out = ctx->launches;
    return FINCH_OK;
}

finch_status finch_device_status(finch_ctx *ctx, void *cuda_stream, int32_t *out) {
    if (!ctx || !out) return FINCH_ERR_INVALID_ARG;
    if (ctx->dry) return FINCH_ERR_UNSUPPORTED;
    cudaStream_t stream = (cudaStream_t)cuda_stream;
    int host = 0;
    if (cudaMemcpyAsync(&host, ctx->d_status, sizeof(int), cudaMemcpyDeviceToHost, stream) != cudaSuccess ||
        cudaMemsetAsync(ctx->d_status, 0, sizeof(int), stream) != cudaSuccess ||
        cudaStreamSynchronize(stream) != cudaSuccess) {
        (void)cudaGetLastError();
        return FINCH_ERR_CUDA;
    }
    *out = host;
    return host ? FINCH_ERR_DEVICE_STATUS : FINCH_OK;
}

}  // extern "C"

// ---------------------------------------------------------------------------------------------------------------
// finch_score_static: scoring for callers that cannot allocate device memory.
//
// finch_score keeps its intermediate results -- per-row softmax statistics, per-group partial column sums, a few
// counters -- in a workspace the caller allocates.  Code that runs where cudaMalloc is off limits -- a plugin inside a serving process that owns
// all device memory and hands none out, a callback that may not block on the allocator, a latency-critical loop
// that must not touch the driver's heap -- has no such workspace to give.  For those callers the scratch is the
// fixed array below, which is part of the library image: every GPU that loads libfinch holds it until the process
// exits.
namespace {

constexpr size_t kStaticRows = size_t(1) << 20;  // prompt rows (layers x query heads x packed prompt tokens): 8 MiB
static __device__ __align__(256) float2 g_static_row_stats[kStaticRows];

constexpr int kMaxDevices = 64;
// device address of the array on each device, filled on first use; contexts on different host threads share it
std::atomic<float2 *> g_static_ptr[kMaxDevices];

// In host code the array's name is only a handle; its device address has to be asked for, once per device, with
// that device current.  The current device is checked on every call: the address belongs to one GPU, and kernels
// launched with another device current would dereference it there.
finch_status static_scratch(int device, float2 **out) {
    if (device < 0 || device >= kMaxDevices) return FINCH_ERR_UNSUPPORTED;
    int current = -1;
    if (cudaGetDevice(&current) != cudaSuccess || current != device) {
        (void)cudaGetLastError();
        return FINCH_ERR_INVALID_ARG;  // the context's device must be the current one
    }
    float2 *p = g_static_ptr[device].load(std::memory_order_acquire);
    if (!p) {
        if (cudaGetSymbolAddress((void **)&p, g_static_row_stats) != cudaSuccess || !p) {
            (void)cudaGetLastError();
            return FINCH_ERR_CUDA;
        }
        g_static_ptr[device].store(p, std::memory_order_release);  // every thread resolves the same address
    }
    *out = p;
    return FINCH_OK;
}

}  // namespace

extern "C" finch_status finch_score_static(finch_ctx *ctx, const finch_tensor *prompt_q, const finch_tensor *cache_k,
                                           const finch_tensor *chunk_k, const finch_batch *batch, float *scores,
                                           float *row_lse, void *cuda_stream) {
    finch_status s = validate_score(ctx, prompt_q, cache_k, chunk_k, batch);
    if (s) return s;
    if (!scores && (size_t)batch->total_cache + batch->total_chunk > 0) return FINCH_ERR_INVALID_ARG;
    const size_t rows = (size_t)ctx->model.L * ctx->model.Hq * (size_t)batch->total_q;
    if (rows > kStaticRows) return FINCH_ERR_WORKSPACE_TOO_SMALL;  // beyond the built-in scratch: use finch_score
    if (ctx->dry) return FINCH_ERR_UNSUPPORTED;
    float2 *row_stats = nullptr;
    if ((s = static_scratch(ctx->cfg.device, &row_stats))) return s;
    return cuda_status(run_score(*ctx, view_of(prompt_q), view_of(cache_k), view_of(chunk_k), view_of(batch), scores,
                                 row_stats, kStaticRows, row_lse, (cudaStream_t)cuda_stream));
}

extern "C" size_t finch_score_static_max_rows(void) { return kStaticRows; }

// Which kernels finch_score_static runs for a batch: the tensor-core kernels keep more than one entry per prompt row
// in the scratch (statistics per key range and softmax group, partial column sums per candidate), so a batch can
// fit the array's row limit and still be too large for them; it then takes the warp-level kernels.
// Which kernels finch_score / finch_step run for a batch (workspace of finch_workspace_bytes): see the header.
extern "C" finch_status finch_score_plan(const finch_ctx *ctx, const finch_batch *batch, int32_t *path, int32_t *window) {
    if (!path) return FINCH_ERR_INVALID_ARG;
    finch_status s = check_batch(ctx, batch);
    if (s) return s;
    const BatchView bv = view_of(batch);
    const int w = score_fused_window(*ctx, bv);
    *path = w > 0 ? FINCH_SCORE_ONE_KERNEL : (score_tc_supported(*ctx) ? FINCH_SCORE_TWO_LAUNCH : FINCH_SCORE_WARP_LEVEL);
    if (window) *window = w;
    return FINCH_OK;
}

extern "C" finch_status finch_score_static_path(const finch_ctx *ctx, const finch_batch *batch, int32_t *tensor_cores) {
    if (!tensor_cores) return FINCH_ERR_INVALID_ARG;
    finch_status s = check_batch(ctx, batch);
    if (s) return s;
    const BatchView bv = view_of(batch);
    const size_t fused = score_fused_scratch(*ctx, bv);
    *tensor_cores = score_tc_supported(*ctx) &&
                    ((fused > 0 && fused <= kStaticRows) || score_tc_scratch_min(*ctx, bv) <= kStaticRows);
    return FINCH_OK;
}

// Prompt-guided scoring with plain FMA dot products (fp32 inputs, head dimensions the tensor-core path does not take).
//
//   lse_simt     one CTA per (64 prompt rows of one query head, unit): sweeps every candidate key and keeps an
//                online (max, sum-exp) per row -> row_stats = (max of the base-2 logits, 1 / sum), row_lse
//   colsum_simt  one CTA per (64 candidate keys, unit): sweeps every prompt row of every head of the group and
//                accumulates exp2(s2 - max) / sum per key -> scores
//
// Keeping the row maximum and the reciprocal sum apart (instead of one log-sum-exp) keeps the exponent's argument
// a small difference even when the logits are large; both kernels form it with the same fused multiply-add
// (dot * scale2 - max), so the weight of a row's largest key is the same in the sum and in the column pass.
//
// A unit is one (layer, selection group, request).  Both kernels tile the logits 64 x 64 with a 4 x 4 register
// micro-tile per thread and walk head_dim in slices of 32 staged through shared memory.  All sums have a fixed
// order, so the scores are bit-identical from run to run.
#include "finch_internal.cuh"

namespace finch {
namespace {

constexpr int kTile = 64;      // rows and keys per CTA tile
constexpr int kSlice = 32;     // head_dim slice staged per iteration
constexpr int kThreads = 256;  // 16 x 16 threads, 4 x 4 logits each

template <typename T>
__device__ __forceinline__ float to_f32(T v);
template <>
__device__ __forceinline__ float to_f32<float>(float v) { return v; }
template <>
__device__ __forceinline__ float to_f32<__nv_bfloat16>(__nv_bfloat16 v) { return __bfloat162float(v); }

// Stage a [64 rows][32 elements] slice of Q (prompt rows p0.. of head h) into shared memory as fp32.
template <typename T>
__device__ __forceinline__ void stage_q(float (*dst)[kSlice + 1], const TensorView &q, const UnitInfo &u, int h, int p0,
                                        int t0) {
    const T *base = (const T *)q.ptr + (int64_t)u.l * q.stride_layer + (int64_t)h * q.stride_head;
    for (int e = threadIdx.x; e < kTile * kSlice; e += kThreads) {
        const int r = e / kSlice, t = e % kSlice;
        const int p = p0 + r;
        dst[r][t] = p < u.n_q ? to_f32<T>(base[(int64_t)(u.q0 + p) * q.stride_tok + t0 + t]) : 0.f;
    }
}

// Stage a [64 keys][32 elements] slice of the candidate keys j0.. of KV head kvh (cache rows first, then chunk rows).
template <typename T>
__device__ __forceinline__ void stage_k(float (*dst)[kSlice + 1], const TensorView &cache_k, const TensorView &chunk_k,
                                        const UnitInfo &u, int kvh, int j0, int t0) {
    const T *cbase = (const T *)cache_k.ptr + (int64_t)u.l * cache_k.stride_layer + (int64_t)kvh * cache_k.stride_head;
    const T *hbase = (const T *)chunk_k.ptr + (int64_t)u.l * chunk_k.stride_layer + (int64_t)kvh * chunk_k.stride_head;
    for (int e = threadIdx.x; e < kTile * kSlice; e += kThreads) {
        const int r = e / kSlice, t = e % kSlice;
        const int j = j0 + r;
        float v = 0.f;
        if (j < u.c)
            v = to_f32<T>(cbase[(int64_t)(u.cache0 + j) * cache_k.stride_tok + t0 + t]);
        else if (j < u.N)
            v = to_f32<T>(hbase[(int64_t)(u.chunk0 + j - u.c) * chunk_k.stride_tok + t0 + t]);
        dst[r][t] = v;
    }
}

// acc[i][j] += sum_t Q[ty + 16 i][t] * K[tx + 16 j][t] over one staged slice.
__device__ __forceinline__ void fma_slice(float (&acc)[4][4], const float (*qs)[kSlice + 1],
                                          const float (*ks)[kSlice + 1], int tx, int ty) {
#pragma unroll 8
    for (int t = 0; t < kSlice; ++t) {
        float a[4], b[4];
#pragma unroll
        for (int i = 0; i < 4; ++i) a[i] = qs[ty + 16 * i][t];
#pragma unroll
        for (int j = 0; j < 4; ++j) b[j] = ks[tx + 16 * j][t];
#pragma unroll
        for (int i = 0; i < 4; ++i)
#pragma unroll
            for (int j = 0; j < 4; ++j) acc[i][j] = fmaf(a[i], b[j], acc[i][j]);
    }
}

template <typename T>
__global__ void __launch_bounds__(kThreads)
lse_simt(ModelView mv, BatchView bv, TensorView q, TensorView cache_k, TensorView chunk_k, float2 *row_stats,
         float *row_lse, int *status) {
    __shared__ float qs[kTile][kSlice + 1];
    __shared__ float ks[kTile][kSlice + 1];
    const UnitInfo u = unit_info(mv, bv, blockIdx.y, blockIdx.z);
    if (!u.ok) {
        if (threadIdx.x == 0) atomicOr(status, FINCH_DEV_BAD_BATCH);
        return;
    }
    if (u.N == 0) return;
    const int row_blocks = (bv.max_q + kTile - 1) / kTile;
    const int hh = blockIdx.x / row_blocks, p0 = (blockIdx.x % row_blocks) * kTile;
    if (p0 >= u.n_q) return;
    const int h = u.G * mv.hpg + hh, kvh = h / mv.g;
    const int tx = threadIdx.x % 16, ty = threadIdx.x / 16;
    const float scale2 = mv.scale * kLog2e;

    float run_max[4], run_sum[4];  // base-2 logits, over this thread's own key columns
    int vis[4];                    // candidates the thread's rows attend to: all, or the row's limit (causal rows)
#pragma unroll
    for (int i = 0; i < 4; ++i) {
        run_max[i] = -INFINITY;
        run_sum[i] = 0.f;
        const int p = p0 + ty + 16 * i;
        vis[i] = u.N;
        if (bv.row_limit && p < u.n_q) vis[i] = max(0, min(u.N, bv.row_limit[u.q0 + p]));
    }
    for (int j0 = 0; j0 < u.N; j0 += kTile) {
        float acc[4][4] = {};
        for (int t0 = 0; t0 < mv.d; t0 += kSlice) {
            __syncthreads();
            stage_q<T>(qs, q, u, h, p0, t0);
            stage_k<T>(ks, cache_k, chunk_k, u, kvh, j0, t0);
            __syncthreads();
            fma_slice(acc, qs, ks, tx, ty);
        }
#pragma unroll
        for (int i = 0; i < 4; ++i) {
            float tile_max = -INFINITY;
#pragma unroll
            for (int j = 0; j < 4; ++j)
                if (j0 + tx + 16 * j < vis[i]) tile_max = fmaxf(tile_max, acc[i][j] * scale2);
            if (tile_max == -INFINITY) continue;
            const float new_max = fmaxf(run_max[i], tile_max);
            float sum = run_sum[i] * exp2f(run_max[i] - new_max);  // exp2(-inf) = 0 on the first tile
#pragma unroll
            for (int j = 0; j < 4; ++j)
                if (j0 + tx + 16 * j < vis[i]) sum += exp2f(fmaf(acc[i][j], scale2, -new_max));
            run_max[i] = new_max;
            run_sum[i] = sum;
        }
    }
    // merge the 16 column owners of each row (the lanes tx = 0..15 of a half warp) with a butterfly
#pragma unroll
    for (int i = 0; i < 4; ++i) {
        float mx = run_max[i], sm = run_sum[i];
#pragma unroll
        for (int off = 1; off < 16; off <<= 1) {
            const float omx = __shfl_xor_sync(0xffffffffu, mx, off);
            const float osm = __shfl_xor_sync(0xffffffffu, sm, off);
            const float nmx = fmaxf(mx, omx);
            const float a = mx == -INFINITY ? 0.f : sm * exp2f(mx - nmx);
            const float b = omx == -INFINITY ? 0.f : osm * exp2f(omx - nmx);
            sm = a + b;  // commutative: both partners get the same bits
            mx = nmx;
        }
        const int p = p0 + ty + 16 * i;
        if (tx == 0 && p < u.n_q) {
            const int64_t row = ((int64_t)u.l * mv.Hq + h) * bv.total_q + u.q0 + p;
            if (bv.self_lse) {  // the keys the row attends to besides the candidates: one more term of the sum
                const float ex = bv.self_lse[row] * kLog2e;
                if (ex > -INFINITY) {
                    const float nmx = fmaxf(mx, ex);
                    sm = sm * exp2f(mx - nmx) + exp2f(ex - nmx);
                    mx = nmx;
                }
            }
            // (max, weight per unit of exp2): 1 / sum, times the fraction of the candidates the row sees when the
            // per-row normalisation is on; a row that sees nothing weighs nothing
            float w = sm > 0.f ? 1.0f / sm : 0.f;
            if (bv.row_norm) w *= (float)vis[i] / (float)u.N;
            row_stats[row] = make_float2(sm > 0.f ? mx : 0.f, w);
            if (row_lse) row_lse[row] = sm > 0.f ? (mx + log2f(sm)) * kLn2 : -INFINITY;
        }
    }
}

template <typename T>
__global__ void __launch_bounds__(kThreads)
colsum_simt(ModelView mv, BatchView bv, TensorView q, TensorView cache_k, TensorView chunk_k,
            const float2 *row_stats, float *scores, int *status) {
    __shared__ float qs[kTile][kSlice + 1];
    __shared__ float ks[kTile][kSlice + 1];
    __shared__ float red[16][kTile];
    const UnitInfo u = unit_info(mv, bv, blockIdx.y, blockIdx.z);
    if (!u.ok) {
        if (threadIdx.x == 0) atomicOr(status, FINCH_DEV_BAD_BATCH);
        return;
    }
    const int j0 = blockIdx.x * kTile;
    if (j0 >= u.N) return;
    const int tx = threadIdx.x % 16, ty = threadIdx.x / 16;
    const float scale2 = mv.scale * kLog2e;

    float col[4] = {0.f, 0.f, 0.f, 0.f};
    for (int hh = 0; hh < mv.hpg; ++hh) {
        const int h = u.G * mv.hpg + hh, kvh = h / mv.g;
        const float2 *stats = row_stats + ((int64_t)u.l * mv.Hq + h) * bv.total_q + u.q0;
        for (int p0 = 0; p0 < u.n_q; p0 += kTile) {
            float acc[4][4] = {};
            for (int t0 = 0; t0 < mv.d; t0 += kSlice) {
                __syncthreads();
                stage_q<T>(qs, q, u, h, p0, t0);
                stage_k<T>(ks, cache_k, chunk_k, u, kvh, j0, t0);
                __syncthreads();
                fma_slice(acc, qs, ks, tx, ty);
            }
#pragma unroll
            for (int i = 0; i < 4; ++i) {
                const int p = p0 + ty + 16 * i;
                if (p >= u.n_q) continue;
                const float2 st = stats[p];
                const int lim = bv.row_limit ? bv.row_limit[u.q0 + p] : u.N;  // keys at or beyond it are masked
#pragma unroll
                for (int j = 0; j < 4; ++j)
                    if (j0 + tx + 16 * j < lim) col[j] = fmaf(exp2f(fmaf(acc[i][j], scale2, -st.x)), st.y, col[j]);
            }
        }
    }
    __syncthreads();
#pragma unroll
    for (int j = 0; j < 4; ++j) red[ty][tx + 16 * j] = col[j];
    __syncthreads();
    if (threadIdx.x < kTile && j0 + threadIdx.x < u.N) {
        float s = 0.f;
#pragma unroll
        for (int r = 0; r < 16; ++r) s += red[r][threadIdx.x];
        scores[((int64_t)u.l * mv.G + u.G) * ((int64_t)bv.total_cache + bv.total_chunk) + u.cache0 + u.chunk0 + j0 +
               threadIdx.x] = s;
    }
}

template <typename T>
cudaError_t launch_t(const Ctx &ctx, const TensorView &q, const TensorView &cache_k, const TensorView &chunk_k,
                     const BatchView &bv, float *scores, float2 *row_stats, float *row_lse,
                     cudaStream_t stream) {
    const ModelView &mv = ctx.model;
    const int units = mv.L * mv.G;
    const int row_blocks = (bv.max_q + kTile - 1) / kTile;
    const int key_tiles = (bv.max_cache + bv.max_chunk + kTile - 1) / kTile;
    if (units == 0 || bv.batch == 0 || row_blocks == 0 || key_tiles == 0) return cudaSuccess;
    dim3 g1(row_blocks * mv.hpg, units, bv.batch);
    lse_simt<T><<<g1, kThreads, 0, stream>>>(mv, bv, q, cache_k, chunk_k, row_stats, row_lse, ctx.d_status);
    dim3 g2(key_tiles, units, bv.batch);
    colsum_simt<T><<<g2, kThreads, 0, stream>>>(mv, bv, q, cache_k, chunk_k, row_stats, scores, ctx.d_status);
    ctx.launches += 2;
    return cudaGetLastError();
}

}  // namespace

cudaError_t launch_score_simt(const Ctx &ctx, const TensorView &q, const TensorView &cache_k, const TensorView &chunk_k,
                              const BatchView &bv, float *scores, float2 *row_stats, float *row_lse,
                              cudaStream_t stream) {
    if (ctx.cfg.dtype == FINCH_F32)
        return launch_t<float>(ctx, q, cache_k, chunk_k, bv, scores, row_stats, row_lse, stream);
    return launch_t<__nv_bfloat16>(ctx, q, cache_k, chunk_k, bv, scores, row_stats, row_lse, stream);
}

}  // namespace finch

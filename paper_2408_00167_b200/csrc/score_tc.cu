// Prompt-guided scoring on the 5th-generation tensor cores (bf16 inputs, prompts of at least 64 rows).
//
// One kernel template, two sweeps over the logits S = Q K^T of a unit (layer, KV head, request):
//
//   kLse     CTA = 128 prompt rows of one query head (the stationary A operand); streams every 128-key tile of the
//            unit as B.  D[row][key] lands in tensor memory with one prompt row per lane, so each thread keeps the
//            online (max, sum exp2) of its own row without any cross-lane traffic  ->  row_stats, row_lse.
//   kColsum  CTA = one 128-key tile (stationary A); streams every 128-row block of every query head of the group
//            as B.  D[key][row]: one key per lane, so the sum over prompt rows of exp2(s - max) / sum is a private
//            running sum per thread  ->  scores.
//
// Warp roles (192 threads): warp 0 lane 0 issues TMA loads (128-byte swizzle) into a 4-stage shared-memory ring,
// warp 1 owns tensor memory and its lane 0 issues tcgen05.mma (128 x 128 x 16, fp32 accumulate) into one of four
// 128-column accumulators, warps 2-5 read accumulators back with tcgen05.ld and do the softmax arithmetic.
// mbarriers connect the three; every wait is bounded and raises FINCH_DEV_TIMEOUT instead of hanging.
// Candidate tiles never straddle the cache/chunk boundary: the cache's rows are tiled first, then the chunk's.
#include <limits.h>

#include "finch_internal.cuh"
#include "sm100_ptx.cuh"

namespace finch {
namespace {

using namespace ptx;

constexpr int kRows = 128;        // rows per operand tile = MMA M = MMA N
constexpr int kStages = 4;        // shared-memory stages of the streamed operand
constexpr int kAccBufs = 4;       // accumulators of 128 fp32 columns in tensor memory (4 x 128 = all 512 columns)
constexpr int kTcThreads = 192;
constexpr int kSlabBytes = kRows * 128;  // one 64-element (128-byte) wide slab of a 128-row tile
constexpr int kAuxBytes = 1024 + 4 * 2 * kRows * 8;  // barriers, then per-warp double-buffered row statistics

enum { kLse = 0, kColsum = 1 };

struct TcParams {
    ModelView mv;
    BatchView bv;
    float2 *row_stats;
    float *row_lse;
    float *scores;
    int *status;
    int min_q;  // requests with fewer prompt rows are left to the warp-level path
};

struct KeyTile {
    int is_chunk;  // which tensor the rows come from
    int row0;      // first token row inside that packed tensor
    int j0;        // candidate index of the tile's first row
    int valid;     // rows of the tile that are candidates (1..128)
};

__device__ __forceinline__ int n_key_tiles(const UnitInfo &u) { return (u.c + kRows - 1) / kRows + (u.m + kRows - 1) / kRows; }

__device__ __forceinline__ KeyTile key_tile(const UnitInfo &u, int t) {
    const int tc = (u.c + kRows - 1) / kRows;
    KeyTile k;
    if (t < tc) {
        k.is_chunk = 0;
        k.row0 = u.cache0 + t * kRows;
        k.j0 = t * kRows;
        k.valid = min(kRows, u.c - t * kRows);
    } else {
        const int tt = t - tc;
        k.is_chunk = 1;
        k.row0 = u.chunk0 + tt * kRows;
        k.j0 = u.c + tt * kRows;
        k.valid = min(kRows, u.m - tt * kRows);
    }
    return k;
}

template <int MODE, int D>
__global__ void __launch_bounds__(kTcThreads, 1)
score_tc_kernel(const __grid_constant__ CUtensorMap q_map, const __grid_constant__ CUtensorMap cache_map,
                const __grid_constant__ CUtensorMap chunk_map, TcParams p) {
    constexpr int kSlabs = D / 64;
    constexpr int kTileBytes = kSlabs * kSlabBytes;
    extern __shared__ uint8_t smem_raw[];
    uint8_t *smem = (uint8_t *)(((uintptr_t)smem_raw + 1023) & ~(uintptr_t)1023);
    uint8_t *stat_tile = smem;
    uint8_t *stage_tiles = smem + kTileBytes;
    uint8_t *aux = stage_tiles + kStages * kTileBytes;
    uint64_t *stat_full = (uint64_t *)aux;
    uint64_t *full = stat_full + 1;
    uint64_t *empty = full + kStages;
    uint64_t *acc_full = empty + kStages;
    uint64_t *acc_empty = acc_full + kAccBufs;
    uint32_t *tmem_slot = (uint32_t *)(acc_empty + kAccBufs);
    volatile int *abort_flag = (volatile int *)(tmem_slot + 1);
    float2 *stats_sm = (float2 *)(aux + 1024);  // [4 warps][2][128] (-max, 1/sum), kColsum only

    const ModelView &mv = p.mv;
    const BatchView &bv = p.bv;
    const UnitInfo u = unit_info(mv, bv, blockIdx.y, blockIdx.z);
    if (!u.ok) {
        if (threadIdx.x == 0) atomicOr(p.status, FINCH_DEV_BAD_BATCH);
        return;
    }
    if (u.n_q < p.min_q || u.N == 0) return;
    const int kvh = u.G;  // one KV head per selection group on this path
    const int q_blocks = (u.n_q + kRows - 1) / kRows;
    const int k_tiles = n_key_tiles(u);

    // ---- what this CTA holds still, and what it streams
    int n_iter, hh_lse = 0, p0_lse = 0;
    KeyTile my_tile{};
    if (MODE == kLse) {
        const int row_blocks = (bv.max_q + kRows - 1) / kRows;
        hh_lse = blockIdx.x / row_blocks;
        p0_lse = (blockIdx.x % row_blocks) * kRows;
        if (p0_lse >= u.n_q) return;
        n_iter = k_tiles;
    } else {
        if ((int)blockIdx.x >= k_tiles) return;
        my_tile = key_tile(u, blockIdx.x);
        n_iter = mv.hpg * q_blocks;
    }

    const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
    if (threadIdx.x == 0) {
        mbar_init(stat_full, 1);
        for (int s = 0; s < kStages; ++s) {
            mbar_init(&full[s], 1);
            mbar_init(&empty[s], 1);
        }
        for (int b = 0; b < kAccBufs; ++b) {
            mbar_init(&acc_full[b], 1);
            mbar_init(&acc_empty[b], 4);  // one arrival per softmax warp
        }
        *abort_flag = 0;
        fence_barrier_init();
    }
    if (warp == 1) {
        tmem_alloc(tmem_slot, 512);
        tmem_relinquish();
    }
    tc_fence_before();
    __syncthreads();
    tc_fence_after();
    const uint32_t tmem_base = *tmem_slot;

    if (warp == 0) {
        // =================================================================== TMA producer
        if (lane == 0) {
            prefetch_tensormap(&q_map);
            prefetch_tensormap(&cache_map);
            prefetch_tensormap(&chunk_map);
            mbar_expect_tx(stat_full, kTileBytes);
            if (MODE == kLse) {
                const int h = u.G * mv.hpg + hh_lse;
                for (int s = 0; s < kSlabs; ++s)
                    tma_load_4d(stat_tile + s * kSlabBytes, &q_map, stat_full, s * 64, u.q0 + p0_lse, h, u.l);
            } else {
                const CUtensorMap *m = my_tile.is_chunk ? &chunk_map : &cache_map;
                for (int s = 0; s < kSlabs; ++s)
                    tma_load_4d(stat_tile + s * kSlabBytes, m, stat_full, s * 64, my_tile.row0, kvh, u.l);
            }
            int issued = 0;
            for (int i = 0; i < n_iter; ++i) {
                const int stage = i % kStages, ph = (i / kStages) & 1;
                if (!mbar_wait(&empty[stage], ph ^ 1, abort_flag)) break;
                mbar_expect_tx(&full[stage], kTileBytes);
                uint8_t *dst = stage_tiles + stage * kTileBytes;
                if (MODE == kLse) {
                    const KeyTile kt = key_tile(u, i);
                    const CUtensorMap *m = kt.is_chunk ? &chunk_map : &cache_map;
                    for (int s = 0; s < kSlabs; ++s)
                        tma_load_4d(dst + s * kSlabBytes, m, &full[stage], s * 64, kt.row0, kvh, u.l);
                } else {
                    const int h = u.G * mv.hpg + i / q_blocks, p0 = (i % q_blocks) * kRows;
                    for (int s = 0; s < kSlabs; ++s)
                        tma_load_4d(dst + s * kSlabBytes, &q_map, &full[stage], s * 64, u.q0 + p0, h, u.l);
                }
                ++issued;
            }
            // no copy may still be in flight when the CTA retires: wait (bounded) for the last ring of loads
            mbar_wait(stat_full, 0, abort_flag);
            for (int i = max(0, issued - kStages); i < issued; ++i)
                mbar_wait(&full[i % kStages], (i / kStages) & 1, abort_flag);
        }
    } else if (warp == 1) {
        // =================================================================== MMA issuer
        if (lane == 0) {
            constexpr uint32_t idesc = idesc_bf16_f32(kRows, kRows);
            const uint32_t a_addr = smem_u32(stat_tile);
            if (mbar_wait(stat_full, 0, abort_flag)) {
                for (int i = 0; i < n_iter; ++i) {
                    const int stage = i % kStages, ph = (i / kStages) & 1;
                    const int buf = i % kAccBufs, bph = (i / kAccBufs) & 1;
                    if (!mbar_wait(&full[stage], ph, abort_flag)) break;
                    if (!mbar_wait(&acc_empty[buf], bph ^ 1, abort_flag)) break;
                    tc_fence_after();
                    const uint32_t b_addr = smem_u32(stage_tiles + stage * kTileBytes);
#pragma unroll
                    for (int k = 0; k < D / 16; ++k) {
                        const uint32_t off = (k / 4) * kSlabBytes + (k % 4) * 32;
                        umma_bf16(tmem_base + buf * kRows, smem_desc_sw128(a_addr + off), smem_desc_sw128(b_addr + off),
                                  idesc, k > 0);
                    }
                    umma_commit(&empty[stage]);   // the stage may be refilled once these MMAs have read it
                    umma_commit(&acc_full[buf]);  // and the accumulator is ready for the softmax warps
                }
            }
        }
    } else {
        // =================================================================== softmax warps (one TMEM lane per thread)
        const int quarter = warp & 3;                       // tcgen05.ld reaches lanes 32*(warp % 4) ..
        const int my_row = quarter * 32 + lane;             // row of the stationary tile this thread owns
        const uint32_t t_lane = tmem_base + ((uint32_t)(quarter * 32) << 16);
        const float scale2 = mv.scale * kLog2e;
        float v[32];
        if (MODE == kLse) {
            float m_raw = -INFINITY, z = 0.f;
            bool done = true;
            for (int i = 0; i < n_iter; ++i) {
                const int buf = i % kAccBufs, bph = (i / kAccBufs) & 1;
                const KeyTile kt = key_tile(u, i);
                // the verdict of a wait is made warp-uniform so that a timeout takes the whole warp out of the loop
                if (!__all_sync(0xffffffffu, mbar_wait(&acc_full[buf], bph, abort_flag))) { done = false; break; }
                tc_fence_after();
                for (int cc = 0; cc * 32 < kt.valid; ++cc) {
                    __syncwarp();
                    tmem_ld_x32(t_lane + buf * kRows + cc * 32, v);
                    const int nv = kt.valid - cc * 32;
                    float cmax = v[0];
                    if (nv >= 32) {
#pragma unroll
                        for (int e = 1; e < 32; ++e) cmax = fmaxf(cmax, v[e]);
                    } else {
#pragma unroll
                        for (int e = 1; e < 32; ++e) cmax = e < nv ? fmaxf(cmax, v[e]) : cmax;
                    }
                    if (cmax > m_raw) {
                        z *= exp2f((m_raw - cmax) * scale2);
                        m_raw = cmax;
                    }
                    const float negm = -(m_raw * scale2);
                    if (nv >= 32) {
#pragma unroll
                        for (int e = 0; e < 32; ++e) z += exp2f(fmaf(v[e], scale2, negm));
                    } else {
#pragma unroll
                        for (int e = 0; e < 32; ++e) z += e < nv ? exp2f(fmaf(v[e], scale2, negm)) : 0.f;
                    }
                }
                tc_fence_before();
                __syncwarp();
                if (lane == 0) mbar_arrive(&acc_empty[buf]);
            }
            const int prow = p0_lse + my_row;
            if (done && prow < u.n_q) {
                const int h = u.G * mv.hpg + hh_lse;
                const int64_t row = ((int64_t)u.l * mv.Hq + h) * bv.total_q + u.q0 + prow;
                const float m2 = m_raw * scale2;
                p.row_stats[row] = make_float2(m2, 1.0f / z);
                if (p.row_lse) p.row_lse[row] = (m2 + log2f(z)) * kLn2;
            }
        } else {
            float col = 0.f;
            bool done = true;
            for (int i = 0; i < n_iter; ++i) {
                const int buf = i % kAccBufs, bph = (i / kAccBufs) & 1;
                const int h = u.G * mv.hpg + i / q_blocks, p0 = (i % q_blocks) * kRows;
                const int nvalid = min(kRows, u.n_q - p0);
                // each warp stages the row block's statistics for itself (no CTA-wide barrier inside this loop)
                float2 *sm = stats_sm + ((warp - 2) * 2 + (i & 1)) * kRows;
                const float2 *gstats = p.row_stats + ((int64_t)u.l * mv.Hq + h) * bv.total_q + u.q0 + p0;
                for (int t = lane; t < kRows; t += 32) {
                    const float2 st = t < nvalid ? gstats[t] : make_float2(0.f, 0.f);
                    sm[t] = make_float2(-st.x, st.y);
                }
                __syncwarp();
                if (!__all_sync(0xffffffffu, mbar_wait(&acc_full[buf], bph, abort_flag))) { done = false; break; }
                tc_fence_after();
                for (int cc = 0; cc * 32 < nvalid; ++cc) {
                    __syncwarp();
                    tmem_ld_x32(t_lane + buf * kRows + cc * 32, v);
                    const int nv = nvalid - cc * 32;
                    if (nv >= 32) {
#pragma unroll
                        for (int e = 0; e < 32; ++e) {
                            const float2 s2 = sm[cc * 32 + e];
                            col = fmaf(exp2f(fmaf(v[e], scale2, s2.x)), s2.y, col);
                        }
                    } else {
#pragma unroll
                        for (int e = 0; e < 32; ++e) {
                            if (e < nv) {
                                const float2 s2 = sm[cc * 32 + e];
                                col = fmaf(exp2f(fmaf(v[e], scale2, s2.x)), s2.y, col);
                            }
                        }
                    }
                }
                tc_fence_before();
                __syncwarp();
                if (lane == 0) mbar_arrive(&acc_empty[buf]);
            }
            if (done && my_row < my_tile.valid)
                p.scores[((int64_t)u.l * mv.G + u.G) * ((int64_t)bv.total_cache + bv.total_chunk) + u.cache0 + u.chunk0 +
                         my_tile.j0 + my_row] = col;
        }
    }

    // ---- common epilogue: everyone meets here, also after a timed-out wait
    tc_fence_before();
    __syncthreads();
    if (threadIdx.x == 0 && *abort_flag) atomicOr(p.status, FINCH_DEV_TIMEOUT);
    if (warp == 1) {
        __syncwarp();
        tc_fence_after();
        tmem_dealloc(tmem_base, 512);
    }
}

// ------------------------------------------------------------------------------------------------ host side

typedef CUresult (*EncodeTiledFn)(CUtensorMap *, CUtensorMapDataType, cuuint32_t, void *, const cuuint64_t *,
                                  const cuuint64_t *, const cuuint32_t *, const cuuint32_t *, CUtensorMapInterleave,
                                  CUtensorMapSwizzle, CUtensorMapL2promotion, CUtensorMapFloatOOBfill);

EncodeTiledFn encode_fn() {
    static EncodeTiledFn fn = []() -> EncodeTiledFn {
        void *p = nullptr;
        cudaDriverEntryPointQueryResult q;
        if (cudaGetDriverEntryPoint("cuTensorMapEncodeTiled", &p, cudaEnableDefault, &q) != cudaSuccess ||
            q != cudaDriverEntryPointSuccess) {
            (void)cudaGetLastError();
            return nullptr;
        }
        return (EncodeTiledFn)p;
    }();
    return fn;
}

// [layers][heads][tokens][d] bf16 view -> 4-D tensor map with a (64 elements x 128 rows) box, 128-byte swizzle.
bool make_map(CUtensorMap *map, const TensorView &t, int d, int64_t tokens, int heads, int layers) {
    EncodeTiledFn fn = encode_fn();
    if (!fn || !t.ptr || tokens <= 0) return false;
    const cuuint64_t dims[4] = {(cuuint64_t)d, (cuuint64_t)tokens, (cuuint64_t)heads, (cuuint64_t)layers};
    const cuuint64_t strides[3] = {(cuuint64_t)t.stride_tok * 2, (cuuint64_t)t.stride_head * 2,
                                   (cuuint64_t)t.stride_layer * 2};
    for (int i = 0; i < 3; ++i)
        if (strides[i] == 0 || strides[i] % 16 || strides[i] >= (1ull << 40)) return false;
    const cuuint32_t box[4] = {64, (cuuint32_t)kRows, 1, 1};
    const cuuint32_t estr[4] = {1, 1, 1, 1};
    return fn(map, CU_TENSOR_MAP_DATA_TYPE_BFLOAT16, 4, const_cast<char *>(t.ptr), dims, strides, box, estr,
              CU_TENSOR_MAP_INTERLEAVE_NONE, CU_TENSOR_MAP_SWIZZLE_128B, CU_TENSOR_MAP_L2_PROMOTION_L2_256B,
              CU_TENSOR_MAP_FLOAT_OOB_FILL_NONE) == CUDA_SUCCESS;
}

template <int D>
cudaError_t launch_d(const Ctx &ctx, const CUtensorMap &qm, const CUtensorMap &cm, const CUtensorMap &hm,
                     const TcParams &p, cudaStream_t stream) {
    constexpr int kSmem = 1024 + (1 + kStages) * (D / 64) * kSlabBytes + kAuxBytes;
    const ModelView &mv = ctx.model;
    const BatchView &bv = p.bv;
    cudaError_t e = cudaFuncSetAttribute(score_tc_kernel<kLse, D>, cudaFuncAttributeMaxDynamicSharedMemorySize, kSmem);
    if (e != cudaSuccess) return e;
    e = cudaFuncSetAttribute(score_tc_kernel<kColsum, D>, cudaFuncAttributeMaxDynamicSharedMemorySize, kSmem);
    if (e != cudaSuccess) return e;
    const int units = mv.L * mv.G;
    const int row_blocks = (bv.max_q + kRows - 1) / kRows;
    const int key_tiles = (bv.max_cache + kRows - 1) / kRows + (bv.max_chunk + kRows - 1) / kRows;
    dim3 g1(row_blocks * mv.hpg, units, bv.batch);
    score_tc_kernel<kLse, D><<<g1, kTcThreads, kSmem, stream>>>(qm, cm, hm, p);
    dim3 g2(key_tiles, units, bv.batch);
    score_tc_kernel<kColsum, D><<<g2, kTcThreads, kSmem, stream>>>(qm, cm, hm, p);
    ctx.launches += 2;
    return cudaGetLastError();
}

}  // namespace

bool score_tc_supported(const Ctx &ctx) {
    return ctx.cfg.dtype == FINCH_BF16 && (ctx.model.d == 64 || ctx.model.d == 128) && ctx.model.kvpg == 1;
}

// Returns cudaErrorNotSupported (and launches nothing) when the tensors cannot be described to the TMA unit; the
// caller then uses the warp-level path for every request.
cudaError_t launch_score_tc(const Ctx &ctx, const TensorView &q, const TensorView &cache_k, const TensorView &chunk_k,
                            const BatchView &bv, float *scores, float2 *row_stats, float *row_lse, int min_q,
                            cudaStream_t stream) {
    const ModelView &mv = ctx.model;
    if (mv.L * mv.G == 0 || bv.batch == 0 || bv.max_q == 0 || bv.max_cache + bv.max_chunk == 0) return cudaSuccess;
    CUtensorMap qm, cm, hm;
    if (!make_map(&qm, q, mv.d, bv.total_q, mv.Hq, mv.L)) return cudaErrorNotSupported;
    const bool have_cache = bv.max_cache > 0, have_chunk = bv.max_chunk > 0;
    if (have_cache && !make_map(&cm, cache_k, mv.d, bv.total_cache, mv.Hkv, mv.L)) return cudaErrorNotSupported;
    if (have_chunk && !make_map(&hm, chunk_k, mv.d, bv.total_chunk, mv.Hkv, mv.L)) return cudaErrorNotSupported;
    if (!have_cache) cm = hm;  // never dereferenced: no request has cache tiles
    if (!have_chunk) hm = cm;
    TcParams p{mv, bv, row_stats, row_lse, scores, ctx.d_status, min_q};
    return mv.d == 64 ? launch_d<64>(ctx, qm, cm, hm, p, stream) : launch_d<128>(ctx, qm, cm, hm, p, stream);
}

}  // namespace finch

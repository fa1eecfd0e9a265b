// Cache compaction: gather the kept K/V rows and positions into the next cache, in kept (ascending) order.
//
// One CTA copies kRowsPerCta output rows of one unit (layer, selection group, request) for every KV head of the
// group, K and V, as 16-byte pieces: consecutive threads move consecutive pieces of a row, so both the gathered
// reads (whole rows) and the writes (contiguous rows) are fully coalesced 128-bit accesses.  A CTA takes 256 rows
// so that the dependent chain in front of the copies (batch metadata -> kept indices -> source addresses) is paid
// once per 128 KiB moved, and every thread has eight 16-byte loads in flight before its first store.
#include <cuda_bf16.h>

#include "finch_internal.cuh"

namespace finch {
namespace {

constexpr int kRowsPerCta = 256;  // = kCompactThreads: one thread fetches one kept index
constexpr int kCompactThreads = 256;

// ---- rotary re-positioning (Method, "Managing the Cache"): a kept key that moves from candidate index j to output
// slot i is rotated by delta = i - j positions; pair t of the row turns by delta * theta^(-2t/d).  Cosine and sine
// come from the context's table (computed in double, one row per distance |delta|; a negative delta flips the sine's
// sign), the rotation itself is fp32, the result is rounded to the storage type.
__device__ __forceinline__ float bf16_lo(uint32_t w) { return __uint_as_float(w << 16); }
__device__ __forceinline__ float bf16_hi(uint32_t w) { return __uint_as_float(w & 0xffff0000u); }
__device__ __forceinline__ uint32_t pack_bf16(float lo, float hi) {  // both rounded to nearest even, one instruction
    const __nv_bfloat162 v = __floats2bfloat162_rn(lo, hi);
    return *(const uint32_t *)&v;
}
__device__ __forceinline__ void rotate_pair(float x, float y, float2 cs, float sign, float &xo, float &yo) {
    const float sn = cs.y * sign;
    xo = fmaf(x, cs.x, -(y * sn));
    yo = fmaf(y, cs.x, x * sn);
}
// 16 bytes of x coordinates and the 16 bytes of their partners (kElems pairs, pairs (t, t + d/2)), rotated in place.
// cs points at the table entries of the kElems pairs.
template <int kElems>
__device__ __forceinline__ void rotate_pieces(uint4 &px, uint4 &py, const float2 *cs, float sign) {
    uint32_t *wx = (uint32_t *)&px, *wy = (uint32_t *)&py;
    float2 t[kElems];
#pragma unroll
    for (int e = 0; e < kElems / 2; ++e) {
        const float4 two = __ldg((const float4 *)cs + e);
        t[2 * e] = make_float2(two.x, two.y);
        t[2 * e + 1] = make_float2(two.z, two.w);
    }
    if (kElems == 4) {  // fp32
#pragma unroll
        for (int e = 0; e < 4; ++e) {
            float xo, yo;
            rotate_pair(__uint_as_float(wx[e]), __uint_as_float(wy[e]), t[e], sign, xo, yo);
            wx[e] = __float_as_uint(xo);
            wy[e] = __float_as_uint(yo);
        }
    } else {  // bf16, two per word
#pragma unroll
        for (int e = 0; e < 4; ++e) {
            float x0, y0, x1, y1;
            rotate_pair(bf16_lo(wx[e]), bf16_lo(wy[e]), t[2 * e], sign, x0, y0);
            rotate_pair(bf16_hi(wx[e]), bf16_hi(wy[e]), t[2 * e + 1], sign, x1, y1);
            wx[e] = pack_bf16(x0, x1);
            wy[e] = pack_bf16(y0, y1);
        }
    }
}
// One 16-byte piece whose pairs are neighbouring coordinates (2t, 2t + 1): kElems / 2 pairs.
template <int kElems>
__device__ __forceinline__ void rotate_interleaved(uint4 &pv, const float2 *cs, float sign) {
    uint32_t *w = (uint32_t *)&pv;
    float2 t[kElems / 2];
#pragma unroll
    for (int e = 0; e < kElems / 4; ++e) {
        const float4 two = __ldg((const float4 *)cs + e);
        t[2 * e] = make_float2(two.x, two.y);
        t[2 * e + 1] = make_float2(two.z, two.w);
    }
    if (kElems == 4) {
#pragma unroll
        for (int e = 0; e < 2; ++e) {
            float xo, yo;
            rotate_pair(__uint_as_float(w[2 * e]), __uint_as_float(w[2 * e + 1]), t[e], sign, xo, yo);
            w[2 * e] = __float_as_uint(xo);
            w[2 * e + 1] = __float_as_uint(yo);
        }
    } else {
#pragma unroll
        for (int e = 0; e < 4; ++e) {
            float xo, yo;
            rotate_pair(bf16_lo(w[e]), bf16_hi(w[e]), t[e], sign, xo, yo);
            w[e] = pack_bf16(xo, yo);
        }
    }
}

// The compaction with re-positioned keys: same decomposition as compact_kernel below (a warp walks the 16-byte
// pieces of [K | V] x KV heads of a row, four rows of loads in flight per thread), but a K piece is rotated between
// its load and its store.  With pairs (t, t + d/2) the thread that owns a piece of the row's first half also moves
// the partner piece of the second half.
template <int kElems>
__global__ void __launch_bounds__(kCompactThreads)
compact_rope_kernel(ModelView mv, BatchView bv, const int *kept_idx, const int *out_len, TensorView cache_k,
                    TensorView cache_v, const int *cache_pos, TensorView chunk_k, TensorView chunk_v,
                    const int *chunk_pos, TensorView out_k, TensorView out_v, int *out_pos, int *status) {
    __shared__ int src_idx[kRowsPerCta];
    dependency_wait();
    const UnitInfo u = unit_info(mv, bv, blockIdx.y, blockIdx.z);
    if (!u.ok) {
        if (threadIdx.x == 0) atomicOr(status, FINCH_DEV_BAD_BATCH);
        return;
    }
    int r = out_len[u.b];
    if (r > u.cap) r = u.cap;
    const int i0 = blockIdx.x * kRowsPerCta;
    if (i0 >= r) return;
    const int rows = min(kRowsPerCta, r - i0);
    const int64_t unit_off = ((int64_t)u.l * mv.G + u.G) * bv.total_cache + u.cache0;
    if (threadIdx.x < rows) {
        int j = kept_idx[unit_off + i0 + threadIdx.x];
        // a distance beyond the table (only possible when out_len exceeds the candidate count) is refused as well
        if (j < 0 || j >= u.N || abs(i0 + (int)threadIdx.x - j) >= mv.rope_rows) {
            atomicOr(status, FINCH_DEV_BAD_INDEX);
            j = -1;
        } else {
            out_pos[unit_off + i0 + threadIdx.x] = j < u.c ? cache_pos[unit_off + j] : chunk_pos[u.chunk0 + j - u.c];
        }
        src_idx[threadIdx.x] = j;
    }
    __syncthreads();

    const int pieces = mv.d * mv.elem_bytes / 16;
    const int per_row = pieces * 2 * mv.kvpg;
    const int tx = threadIdx.x & 31, ty = threadIdx.x >> 5;
    constexpr int kRowsInFlight = kCompactThreads / 32;
    constexpr int kBatch = 4;
    const bool split_pairs = mv.rope_pairing == 0;
    const int half = mv.d / 2;
    for (int cs = tx; cs < per_row; cs += 32) {
        const int piece = cs % pieces, which = cs / pieces;
        const int kvh = u.G * mv.kvpg + which / 2;
        const bool is_v = which & 1;
        // with pairs (t, t + d/2) the second half of a K row is written by the owner of the first half
        if (!is_v && split_pairs && piece >= pieces / 2) continue;
        const bool two = !is_v && split_pairs;  // this thread moves a partner piece as well
        const TensorView &ca = is_v ? cache_v : cache_k;
        const TensorView &ch = is_v ? chunk_v : chunk_k;
        const TensorView &dst = is_v ? out_v : out_k;
        const int64_t e = mv.elem_bytes;
        const char *ca_base = ca.ptr + ((int64_t)u.l * ca.stride_layer + (int64_t)kvh * ca.stride_head +
                                        (int64_t)u.cache0 * ca.stride_tok) * e + piece * 16;
        const char *ch_base = ch.ptr + ((int64_t)u.l * ch.stride_layer + (int64_t)kvh * ch.stride_head +
                                        (int64_t)(u.chunk0 - u.c) * ch.stride_tok) * e + piece * 16;
        char *dst_base = const_cast<char *>(dst.ptr) + ((int64_t)u.l * dst.stride_layer + (int64_t)kvh * dst.stride_head +
                                                        (int64_t)(u.cache0 + i0) * dst.stride_tok) * e + piece * 16;
        const int64_t ca_step = ca.stride_tok * e, ch_step = ch.stride_tok * e, dst_step = dst.stride_tok * e;
        const int half_bytes = half * mv.elem_bytes;  // distance to the partner piece (pairs (t, t + d/2))
        // first pair of this piece: kElems pairs per piece with split pairs, kElems / 2 with neighbouring pairs
        const float2 *table = mv.rope_table + (split_pairs ? piece * kElems : piece * (kElems / 2));
#pragma unroll 1
        for (int k0 = 0; k0 * kRowsInFlight < rows; k0 += kBatch) {
            uint4 a[kBatch], b[kBatch];
#pragma unroll
            for (int k = 0; k < kBatch; ++k) {  // this batch's loads first ..
                const int row = ty + (k0 + k) * kRowsInFlight;
                const int j = row < rows ? src_idx[row] : -1;
                if (j >= 0) {
                    const char *src = j < u.c ? ca_base + j * ca_step : ch_base + j * ch_step;
                    a[k] = __ldg((const uint4 *)src);
                    if (two) b[k] = __ldg((const uint4 *)(src + half_bytes));
                }
            }
#pragma unroll
            for (int k = 0; k < kBatch; ++k) {  // .. then the rotations and the stores
                const int row = ty + (k0 + k) * kRowsInFlight;
                const int j = row < rows ? src_idx[row] : -1;
                if (j < 0) continue;
                const int delta = i0 + row - j;
                const float2 *cs_row = table + (int64_t)abs(delta) * half;
                const float sign = delta < 0 ? -1.f : 1.f;
                if (two) {
                    rotate_pieces<kElems>(a[k], b[k], cs_row, sign);
                    *(uint4 *)(dst_base + row * dst_step + half_bytes) = b[k];
                } else if (!is_v) {
                    rotate_interleaved<kElems>(a[k], cs_row, sign);
                }
                *(uint4 *)(dst_base + row * dst_step) = a[k];
            }
        }
    }
}

__global__ void __launch_bounds__(kCompactThreads)
compact_kernel(ModelView mv, BatchView bv, const int *kept_idx, const int *out_len, TensorView cache_k,
               TensorView cache_v, const int *cache_pos, TensorView chunk_k, TensorView chunk_v, const int *chunk_pos,
               TensorView out_k, TensorView out_v, int *out_pos, int *status) {
    __shared__ int src_idx[kRowsPerCta];
    dependency_wait();  // no early launch of the next kernel: this grid runs in many waves and needs every slot
    const UnitInfo u = unit_info(mv, bv, blockIdx.y, blockIdx.z);
    if (!u.ok) {
        if (threadIdx.x == 0) atomicOr(status, FINCH_DEV_BAD_BATCH);
        return;
    }
    int r = out_len[u.b];
    if (r > u.cap) r = u.cap;
    const int i0 = blockIdx.x * kRowsPerCta;
    if (i0 >= r) return;
    const int rows = min(kRowsPerCta, r - i0);
    const int64_t unit_off = ((int64_t)u.l * mv.G + u.G) * bv.total_cache + u.cache0;

    if (threadIdx.x < rows) {
        int j = kept_idx[unit_off + i0 + threadIdx.x];
        if (j < 0 || j >= u.N) {
            atomicOr(status, FINCH_DEV_BAD_INDEX);
            j = -1;
        } else {
            out_pos[unit_off + i0 + threadIdx.x] = j < u.c ? cache_pos[unit_off + j] : chunk_pos[u.chunk0 + j - u.c];
        }
        src_idx[threadIdx.x] = j;
    }
    __syncthreads();

    const int pieces = mv.d * mv.elem_bytes / 16;  // 16-byte pieces per row
    const int per_row = pieces * 2 * mv.kvpg;      // K and V, every KV head of the group
    // A warp owns 32 consecutive pieces of an output row (fully coalesced) and walks the CTA's rows eight apart;
    // everything that does not depend on the row is computed once per thread, outside the row loop.
    const int tx = threadIdx.x & 31, ty = threadIdx.x >> 5;
    constexpr int kRowsInFlight = kCompactThreads / 32;
    for (int cs = tx; cs < per_row; cs += 32) {
        const int piece = cs % pieces, which = cs / pieces;  // which = kv * 2 + {0: K, 1: V}
        const int kvh = u.G * mv.kvpg + which / 2;
        const bool is_v = which & 1;
        const TensorView &ca = is_v ? cache_v : cache_k;
        const TensorView &ch = is_v ? chunk_v : chunk_k;
        const TensorView &dst = is_v ? out_v : out_k;
        const int64_t e = mv.elem_bytes;
        const char *ca_base = ca.ptr + ((int64_t)u.l * ca.stride_layer + (int64_t)kvh * ca.stride_head +
                                        (int64_t)u.cache0 * ca.stride_tok) * e + piece * 16;
        const char *ch_base = ch.ptr + ((int64_t)u.l * ch.stride_layer + (int64_t)kvh * ch.stride_head +
                                        (int64_t)(u.chunk0 - u.c) * ch.stride_tok) * e + piece * 16;
        char *dst_base = const_cast<char *>(dst.ptr) + ((int64_t)u.l * dst.stride_layer + (int64_t)kvh * dst.stride_head +
                                                        (int64_t)(u.cache0 + i0) * dst.stride_tok) * e + piece * 16;
        const int64_t ca_step = ca.stride_tok * e, ch_step = ch.stride_tok * e, dst_step = dst.stride_tok * e;
        constexpr int kBatch = 8;  // rows per thread whose loads are issued before the first store
#pragma unroll 1
        for (int k0 = 0; k0 * kRowsInFlight < rows; k0 += kBatch) {
            uint4 v[kBatch];
#pragma unroll
            for (int k = 0; k < kBatch; ++k) {  // all of this batch's loads first ..
                const int row = ty + (k0 + k) * kRowsInFlight;
                const int j = row < rows ? src_idx[row] : -1;
                if (j >= 0) v[k] = __ldg((const uint4 *)(j < u.c ? ca_base + j * ca_step : ch_base + j * ch_step));
            }
#pragma unroll
            for (int k = 0; k < kBatch; ++k) {  // .. then its stores
                const int row = ty + (k0 + k) * kRowsInFlight;
                if (row < rows && src_idx[row] >= 0) *(uint4 *)(dst_base + row * dst_step) = v[k];
            }
        }
    }
}

}  // namespace

cudaError_t launch_compact(const Ctx &ctx, const int *kept_idx, const int *out_len, const TensorView &cache_k,
                           const TensorView &cache_v, const int *cache_pos, const TensorView &chunk_k,
                           const TensorView &chunk_v, const int *chunk_pos, const BatchView &bv, const TensorView &out_k,
                           const TensorView &out_v, int *out_pos, cudaStream_t stream) {
    const ModelView &mv = ctx.model;
    const int units = mv.L * mv.G;
    const int row_blocks = (bv.max_budget + kRowsPerCta - 1) / kRowsPerCta;
    if (units == 0 || bv.batch == 0 || row_blocks == 0) return cudaSuccess;
    dim3 grid(row_blocks, units, bv.batch);
    ctx.launches += 1;
    if (mv.rope_theta > 0.f) {
        auto kernel = mv.elem_bytes == 4 ? compact_rope_kernel<4> : compact_rope_kernel<8>;
        return launch_chained(kernel, grid, dim3(kCompactThreads), 0, stream, mv, bv, kept_idx, out_len, cache_k, cache_v,
                              cache_pos, chunk_k, chunk_v, chunk_pos, out_k, out_v, out_pos, ctx.d_status);
    }
    return launch_chained(compact_kernel, grid, dim3(kCompactThreads), 0, stream, mv, bv, kept_idx, out_len, cache_k, cache_v,
                          cache_pos, chunk_k, chunk_v, chunk_pos, out_k, out_v, out_pos, ctx.d_status);
}

}  // namespace finch

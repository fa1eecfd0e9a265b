// Cache compaction: gather the kept K/V rows and positions into the next cache, in kept (ascending) order.
//
// One CTA copies kRowsPerCta output rows of one unit (layer, selection group, request) for every KV head of the
// group, K and V, as 16-byte pieces: consecutive threads move consecutive pieces of a row, so both the gathered
// reads (whole rows) and the writes (contiguous rows) are fully coalesced 128-bit accesses.  A CTA takes 256 rows
// so that the dependent chain in front of the copies (batch metadata -> kept indices -> source addresses) is paid
// once per 128 KiB moved, and every thread has eight 16-byte loads in flight before its first store.
#include "finch_internal.cuh"

namespace finch {
namespace {

constexpr int kRowsPerCta = 256;  // = kCompactThreads: one thread fetches one kept index
constexpr int kCompactThreads = 256;

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
    return launch_chained(compact_kernel, grid, dim3(kCompactThreads), 0, stream, mv, bv, kept_idx, out_len, cache_k, cache_v,
                          cache_pos, chunk_k, chunk_v, chunk_pos, out_k, out_v, out_pos, ctx.d_status);
}

}  // namespace finch

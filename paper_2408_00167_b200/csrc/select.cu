// Top-r selection per (layer, selection group, request) without a sort.
//
// One CTA per unit.  Scores are mapped to order-preserving 32-bit keys; four 8-bit radix passes (most significant
// digit first) locate the key T of the r-th largest score and how many candidates are strictly above it.  A final
// ordered sweep keeps every candidate above T plus the lowest-indexed candidates equal to T until r are kept, and
// writes the kept indices in increasing order (two block-wide prefix sums per 4096 candidates).
#include "finch_internal.cuh"

namespace finch {
namespace {

constexpr int kSelThreadsWide = 1024;  // units of more than 1024 candidates: two CTAs per SM
constexpr int kSelThreadsSmall = 256;  // short units: eight CTAs per SM, so that many small units run in one wave

// Order-preserving key: larger score <=> larger key.  -0 is folded into +0; NaN gets key 0, below every number.
__device__ __forceinline__ uint32_t order_key(float s) {
    if (s != s) return 0u;
    uint32_t u = __float_as_uint(s);
    if ((u << 1) == 0u) u = 0u;  // -0 -> +0
    return (u & 0x80000000u) ? ~u : (u | 0x80000000u);
}

// 32 registers per thread, so 2048 threads per SM whatever the CTA size: two CTAs of 1024 threads (256 units of 4096
// candidates run in one wave) or eight of 256 (1024 units of 1024 candidates do)
template <int kSelThreads>
__global__ void __launch_bounds__(kSelThreads, 2048 / kSelThreads)
select_kernel(ModelView mv, BatchView bv, const float *scores, int *kept_idx, int *out_len, int smem_keys, int *status) {
    constexpr int kSelWarps = kSelThreads / 32;
    extern __shared__ uint32_t key_cache[];  // the first min(N, smem_keys) keys
    __shared__ int hist[256];
    __shared__ int warp_tot[2][kSelWarps];
    __shared__ int sel_digit, sel_above;

    dependency_wait();
    dependents_may_launch();
    const int unit = blockIdx.x;
    const UnitInfo u = unit_info(mv, bv, unit, blockIdx.y);
    const int N = u.N;
    int r = bv.budget[u.b];
    r = r < N ? r : N;
    r = r < 0 ? 0 : r;
    if (!u.ok || r > u.cap || r > bv.max_budget) {  // block-uniform
        if (threadIdx.x == 0) {
            atomicOr(status, FINCH_DEV_BAD_BATCH);
            if (unit == 0) out_len[u.b] = 0;
        }
        return;
    }
    if (unit == 0 && threadIdx.x == 0) out_len[u.b] = r;
    if (r == 0) return;

    const float *sc = scores + ((int64_t)u.l * mv.G + u.G) * ((int64_t)bv.total_cache + bv.total_chunk) + u.cache0 +
                      u.chunk0;
    int *kept = kept_idx + ((int64_t)u.l * mv.G + u.G) * bv.total_cache + u.cache0;

    if (r == N) {  // a budget at or above the candidate count keeps everything, in order
        for (int j = threadIdx.x; j < N; j += kSelThreads) kept[j] = j;
        return;
    }

    const int n_cached = N < smem_keys ? N : smem_keys;
    for (int j = threadIdx.x; j < n_cached; j += kSelThreads) key_cache[j] = order_key(sc[j]);
    __syncthreads();
    auto key_at = [&](int j) -> uint32_t { return j < n_cached ? key_cache[j] : order_key(sc[j]); };

    // ---- radix search for the r-th largest key
    uint32_t prefix = 0, mask = 0;
    int remaining = r;  // rank, among the keys matching the prefix, of the key we look for (1 = largest)
    for (int shift = 24; shift >= 0; shift -= 8) {
        if (threadIdx.x < 256) hist[threadIdx.x] = 0;
        __syncthreads();
        for (int j = threadIdx.x; j < N; j += kSelThreads) {
            const uint32_t k = key_at(j);
            if ((k & mask) == prefix) atomicAdd(&hist[(k >> shift) & 255u], 1);
        }
        __syncthreads();
        if (threadIdx.x < 32) {
            // lane i owns digits 255-8i .. 248-8i (descending); find the digit where the running count reaches
            // `remaining`
            const int lane = threadIdx.x;
            int mine = 0;
#pragma unroll
            for (int t = 0; t < 8; ++t) mine += hist[255 - 8 * lane - t];
            int incl = mine;
#pragma unroll
            for (int off = 1; off < 32; off <<= 1) {
                const int v = __shfl_up_sync(0xffffffffu, incl, off);
                if (lane >= off) incl += v;
            }
            int above = incl - mine;
            if (above < remaining && remaining <= incl) {
                for (int t = 0; t < 8; ++t) {
                    const int digit = 255 - 8 * lane - t;
                    const int cnt = hist[digit];
                    if (remaining <= above + cnt) {
                        sel_digit = digit;
                        sel_above = above;
                        break;
                    }
                    above += cnt;
                }
            }
        }
        __syncthreads();
        prefix |= (uint32_t)sel_digit << shift;
        mask |= 255u << shift;
        remaining -= sel_above;
        __syncthreads();
    }
    const uint32_t T = prefix;
    const int ties_to_keep = remaining;  // >= 1

    // ---- ordered sweep: keep key > T, and the first `ties_to_keep` keys == T.  A thread takes four consecutive
    // candidates, so two block-wide exclusive scans per 4096 candidates (ties before me, kept before me) place every
    // kept index; the output is ascending by construction.
    const int lane = threadIdx.x & 31, warp = threadIdx.x >> 5;
    auto block_scan = [&](int v, int *buf, int &total) -> int {  // exclusive prefix of v over the block, in thread order
        int incl = v;
#pragma unroll
        for (int off = 1; off < 32; off <<= 1) {
            const int up = __shfl_up_sync(0xffffffffu, incl, off);
            if (lane >= off) incl += up;
        }
        if (lane == 31) buf[warp] = incl;
        __syncthreads();
        if (warp == 0) {
            int t = lane < kSelWarps ? buf[lane] : 0;
#pragma unroll
            for (int off = 1; off < 32; off <<= 1) {
                const int up = __shfl_up_sync(0xffffffffu, t, off);
                if (lane >= off) t += up;
            }
            if (lane < kSelWarps) buf[lane] = t;  // inclusive totals of the warps
        }
        __syncthreads();
        total = buf[kSelWarps - 1];
        return (warp ? buf[warp - 1] : 0) + incl - v;
    };
    if (N <= kSelThreads) {
        // one candidate per thread at most: ballots and the 32 warp totals are cheaper than two scans
        const int j = threadIdx.x;
        const uint32_t k = j < N ? key_at(j) : 0u;
        const bool gt = j < N && k > T;
        const bool eq = j < N && k == T;
        const uint32_t eq_ballot = __ballot_sync(0xffffffffu, eq);
        if (lane == 0) warp_tot[0][warp] = __popc(eq_ballot);
        __syncthreads();
        int eq_before = 0;
        for (int w = 0; w < warp; ++w) eq_before += warp_tot[0][w];
        eq_before += __popc(eq_ballot & ((1u << lane) - 1u));
        const bool keep = gt || (eq && eq_before < ties_to_keep);
        const uint32_t keep_ballot = __ballot_sync(0xffffffffu, keep);
        if (lane == 0) warp_tot[1][warp] = __popc(keep_ballot);
        __syncthreads();
        int keep_before = 0;
        for (int w = 0; w < warp; ++w) keep_before += warp_tot[1][w];
        keep_before += __popc(keep_ballot & ((1u << lane) - 1u));
        if (keep) kept[keep_before] = j;
        return;
    }
    constexpr int kPerThread = 4;
    int base_eq = 0, base_keep = 0;
    for (int j0 = 0; j0 < N; j0 += kSelThreads * kPerThread) {
        const int j = j0 + threadIdx.x * kPerThread;
        uint32_t k[kPerThread];
#pragma unroll
        for (int e = 0; e < kPerThread; ++e) k[e] = j + e < N ? key_at(j + e) : 0u;
        int n_eq = 0;
#pragma unroll
        for (int e = 0; e < kPerThread; ++e) n_eq += (j + e < N && k[e] == T) ? 1 : 0;
        int eq_all;
        int eq_before = base_eq + block_scan(n_eq, warp_tot[0], eq_all);
        bool keep[kPerThread];
        int n_keep = 0;
#pragma unroll
        for (int e = 0; e < kPerThread; ++e) {
            const bool in = j + e < N;
            const bool eq = in && k[e] == T;
            keep[e] = in && (k[e] > T || (eq && eq_before < ties_to_keep));
            eq_before += eq ? 1 : 0;
            n_keep += keep[e] ? 1 : 0;
        }
        int keep_all;
        int slot = base_keep + block_scan(n_keep, warp_tot[1], keep_all);
#pragma unroll
        for (int e = 0; e < kPerThread; ++e)
            if (keep[e]) kept[slot++] = j + e;
        base_eq += eq_all;
        base_keep += keep_all;
        // the next iteration's first scan writes warp_tot[0] after this iteration's last barrier, and warp_tot[1]
        // after two more: every read above has been made by then
    }
}

}  // namespace

cudaError_t launch_select(const Ctx &ctx, const float *scores, const BatchView &bv, int *kept_idx, int *out_len,
                          cudaStream_t stream) {
    const ModelView &mv = ctx.model;
    const int units = mv.L * mv.G;
    if (units == 0 || bv.batch == 0) return cudaSuccess;
    const int max_n = bv.max_cache + bv.max_chunk;
    int smem_keys = max_n < 40960 ? max_n : 40960;  // up to 160 KiB of keys on chip; longer inputs re-read global
    if (smem_keys < 1) smem_keys = 1;
    const size_t smem = (size_t)smem_keys * sizeof(uint32_t);
    dim3 grid(units, bv.batch);
    ctx.launches += 1;
    if (max_n <= 1024)
        return launch_chained(select_kernel<kSelThreadsSmall>, grid, dim3(kSelThreadsSmall), smem, stream, mv, bv, scores,
                              (int *)kept_idx, out_len, smem_keys, ctx.d_status);
    cudaError_t e =
        cudaFuncSetAttribute(select_kernel<kSelThreadsWide>, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)smem);
    if (e != cudaSuccess) return e;
    return launch_chained(select_kernel<kSelThreadsWide>, grid, dim3(kSelThreadsWide), smem, stream, mv, bv, scores,
                          (int *)kept_idx, out_len, smem_keys, ctx.d_status);
}

}  // namespace finch

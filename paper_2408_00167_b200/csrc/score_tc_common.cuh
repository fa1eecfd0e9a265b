// Pieces shared by the tensor-core scoring kernels: tile geometry, the candidate view, the packed fp32 arithmetic of
// the two sweeps (row log-sum-exp, column sums), the merge of partial row statistics and the TMA tensor maps.
#pragma once

#include <limits.h>

#include "finch_internal.cuh"
#include "sm100_ptx.cuh"

namespace finch {
namespace tc {

using namespace ptx;

constexpr int kRows = 128;       // rows per operand tile = MMA M = MMA N
constexpr int kSub = 64;         // prompt rows per sub-block (two per query tile)
constexpr int kQTiles = 4;       // query tiles resident at a time
constexpr int kGroups = 4;       // softmax groups (four warps each); accumulator number A goes to group A % 4
constexpr int kPlanBoundsInts = 1024;  // room for the per-CTA item bounds in the scratch (grid + 1 <= this)
constexpr int kAccBufs = 4;      // accumulators of 128 fp32 columns in tensor memory (all 512 columns), one per group
constexpr int kMaxStages = 4;    // key-tile ring
constexpr int kTcThreads = 64 + kGroups * 128;
constexpr int kSlabBytes = kRows * 128;                 // a 64-element (128-byte) wide slab of a 128-row tile
constexpr int kStatsBytes = 2 * kQTiles * kRows * 8;  // (-ref, weight) of the resident rows, double-buffered
constexpr int kLimitBytes = 2 * kQTiles * kRows * 4;  // visible-candidate count of the resident rows (masked variant)
constexpr int kAuxBytes = 1024 + kStatsBytes + kLimitBytes;
constexpr int kSmemLimit = 232448;                      // 227 KiB per CTA

enum { kLse = 0, kColsum = 1 };

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

// The group's prompt rows as a list of 64-row sub-blocks, head-major then position: sub-block sb covers rows
// [p0, p0 + valid) of the group's query head hh.  Query tile t packs sub-blocks 2t and 2t + 1.
struct SubBlock {
    int hh, p0, valid;
};
__device__ __forceinline__ SubBlock sub_block(int sb, int sbq, int n_sb, int n_q) {
    SubBlock s;
    s.hh = sb / sbq;
    s.p0 = (sb % sbq) * kSub;
    s.valid = sb < n_sb ? min(kSub, n_q - s.p0) : 0;
    return s;
}

__device__ __forceinline__ float ex2(float x) {
    float y;
    asm("ex2.approx.ftz.f32 %0, %1;" : "=f"(y) : "f"(x));
    return y;
}

// Packed pairs of fp32 (sm_100 executes these as one instruction on the FMA pipe).
__device__ __forceinline__ uint64_t pack2(float lo, float hi) {
    uint64_t r;
    asm("mov.b64 %0, {%1, %2};" : "=l"(r) : "f"(lo), "f"(hi));
    return r;
}
__device__ __forceinline__ void unpack2(uint64_t v, float &lo, float &hi) {
    asm("mov.b64 {%0, %1}, %2;" : "=f"(lo), "=f"(hi) : "l"(v));
}
__device__ __forceinline__ uint64_t fma2(uint64_t a, uint64_t b, uint64_t c) {
    uint64_t r;
    asm("fma.rn.f32x2 %0, %1, %2, %3;" : "=l"(r) : "l"(a), "l"(b), "l"(c));
    return r;
}
__device__ __forceinline__ float4 lds128(uint32_t addr) {
    float4 v;
    asm volatile("ld.shared.v4.f32 {%0, %1, %2, %3}, [%4];" : "=f"(v.x), "=f"(v.y), "=f"(v.z), "=f"(v.w) : "r"(addr));
    return v;
}
__device__ __forceinline__ uint64_t add2(uint64_t a, uint64_t b) {
    uint64_t r;
    asm("add.rn.f32x2 %0, %1, %2;" : "=l"(r) : "l"(a), "l"(b));
    return r;
}

// kLse: fold 32 columns (keys) of one accumulator row into the row's running (reference, sum of exp2).
// The reference is the maximum of the row's first chunk, not the running maximum: any reference works as long as
// the sum stays finite, and skipping the per-element maximum saves a quarter of the instructions.  If the sum
// overflows (a later logit more than ~2^7 base-2 units above the reference, or many nearly that far) the reference
// moves up and the chunk is redone.  Columns at or beyond nv hold no key and count nothing.
__device__ __forceinline__ void lse_chunk(const uint32_t (&r)[32], int nv, float scale2, float &m_raw, float &z) {
    float v[32];
#pragma unroll
    for (int e = 0; e < 32; ++e) v[e] = __uint_as_float(r[e]);
    if (nv < 32) {
#pragma unroll
        for (int e = 1; e < 32; ++e) v[e] = e < nv ? v[e] : -INFINITY;
    }
    if (m_raw == -INFINITY) {
        float cmax = v[0];
#pragma unroll
        for (int e = 1; e < 32; ++e) cmax = fmaxf(cmax, v[e]);
        m_raw = cmax;
    }
    for (int attempt = 0; attempt < 2; ++attempt) {
        const float negm = -(m_raw * scale2);
        const uint64_t s2 = pack2(scale2, scale2), n2 = pack2(negm, negm);
        uint64_t acc0 = 0, acc1 = 0;  // two pairs of partial sums (+0.0f bit patterns)
#pragma unroll
        for (int e = 0; e < 32; e += 4) {
            float x0, x1, x2, x3;
            unpack2(fma2(pack2(v[e], v[e + 1]), s2, n2), x0, x1);
            unpack2(fma2(pack2(v[e + 2], v[e + 3]), s2, n2), x2, x3);
            acc0 = add2(acc0, pack2(ex2(x0), ex2(x1)));
            acc1 = add2(acc1, pack2(ex2(x2), ex2(x3)));
        }
        float a0, a1, a2, a3;
        unpack2(acc0, a0, a1);
        unpack2(acc1, a2, a3);
        const float zn = z + ((a0 + a1) + (a2 + a3));
        if (!(zn > 3.0e38f)) {  // finite -- or NaN, on a lane that holds no prompt row: nothing to repair
            z = zn;
            break;
        }
        // overflow: move the reference up and redo the chunk
        float cmax = v[0];
#pragma unroll
        for (int e = 1; e < 32; ++e) cmax = fmaxf(cmax, v[e]);
        // The new reference must cover the chunk's largest logit and what has been summed so far (z = 2^e * [1, 2)
        // against the old reference, e from z's exponent field), so that the redone sum is at most 1 + 32.  The
        // factor between the two references (the same rounded products the chunks subtract) is applied in two
        // halves, since z may be near 2^127 while the factor is below the smallest normal number.
        const float lift = (float)(((__float_as_int(z) >> 23) & 0xff) - 126);
        const float m_new = fmaxf(cmax, fmaf(lift, __frcp_rn(scale2), m_raw));
        const float half_d = 0.5f * (__fmul_rn(m_raw, scale2) - __fmul_rn(m_new, scale2));
        z = (z * ex2(half_d)) * ex2(half_d);
        m_raw = m_new;
    }
}

// `live` is false on lanes whose row of the query tile holds no prompt row: they take part in the (warp-wide)
// loads but skip the arithmetic, whose input would be whatever the shared memory held before.
// lane_valid (masked variant): how many of the tile's columns this lane's row attends to; may be <= 0.
template <bool MASK>
__device__ __forceinline__ void lse_accumulate(uint32_t taddr, int valid, float scale2, bool live, float &m_raw,
                                               float &z, int lane_valid) {
    // one 32-column chunk at a time: with four softmax warps per scheduler the other warps cover the tensor-memory
    // latency, and a single register buffer keeps the kernel inside its register budget
#pragma unroll 1
    for (int cc = 0; cc * 32 < valid; ++cc) {
        uint32_t r[32];
        __syncwarp();
        tmem_ld_x32_issue(taddr + cc * 32, r);
        tmem_ld_x32_wait(r);
        if (MASK) {
            const int nv = min(valid, lane_valid) - cc * 32;
            if (live && nv > 0) lse_chunk(r, nv, scale2, m_raw, z);
        } else {
            if (live) lse_chunk(r, valid - cc * 32, scale2, m_raw, z);
        }
    }
}

// kColsum: add to (c0, c1) the weights exp2(s * scale2 - ref_r) * w_r of one accumulator row (a key) over the valid
// prompt rows of the query tile: v0 rows in its first 64-row half, v1 in its second.  The statistics are staged
// in pairs of rows, (-ref_a, -ref_b, w_a, w_b), so that one 128-bit load feeds two packed operations.
// Masked variant: lim2 holds, per pair of rows, how many candidates each row attends to; this thread's key has
// candidate index j and counts for a row only if j is below that row's number.
template <bool MASK>
__device__ __forceinline__ void colsum_chunk(const uint32_t (&r)[32], int nv, float scale2, uint32_t sm4, float &c0,
                                             float &c1, const int2 *lim2, int j) {
    float v[32];
#pragma unroll
    for (int e = 0; e < 32; ++e) v[e] = __uint_as_float(r[e]);
    if (nv < 32) {
#pragma unroll
        for (int e = 0; e < 32; ++e) v[e] = e < nv ? v[e] : -INFINITY;  // rows past the prompt weigh nothing
    }
    const uint64_t s2 = pack2(scale2, scale2);
    uint64_t acc = pack2(c0, c1);
#pragma unroll
    for (int e = 0; e < 32; e += 2) {
        const float4 s4 = lds128(sm4 + (e / 2) * 16);  // two prompt rows: (-ref_a, -ref_b, w_a, w_b)
        float x0, x1;
        unpack2(fma2(pack2(v[e], v[e + 1]), s2, pack2(s4.x, s4.y)), x0, x1);
        if (MASK) {
            const int2 l2 = lim2[e / 2];
            x0 = j < l2.x ? x0 : -INFINITY;  // exp2(-inf) = 0: the row does not see this key
            x1 = j < l2.y ? x1 : -INFINITY;
        }
        acc = fma2(pack2(ex2(x0), ex2(x1)), pack2(s4.z, s4.w), acc);
    }
    unpack2(acc, c0, c1);
}

template <bool MASK>
__device__ __forceinline__ void colsum_accumulate(uint32_t taddr, int v0, int v1, float scale2, const float2 *sm,
                                                  float &c0, float &c1, const int *lim, int j) {
    const uint32_t sm4 = smem_u32(sm);  // shared-window address: the loads below are ld.shared, not generic
    // chunks 0 and 1 cover the tile's first 64-row half (always present), chunks 2 and 3 the second half
    const int last = v1 > 0 ? 4 : 2;
#pragma unroll 1
    for (int cc = 0; cc < last; ++cc) {
        uint32_t r[32];
        __syncwarp();
        tmem_ld_x32_issue(taddr + cc * 32, r);
        tmem_ld_x32_wait(r);
        colsum_chunk<MASK>(r, (cc < 2 ? v0 : v1) - (cc & 1) * 32, scale2, sm4 + cc * 256, c0, c1,
                           (const int2 *)lim + cc * 16, j);
    }
}


// ---- merging partial row statistics.  A part is (reference, sum of exp2 against that reference), both in base-2
// logit units; parts are folded in a fixed order into a running (M, Z), then turned into the pair the column
// sweep uses: weights are exp2(s2 - R) * w with R = M + floor(log2 Z) and w = 2^floor(log2 Z) / Z in (1/2, 1], so
// the exponent never exceeds a few units whatever reference the parts were summed against.
__device__ __forceinline__ void merge_part(float2 pm, float &M, float &Z) {
    if (!(pm.y > 0.f)) return;  // a part that saw none of this row's logits
    // A part's sum can be as large as 2^127 against a reference that far below its largest logit: move the sum's
    // exponent into the reference first, so that neither factor below leaves the fp32 range.
    const int bits = __float_as_int(pm.y);  // pm.y >= 1: a normal number
    const int e = ((bits >> 23) & 0xff) - 127;
    const float px = pm.x + (float)e, py = __int_as_float((bits & 0x007fffff) | 0x3f800000);
    const float nm = fmaxf(M, px);
    Z = Z * ex2(M - nm) + py * ex2(px - nm);
    M = nm;
}
// One more part with sum 1 whose reference is a natural-log value (the keys a row attends to besides the candidates).
__device__ __forceinline__ void merge_self_term(float lse_nat, float &M, float &Z) {
    const float px = lse_nat * kLog2e;
    if (px > -INFINITY) {
        const float nm = fmaxf(M, px);
        Z = Z * ex2(M - nm) + ex2(px - nm);
        M = nm;
    }
}
// (M, Z) -> (-R, w); lse_nat receives the row's natural-log sum-exp.  A row that attends to nothing (Z = 0) weighs
// nothing: (0, 0) and -inf.
__device__ __forceinline__ float2 merged_pair(float M, float Z, float &lse_nat) {
    if (!(Z > 0.f)) {
        lse_nat = -INFINITY;
        return make_float2(0.f, 0.f);
    }
    // Z = 2^k * [1, 2) (a sum of terms in [1, 2) times factors <= 1, the largest of them 1)
    const int zbits = __float_as_int(Z);
    const int k = ((zbits >> 23) & 0xff) - 127;
    const float w = __fdividef(1.0f, __int_as_float((zbits & 0x007fffff) | 0x3f800000));
    lse_nat = (M + log2f(Z)) * kLn2;
    return make_float2(-(M + (float)k), w);
}

// ------------------------------------------------------------------------------------------------ host side

typedef CUresult (*EncodeTiledFn)(CUtensorMap *, CUtensorMapDataType, cuuint32_t, void *, const cuuint64_t *,
                                  const cuuint64_t *, const cuuint32_t *, const cuuint32_t *, CUtensorMapInterleave,
                                  CUtensorMapSwizzle, CUtensorMapL2promotion, CUtensorMapFloatOOBfill);

inline EncodeTiledFn encode_fn() {
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

// [layers][heads][tokens][d] bf16 view -> 4-D tensor map with a (64 elements x box_rows) box, 128-byte swizzle.
inline bool make_map(CUtensorMap *map, const TensorView &t, int d, int64_t tokens, int heads, int layers, int box_rows) {
    EncodeTiledFn fn = encode_fn();
    if (!fn || !t.ptr || tokens <= 0) return false;
    const cuuint64_t dims[4] = {(cuuint64_t)d, (cuuint64_t)tokens, (cuuint64_t)heads, (cuuint64_t)layers};
    const cuuint64_t strides[3] = {(cuuint64_t)t.stride_tok * 2, (cuuint64_t)t.stride_head * 2,
                                   (cuuint64_t)t.stride_layer * 2};
    for (int i = 0; i < 3; ++i)
        if (strides[i] == 0 || strides[i] % 16 || strides[i] >= (1ull << 40)) return false;
    const cuuint32_t box[4] = {64, (cuuint32_t)box_rows, 1, 1};
    const cuuint32_t estr[4] = {1, 1, 1, 1};
    return fn(map, CU_TENSOR_MAP_DATA_TYPE_BFLOAT16, 4, const_cast<char *>(t.ptr), dims, strides, box, estr,
              CU_TENSOR_MAP_INTERLEAVE_NONE, CU_TENSOR_MAP_SWIZZLE_128B, CU_TENSOR_MAP_L2_PROMOTION_L2_256B,
              CU_TENSOR_MAP_FLOAT_OOB_FILL_NONE) == CUDA_SUCCESS;
}

}  // namespace tc
}  // namespace finch

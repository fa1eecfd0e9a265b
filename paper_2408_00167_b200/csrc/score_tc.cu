// Prompt-guided scoring on the 5th-generation tensor cores (bf16 inputs, head_dim 64 or 128).
//
// One kernel template, two sweeps over the logits S = Q K^T of a unit (layer, KV head, request).  A CTA owns one
// split of the unit's 128-key tiles and keeps up to four 128-row tiles of the group's prompt queries resident in
// shared memory (a tile packs two 64-row sub-blocks, possibly of two query heads); the key tiles stream past them
// through a TMA ring, each read once per sweep.
//
//   kLse     D = Qtile x Ktile^T lands in tensor memory with one prompt row per lane, so each thread keeps the
//            online (max, sum exp2) of its own rows without cross-lane traffic -> per-split partial row statistics.
//   kColsum  D = Ktile x Qtile^T: one key per lane, so the sum over prompt rows of exp2(s - max) / sum is a private
//            running sum per thread -> scores.  Its prologue merges the splits' partial statistics (fixed order).
//
// Warp roles (576 threads): warp 0 lane 0 issues TMA loads (128-byte swizzle), warp 1 owns tensor memory and its
// lane 0 issues tcgen05.mma (128 x 128 x 16, fp32 accumulate), warps 2-17 form four softmax groups of four warps.
// Accumulators (key tile x query tile) are dealt to the groups round-robin, each group owning one 128-column
// accumulator: every scheduler then has four softmax warps, enough to keep the MUFU unit busy while one of them
// waits for its next accumulator.  Sums never cross threads: the first sweep keeps per-group partial statistics,
// the second writes per-group partial column sums that a small kernel adds in a fixed order.  mbarriers connect the
// roles; every wait is bounded and raises FINCH_DEV_TIMEOUT instead of hanging.  Candidate tiles never straddle the cache/chunk
// boundary: the cache's rows are tiled first, then the chunk's.
#include "score_tc_common.cuh"

namespace finch {
namespace {

using namespace ptx;
using namespace tc;

struct TcParams {
    ModelView mv;
    BatchView bv;
    float2 *partial;   // [splits][kGroups][L][Hq][total_q] (reference base-2 logit, sum exp2) per prompt row and part
    float2 *merged;    // [L][Hq][total_q] (-reference, weight) per prompt row after merging the parts
    float *row_lse;    // nullable
    float *scores;
    float *score_parts;  // [kGroups][L][G][total_cand] per-group partial column sums
    int *status;
    int splits;        // key splits per unit (grid x)
    int stages;        // key-tile ring depth that fits beside the resident queries
    int q_tiles;       // query tiles resident at a time (1..4), sized from the batch's longest prompt
    int n_items;       // work items = splits x units x requests, walked by a persistent grid
    const int *bounds;              // [grid + 1] first item of every CTA (work-weighted), or null: equal item counts
    unsigned long long *work_prefix;  // [batch + 1] accumulators of all items of the requests before b (plan scratch)
    // `mv` is the scoring view: one scoring unit per KV head.  A selection group that spans several KV heads (one
    // group per layer) is the sum of its heads' units, taken when the partial sums are combined.
    int out_groups;         // selection groups per layer
    int units_per_group;    // KV heads (scoring units) per selection group
};

// One work item = one key split of one unit.  A CTA walks a contiguous range of items (split fastest), so that
// consecutive items usually belong to the same unit and the resident query tiles can stay where they are.
struct Item {
    UnitInfo u;
    int key;  // identifies (unit, request): items with equal keys share their query tiles
    int split, t0, t1, tps, k_tiles;
    int sbq, n_sb, n_qt, n_chunks;
    bool run;
};

// A role's position in its CTA's item range.  Items are walked in order, so the position (split, group, layer,
// request) advances by counting, and everything that depends on the request alone (its batch metadata, tile counts)
// is computed when the request changes: per item there is no division and no load from global memory.  A role
// thread that stalls at every item boundary stalls the pipeline behind it.
struct Walk {
    int w, split, key, l, G, b;
    UnitInfo req;  // metadata of request `req.b` (-1: none read yet); l and G are not kept here
    int k_tiles, tps, sbq, n_sb, n_qt, n_chunks;
    bool req_run;  // the request has prompt rows for this path and candidates
};

__device__ __forceinline__ void walk_init(Walk &k, const TcParams &p, int w0) {
    const int units = p.mv.L * p.mv.G;
    k.w = w0;
    k.split = w0 % p.splits;
    k.key = w0 / p.splits;
    const int unit = k.key % units;
    k.b = k.key / units;
    k.l = unit / p.mv.G;
    k.G = unit % p.mv.G;
    k.req.b = -1;
}

__device__ __forceinline__ void walk_next(Walk &k, const TcParams &p) {
    ++k.w;
    if (++k.split == p.splits) {
        k.split = 0;
        ++k.key;
        if (++k.G == p.mv.G) {
            k.G = 0;
            if (++k.l == p.mv.L) {
                k.l = 0;
                ++k.b;
            }
        }
    }
}

__device__ __forceinline__ Item walk_item(Walk &k, const TcParams &p, bool report) {
    if (k.req.b != k.b) {
        k.req = unit_info(p.mv, p.bv, 0, k.b);
        const UnitInfo &u = k.req;
        k.req_run = u.ok && u.n_q > 0 && u.N > 0;
        k.k_tiles = n_key_tiles(u);
        k.tps = (k.k_tiles + p.splits - 1) / p.splits;  // key tiles per split
        k.sbq = (u.n_q + kSub - 1) / kSub;              // sub-blocks per query head
        k.n_sb = p.mv.hpg * k.sbq;
        k.n_qt = (k.n_sb + 1) / 2;  // query tiles of the group
        k.n_chunks = (k.n_qt + p.q_tiles - 1) / p.q_tiles;
    }
    Item it;
    it.u = k.req;
    it.u.l = k.l;
    it.u.G = k.G;
    it.key = k.key;
    it.split = k.split;
    it.k_tiles = k.k_tiles;
    it.tps = k.tps;
    it.sbq = k.sbq;
    it.n_sb = k.n_sb;
    it.n_qt = k.n_qt;
    it.n_chunks = k.n_chunks;
    it.t0 = k.split * k.tps;
    it.t1 = min(k.k_tiles, it.t0 + k.tps);
    it.run = k.req_run && it.t0 < it.t1;
    if (!k.req.ok && report) atomicOr(p.status, FINCH_DEV_BAD_BATCH);
    return it;
}

// MASK: the batch gives every query row a number of candidates it attends to (causal rows); both sweeps then mask
// the (row, key) pairs beyond it.  The unmasked instantiation contains none of that code.
template <int MODE, int D, bool MASK>
__global__ void __launch_bounds__(kTcThreads, 1)
score_tc_kernel(const __grid_constant__ CUtensorMap q_map, const __grid_constant__ CUtensorMap cache_map,
                const __grid_constant__ CUtensorMap chunk_map, TcParams p) {
    constexpr int kSlabs = D / 64;
    constexpr int kTileBytes = kSlabs * kSlabBytes;
    constexpr int kSubBytes = kSub * 128;  // the 64 rows of one sub-block inside one slab
    extern __shared__ uint8_t smem_raw[];
    uint8_t *smem = (uint8_t *)(((uintptr_t)smem_raw + 1023) & ~(uintptr_t)1023);
    uint8_t *q_res = smem;
    uint8_t *k_ring = smem + p.q_tiles * kTileBytes;
    uint8_t *aux = k_ring + p.stages * kTileBytes;
    uint64_t *q_full = (uint64_t *)aux;
    uint64_t *full = q_full + 1;
    uint64_t *empty = full + kMaxStages;
    uint64_t *acc_full = empty + kMaxStages;
    uint64_t *acc_empty = acc_full + kAccBufs;
    uint64_t *stats_ready = acc_empty + kAccBufs;  // all softmax warps have staged their share of the statistics
    uint32_t *tmem_slot = (uint32_t *)(stats_ready + 1);
    volatile int *abort_flag = (volatile int *)(tmem_slot + 1);
    float2 *stats_sm = (float2 *)(aux + 1024);  // [2][q_tiles * 128] row statistics, kColsum only
    int *lim_sm = (int *)(aux + 1024 + kStatsBytes);  // [2][q_tiles * 128] visible candidates per row, masked kColsum

    const ModelView &mv = p.mv;
    const BatchView &bv = p.bv;
    const int64_t rows_total = (int64_t)mv.L * mv.Hq * bv.total_q;

    const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
    if (threadIdx.x == 0) {
        mbar_init(q_full, 1);
        for (int s = 0; s < kMaxStages; ++s) {
            mbar_init(&full[s], 1);
            mbar_init(&empty[s], 1);
        }
        for (int b = 0; b < kAccBufs; ++b) {
            mbar_init(&acc_full[b], 1);
            mbar_init(&acc_empty[b], 4);  // one arrival per softmax warp of the owning group
        }
        mbar_init(stats_ready, 4 * kGroups);
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
    // Barriers and tensor memory are set up; what follows reads what earlier kernels of the stream wrote.  The
    // second sweep's loads and MMAs read only the step's inputs, which were complete before the first sweep began;
    // what its immediate predecessors produce (the merged row statistics) is read by the softmax warps alone, so
    // only they wait, and the tensor pipe already fills the accumulators while the statistics are being merged.
    if (MODE == kLse || warp >= 2) {
        dependency_wait();
        dependents_may_launch();
    }
    // this CTA's contiguous range of work items
    const int w0 = p.bounds ? p.bounds[blockIdx.x] : (int)((int64_t)blockIdx.x * p.n_items / gridDim.x);
    const int w1 = p.bounds ? p.bounds[blockIdx.x + 1] : (int)((int64_t)(blockIdx.x + 1) * p.n_items / gridDim.x);

    // Every role walks the same items and keeps the same running counters (key tiles loaded, query loads,
    // accumulators per group), so barrier phases stay in step across items without any extra handshake.
    if (warp == 0) {
        // =================================================================== TMA producer
        if (lane == 0) {
            prefetch_tensormap(&q_map);
            prefetch_tensormap(&cache_map);
            prefetch_tensormap(&chunk_map);
            int kcnt = 0, qcnt = 0, pst = 0, pph = 0, last_stage = 0, last_ph = 0, prev_stage = 0, prev_ph = 0, q_key = -1;
            bool ok = true;
            Walk wk;
            walk_init(wk, p, w0);
            for (; wk.w < w1 && ok; walk_next(wk, p)) {
                const Item it = walk_item(wk, p, true);
                if (!it.run) continue;
                const UnitInfo &u = it.u;
                for (int c = 0; c < it.n_chunks && ok; ++c) {
                    if (!(it.n_chunks == 1 && q_key == it.key)) {  // the resident query tiles are not this item's
                        // every MMA of the previous work must have read them.  The two groups' streams are issued
                        // in no fixed order, so wait for the release of the last key tile of each (the last two loaded)
                        if (kcnt > 1 && !mbar_wait(&empty[prev_stage], prev_ph, abort_flag)) { ok = false; break; }
                        if (kcnt > 0 && !mbar_wait(&empty[last_stage], last_ph, abort_flag)) { ok = false; break; }
                        const int qt0 = c * p.q_tiles;
                        const int nload = min(2 * min(p.q_tiles, it.n_qt - qt0), it.n_sb - 2 * qt0);
                        mbar_expect_tx(q_full, nload * kSlabs * kSubBytes);
                        for (int sl = 0; sl < nload; ++sl) {
                            const SubBlock sb = sub_block(2 * qt0 + sl, it.sbq, it.n_sb, u.n_q);
                            uint8_t *dst = q_res + (sl / 2) * kTileBytes + (sl % 2) * kSubBytes;
                            for (int s = 0; s < kSlabs; ++s)
                                tma_load_4d(dst + s * kSlabBytes, &q_map, q_full, s * 64, u.q0 + sb.p0,
                                            u.G * mv.hpg + sb.hh, u.l);
                        }
                        ++qcnt;
                        q_key = it.n_chunks == 1 ? it.key : -1;
                    }
                    for (int t = it.t0; t < it.t1; ++t, ++kcnt) {
                        const int stage = pst, ph = pph;
                        if (++pst == p.stages) {
                            pst = 0;
                            pph ^= 1;
                        }
                        if (!mbar_wait_relaxed(&empty[stage], ph ^ 1, abort_flag, 500)) { ok = false; break; }
                        mbar_expect_tx(&full[stage], kTileBytes);
                        const KeyTile kt = key_tile(u, t);
                        const CUtensorMap *m = kt.is_chunk ? &chunk_map : &cache_map;
                        for (int s = 0; s < kSlabs; ++s)
                            tma_load_4d(k_ring + stage * kTileBytes + s * kSlabBytes, m, &full[stage], s * 64, kt.row0,
                                        u.G, u.l);
                        prev_stage = last_stage;
                        prev_ph = last_ph;
                        last_stage = stage;
                        last_ph = ph;
                    }
                }
            }
            // no copy may still be in flight when the CTA retires: wait (bounded) for the last loads issued
            if (qcnt) mbar_wait(q_full, (qcnt - 1) & 1, abort_flag);
            for (int i = max(0, kcnt - p.stages); i < kcnt; ++i)
                mbar_wait(&full[i % p.stages], (i / p.stages) & 1, abort_flag);
        }
    } else if (warp == 1) {
        // =================================================================== MMA issuer
        if (lane == 0) {
            constexpr uint32_t idesc = idesc_bf16_f32(kRows, kRows);
            const uint64_t q_desc = smem_desc_sw128(smem_u32(q_res)), ring_desc = smem_desc_sw128(smem_u32(k_ring));
            // Accumulators are issued in order (item, key tile, query tile); number A lands in buffer A % 4, which
            // belongs to softmax group A % 4.  With equal work per accumulator the groups free their buffers in the
            // same rotation, so in-order issue does not starve anyone.
            bool ok = true;
            int A = 0, qcnt = 0, q_key = -1, st = 0, sph = 0;
            Walk wk;
            walk_init(wk, p, w0);
            for (; wk.w < w1 && ok; walk_next(wk, p)) {
                const Item it = walk_item(wk, p, false);
                if (!it.run) continue;
                for (int c = 0; c < it.n_chunks && ok; ++c) {
                    const int nqt = min(p.q_tiles, it.n_qt - c * p.q_tiles);
                    if (!(it.n_chunks == 1 && q_key == it.key)) {
                        if (!mbar_wait(q_full, qcnt & 1, abort_flag)) { ok = false; break; }
                        ++qcnt;
                        q_key = it.n_chunks == 1 ? it.key : -1;
                    }
                    for (int t = it.t0; t < it.t1 && ok; ++t) {
                        if (!mbar_wait(&full[st], sph, abort_flag)) { ok = false; break; }
                        const uint64_t kd = ring_desc + (uint64_t)((st * kTileBytes) >> 4);
                        for (int qb = 0; qb < nqt; ++qb, ++A) {
                            const int buf = A & 3;
                            if (!mbar_wait(&acc_empty[buf], ((A >> 2) & 1) ^ 1, abort_flag)) { ok = false; break; }
                            tc_fence_after();
                            // one descriptor per operand tile; the K = 16 steps only advance its address field
                            const uint64_t qd = q_desc + (uint64_t)((qb * kTileBytes) >> 4);
                            const uint64_t a_desc = MODE == kLse ? qd : kd, b_desc = MODE == kLse ? kd : qd;
                            const uint32_t d_addr = tmem_base + buf * kRows;
#pragma unroll
                            for (int k = 0; k < D / 16; ++k) {
                                const uint64_t off = (uint64_t)(((k / 4) * kSlabBytes + (k % 4) * 32) >> 4);
                                if (k == 0)
                                    umma_bf16_first(d_addr, a_desc + off, b_desc + off, idesc);
                                else
                                    umma_bf16_acc(d_addr, a_desc + off, b_desc + off, idesc);
                            }
                            umma_commit(&acc_full[buf]);  // the accumulator is ready for its softmax group
                        }
                        if (ok) umma_commit(&empty[st]);  // the stage may be refilled once these MMAs have read it
                        if (++st == p.stages) {
                            st = 0;
                            sph ^= 1;
                        }
                    }
                }
            }
        }
    } else {
        // =================================================================== softmax warps (one TMEM lane per thread)
        const int quarter = warp & 3;            // tcgen05.ld reaches lanes 32 * (warp % 4) ..
        const int sw = warp - 2;                 // softmax warp 0..15
        const int g = sw >> 2;                   // softmax group = the accumulator buffer it owns
        const int my_row = quarter * 32 + lane;  // row of the A tile this thread owns
        const uint32_t t_acc = tmem_base + ((uint32_t)(quarter * 32) << 16) + g * kRows;
        const float scale2 = mv.scale * kLog2e;
        int A = 0, mine = 0, q_key = -1, epoch = 0;  // mine = accumulators this group has consumed (barrier phase)
        bool ok = true;
        Walk wk;
        walk_init(wk, p, w0);
        for (; wk.w < w1 && ok; walk_next(wk, p)) {
            const Item it = walk_item(wk, p, false);
            if (!it.run) continue;
            const UnitInfo &u = it.u;
            const int t0 = it.t0, t1 = it.t1, sbq = it.sbq, n_sb = it.n_sb;
            for (int c = 0; c < it.n_chunks && ok; ++c) {
                const int qt0 = c * p.q_tiles;
                const int nqt = min(p.q_tiles, it.n_qt - qt0);
                const bool new_rows = !(it.n_chunks == 1 && q_key == it.key);
                q_key = it.n_chunks == 1 ? it.key : -1;
                if (MODE == kLse) {
                    float m_raw[kQTiles], z[kQTiles];
                    uint32_t live_mask = 0;  // bit qb: this thread's row of query tile qb holds a prompt row
                    int lim[kQTiles];        // masked variant: candidates that row attends to
#pragma unroll
                    for (int k = 0; k < kQTiles; ++k) {
                        m_raw[k] = -INFINITY;
                        z[k] = 0.f;
                        lim[k] = 0;
                        const SubBlock sb = sub_block(2 * (qt0 + k) + my_row / kSub, sbq, n_sb, u.n_q);
                        if (k < nqt && my_row % kSub < sb.valid) {
                            live_mask |= 1u << k;
                            if (MASK) lim[k] = max(0, min(u.N, bv.row_limit[u.q0 + sb.p0 + my_row % kSub]));
                        }
                    }
                    for (int t = t0; t < t1 && ok; ++t) {
                        const KeyTile kt = key_tile(u, t);
#pragma unroll 1
                        for (int qb = 0; qb < nqt && ok; ++qb, ++A) {
                            if ((A & 3) != g) continue;  // another group's accumulator
                            // a wait's verdict is made warp-uniform so that a timeout takes the whole warp out
                            if (!__all_sync(0xffffffffu, mbar_wait(&acc_full[g], mine & 1, abort_flag))) { ok = false; break; }
                            ++mine;
                            tc_fence_after();
                            float mc = 0.f, zc = 0.f;  // the running statistics of query tile qb (kept in registers)
                            int limc = 0;
#pragma unroll
                            for (int k = 0; k < kQTiles; ++k)
                                if (k == qb) {
                                    mc = m_raw[k];
                                    zc = z[k];
                                    if (MASK) limc = lim[k];
                                }
                            lse_accumulate<MASK>(t_acc, kt.valid, scale2, (live_mask >> qb) & 1u, mc, zc, limc - kt.j0);
#pragma unroll
                            for (int k = 0; k < kQTiles; ++k)
                                if (k == qb) {
                                    m_raw[k] = mc;
                                    z[k] = zc;
                                }
                            tc_fence_before();
                            __syncwarp();
                            if (lane == 0) mbar_arrive(&acc_empty[g]);
                        }
                    }
                    if (ok) {  // every group reports every row of the chunk: (-inf, 0) where it saw no accumulator
#pragma unroll
                        for (int qb = 0; qb < kQTiles; ++qb) {
                            if (qb >= nqt) continue;
                            const SubBlock sb = sub_block(2 * (qt0 + qb) + my_row / kSub, sbq, n_sb, u.n_q);
                            const int r = my_row % kSub;
                            if (r < sb.valid) {
                                const int64_t row =
                                    ((int64_t)u.l * mv.Hq + u.G * mv.hpg + sb.hh) * bv.total_q + u.q0 + sb.p0 + r;
                                p.partial[(it.split * kGroups + g) * rows_total + row] =
                                    make_float2(m_raw[qb] * scale2, z[qb]);
                            }
                        }
                    }
                } else {
                    // The merged statistics of the resident rows are staged once per CTA, every softmax warp its
                    // share, into one of two buffers; a warp that has passed the barrier of epoch e has seen all
                    // warps finish epoch e - 1, so the buffer of epoch e + 1 (= that of e - 1) is free by then.
                    if (new_rows) {
                        float2 *dst = stats_sm + (epoch & 1) * kQTiles * kRows;
                        for (int idx = sw * 32 + lane; idx < nqt * kRows; idx += 16 * 32) {
                            const int r = idx % kRows;
                            const SubBlock sb = sub_block(2 * (qt0 + idx / kRows) + r / kSub, sbq, n_sb, u.n_q);
                            float2 out = make_float2(0.f, 0.f);
                            if (r % kSub < sb.valid)
                                out = p.merged[((int64_t)u.l * mv.Hq + u.G * mv.hpg + sb.hh) * bv.total_q + u.q0 + sb.p0 +
                                               r % kSub];
                            // rows 2k and 2k+1 share one float4: (-ref_2k, -ref_2k+1, w_2k, w_2k+1)
                            float *smf = (float *)dst + (idx >> 1) * 4 + (idx & 1);
                            smf[0] = out.x;
                            smf[2] = out.y;
                            if (MASK)
                                lim_sm[(epoch & 1) * kQTiles * kRows + idx] =
                                    r % kSub < sb.valid ? max(0, min(u.N, bv.row_limit[u.q0 + sb.p0 + r % kSub])) : 0;
                        }
                        __syncwarp();
                        if (lane == 0) mbar_arrive(stats_ready);
                        if (!__all_sync(0xffffffffu, mbar_wait(stats_ready, epoch & 1, abort_flag))) { ok = false; break; }
                        ++epoch;
                    }
                    const float2 *sm = stats_sm + ((epoch - 1) & 1) * kQTiles * kRows;
                    float *part = p.score_parts + ((int64_t)g * mv.L * mv.G + (int64_t)u.l * mv.G + u.G) *
                                                      ((int64_t)bv.total_cache + bv.total_chunk) +
                                  u.cache0 + u.chunk0;
                    for (int t = t0; t < t1 && ok; ++t) {
                        const KeyTile kt = key_tile(u, t);
                        float c0 = 0.f, c1 = 0.f;
#pragma unroll 1
                        for (int qb = 0; qb < nqt && ok; ++qb, ++A) {
                            if ((A & 3) != g) continue;
                            if (!__all_sync(0xffffffffu, mbar_wait(&acc_full[g], mine & 1, abort_flag))) { ok = false; break; }
                            ++mine;
                            tc_fence_after();
                            const int v0 = sub_block(2 * (qt0 + qb), sbq, n_sb, u.n_q).valid;
                            const int v1 = sub_block(2 * (qt0 + qb) + 1, sbq, n_sb, u.n_q).valid;
                            colsum_accumulate<MASK>(t_acc, v0, v1, scale2, sm + qb * kRows, c0, c1,
                                                    lim_sm + ((epoch - 1) & 1) * kQTiles * kRows + qb * kRows,
                                                    kt.j0 + my_row);
                            tc_fence_before();
                            __syncwarp();
                            if (lane == 0) mbar_arrive(&acc_empty[g]);
                        }
                        if (ok && my_row < kt.valid) {  // this group's share of the key's score (0 if it had none)
                            float *dst = part + kt.j0 + my_row;
                            const float col = c0 + c1;
                            *dst = c == 0 ? col : *dst + col;  // later query chunks add to the first chunk's sums
                        }
                    }
                }
            }
        }
    }

    // ---- common epilogue: everyone meets here, also after a timed-out wait.  The role warps ran one lane only:
    // bring each warp back together first, the CTA barrier must be executed by whole warps.
    __syncwarp();
    tc_fence_before();
    __syncthreads();
    if (threadIdx.x == 0 && *abort_flag) atomicOr(p.status, FINCH_DEV_TIMEOUT);
    if (warp == 1) {
        __syncwarp();
        tc_fence_after();
        tmem_dealloc(tmem_base, 512);
    }
}

// With several requests in the batch the items differ in size (accumulators = key tiles x query tiles of their
// request), so equal item counts per CTA would leave the grid waiting for the CTAs that drew the long prompts and
// large caches.  This one-block kernel sums the work per request (items are ordered request-major, and all items
// of a request cost about the same), then gives every CTA of the persistent grid a contiguous item range of about
// equal work: bounds[i] = the item at which the running work passes i / n_ctas of the total.
__global__ void __launch_bounds__(1024)
plan_items_kernel(TcParams p, int *bounds, int n_ctas) {
    __shared__ unsigned long long warp_sum[32];
    __shared__ unsigned long long carry_s;
    const ModelView &mv = p.mv;
    const BatchView &bv = p.bv;
    const int tid = threadIdx.x, lane = tid & 31, wid = tid >> 5;
    dependency_wait();
    dependents_may_launch();
    const unsigned long long ipr = (unsigned long long)mv.L * mv.G * p.splits;  // items per request
    if (tid == 0) {
        carry_s = 0;
        p.work_prefix[0] = 0;
    }
    __syncthreads();
    for (int base = 0; base < bv.batch; base += 1024) {
        const int b = base + tid;
        unsigned long long cost = 0;
        if (b < bv.batch) {
            const UnitInfo u = unit_info(mv, bv, 0, b);
            if (u.ok && u.n_q > 0 && u.N > 0) {
                const int sb = mv.hpg * ((u.n_q + kSub - 1) / kSub);
                // key tiles of one split x query tiles, plus a little for the item's fixed costs
                cost = ipr * (unsigned long long)((n_key_tiles(u) + p.splits - 1) / p.splits * ((sb + 1) / 2) + 2);
            }
        }
        unsigned long long incl = cost;
#pragma unroll
        for (int d = 1; d < 32; d <<= 1) {
            const unsigned long long up = __shfl_up_sync(0xffffffffu, incl, d);
            if (lane >= d) incl += up;
        }
        if (lane == 31) warp_sum[wid] = incl;
        __syncthreads();
        unsigned long long before = carry_s;
        for (int w = 0; w < wid; ++w) before += warp_sum[w];
        if (b < bv.batch) p.work_prefix[b + 1] = before + incl;
        __syncthreads();
        if (tid == 1023) carry_s = before + incl;
        __syncthreads();
    }
    const unsigned long long total = carry_s;
    for (int i = tid; i <= n_ctas; i += 1024) {
        int item;
        if (i == 0) {
            item = 0;
        } else if (i == n_ctas || total == 0) {
            item = p.n_items;
        } else {
            const unsigned long long target = total / n_ctas * i + total % n_ctas * i / n_ctas;
            int lo = 0, hi = bv.batch - 1;  // the last request whose prefix is <= target
            while (lo < hi) {
                const int mid = (lo + hi + 1) >> 1;
                if (p.work_prefix[mid] <= target) lo = mid; else hi = mid - 1;
            }
            const unsigned long long span = p.work_prefix[lo + 1] - p.work_prefix[lo];
            const unsigned long long into = span ? (target - p.work_prefix[lo]) * ipr / span : 0;
            item = (int)((unsigned long long)lo * ipr + (into < ipr ? into : ipr));
        }
        bounds[i] = item;
    }
}

// Merge the per-split, per-group partial statistics of every prompt row (fixed order) into the pair the column pass
// uses: weights are exp2(s2 - R) * w with R = M + floor(log2 Z) and w = 2^floor(log2 Z) / Z in (1/2, 1], so the
// exponent never exceeds a few units whatever reference the parts were summed against.
__global__ void __launch_bounds__(128)
merge_stats_kernel(TcParams p) {
    const ModelView &mv = p.mv;
    const BatchView &bv = p.bv;
    dependents_may_launch();  // before the wait: the second sweep's CTAs may take over SMs as the first sweep's retire
    dependency_wait();
    const int h = blockIdx.y % mv.Hq, l = blockIdx.y / mv.Hq;
    const UnitInfo u = unit_info(mv, bv, l * mv.G + h / mv.hpg, blockIdx.z);
    if (!u.ok || u.n_q == 0 || u.N == 0) return;
    const int pr = blockIdx.x * 128 + threadIdx.x;
    if (pr >= u.n_q) return;
    const int k_tiles = n_key_tiles(u);
    const int tps = (k_tiles + p.splits - 1) / p.splits;
    const int64_t rows_total = (int64_t)mv.L * mv.Hq * bv.total_q;
    const int64_t row = ((int64_t)l * mv.Hq + h) * bv.total_q + u.q0 + pr;
    float M = -INFINITY, Z = 0.f;
    const int n_parts = ((k_tiles + tps - 1) / tps) * kGroups;  // splits that hold key tiles x softmax groups
    // all loads first (they are independent), eight at a time, then the merge in part order
#pragma unroll 1
    for (int i0 = 0; i0 < n_parts; i0 += 8) {
        float2 part[8];
#pragma unroll
        for (int i = 0; i < 8; ++i)
            part[i] = i0 + i < n_parts ? p.partial[(int64_t)(i0 + i) * rows_total + row] : make_float2(0.f, 0.f);
#pragma unroll
        for (int i = 0; i < 8; ++i) merge_part(part[i], M, Z);
    }
    if (bv.self_lse) merge_self_term(bv.self_lse[row], M, Z);  // the keys the row attends to besides the candidates
    float lse_nat;
    float2 out = merged_pair(M, Z, lse_nat);
    if (bv.row_limit && bv.row_norm)  // per-row normalisation: times the fraction of the candidates the row sees
        out.y *= (float)max(0, min(u.N, bv.row_limit[u.q0 + pr])) / (float)u.N;
    p.merged[row] = out;
    if (p.row_lse) p.row_lse[row] = lse_nat;
}

// scores = the partial column sums of the selection group's KV heads (one scoring unit each), four per head, added in
// a fixed order: heads ascending, softmax groups ascending.  A request without prompt rows has no accumulators and
// no partial sums: its scores are the empty sum, zero.
constexpr int kCombinePerThread = 4;

__global__ void __launch_bounds__(256)
combine_scores_kernel(TcParams p) {
    const ModelView &mv = p.mv;
    const BatchView &bv = p.bv;
    dependency_wait();  // many waves of small CTAs: the next kernel's CTAs must not take their slots early
    const int l = blockIdx.y / p.out_groups, og = blockIdx.y % p.out_groups;
    const UnitInfo u = unit_info(mv, bv, l * mv.G + og * p.units_per_group, blockIdx.z);
    if (!u.ok) return;
    const int64_t cand = (int64_t)bv.total_cache + bv.total_chunk;
    const int64_t gstride = (int64_t)mv.L * mv.G * cand;
    // four keys per thread, 256 apart: every load is coalesced and a thread has up to 16 of them in flight
    float s[kCombinePerThread];
    int64_t within[kCombinePerThread];
#pragma unroll
    for (int i = 0; i < kCombinePerThread; ++i) {
        const int j = (blockIdx.x * kCombinePerThread + i) * 256 + threadIdx.x;
        within[i] = j < u.N ? (int64_t)u.cache0 + u.chunk0 + j : -1;
        s[i] = 0.f;
    }
    if (u.n_q > 0) {
        for (int k = 0; k < p.units_per_group; ++k) {
            const int64_t base = ((int64_t)l * mv.G + og * p.units_per_group + k) * cand;
#pragma unroll
            for (int g = 0; g < kGroups; ++g)
#pragma unroll
                for (int i = 0; i < kCombinePerThread; ++i)
                    if (within[i] >= 0) s[i] += p.score_parts[g * gstride + base + within[i]];
        }
    }
#pragma unroll
    for (int i = 0; i < kCombinePerThread; ++i)
        if (within[i] >= 0) p.scores[((int64_t)l * p.out_groups + og) * cand + within[i]] = s[i];
}

// ------------------------------------------------------------------------------------------------ host side

// Key splits per unit: the smallest count (at most max_splits, at least one key tile each) whose grid fills whole
// waves of SMs best.
int choose_splits(int ctas_per_split, int key_tiles, int sm_count, int max_splits) {
    int best = 1;
    double best_eff = 0.0;
    for (int s = 1; s <= max_splits && s <= key_tiles; ++s) {
        const double waves = (double)ctas_per_split * s / sm_count;
        const double eff = waves / (double)((long long)waves + (waves > (long long)waves ? 1 : 0));
        if (eff > best_eff * 1.05) {
            best_eff = eff;
            best = s;
        }
    }
    return best;
}

template <int D, bool MASK>
cudaError_t launch_d(const Ctx &ctx, const CUtensorMap &qm, const CUtensorMap &cm, const CUtensorMap &hm, TcParams p,
                     cudaStream_t stream) {
    constexpr int kTileBytes = (D / 64) * kSlabBytes;
    const ModelView &mv = p.mv;  // the scoring view
    const BatchView &bv = p.bv;
    const int sub_blocks = mv.hpg * ((bv.max_q + kSub - 1) / kSub);
    p.q_tiles = min(kQTiles, (sub_blocks + 1) / 2);
    p.stages = min(kMaxStages, (kSmemLimit - 1024 - kAuxBytes - p.q_tiles * kTileBytes) / kTileBytes);
    if (p.stages < 2) return cudaErrorNotSupported;
    const int smem = 1024 + (p.q_tiles + p.stages) * kTileBytes + kAuxBytes;
    cudaError_t e = cudaFuncSetAttribute(score_tc_kernel<kLse, D, MASK>, cudaFuncAttributeMaxDynamicSharedMemorySize, smem);
    if (e != cudaSuccess) return e;
    e = cudaFuncSetAttribute(score_tc_kernel<kColsum, D, MASK>, cudaFuncAttributeMaxDynamicSharedMemorySize, smem);
    if (e != cudaSuccess) return e;
    p.n_items = p.splits * mv.L * mv.G * bv.batch;
    const int sms = ctx.sm_count > 0 ? ctx.sm_count : 148;
    dim3 grid(p.n_items < sms ? p.n_items : sms);  // persistent: one CTA per SM walks a contiguous range of items
    if (bv.batch > 1 && (int)grid.x < kPlanBoundsInts) {  // requests of different sizes: ranges of equal work
        int *bounds = (int *)(p.work_prefix + bv.batch + 1);
        e = launch_chained(plan_items_kernel, dim3(1), dim3(1024), 0, stream, p, bounds, (int)grid.x);
        if (e != cudaSuccess) return e;
        p.bounds = bounds;
        ctx.launches += 1;
    }
    e = launch_chained(score_tc_kernel<kLse, D, MASK>, grid, dim3(kTcThreads), smem, stream, qm, cm, hm, p);
    if (e != cudaSuccess) return e;
    dim3 mgrid((bv.max_q + 127) / 128, mv.L * mv.Hq, bv.batch);
    e = launch_chained(merge_stats_kernel, mgrid, dim3(128), 0, stream, p);
    if (e != cudaSuccess) return e;
    e = launch_chained(score_tc_kernel<kColsum, D, MASK>, grid, dim3(kTcThreads), smem, stream, qm, cm, hm, p);
    if (e != cudaSuccess) return e;
    dim3 cgrid((bv.max_cache + bv.max_chunk + 256 * kCombinePerThread - 1) / (256 * kCombinePerThread), mv.L * p.out_groups,
               bv.batch);
    ctx.launches += 4;
    return launch_chained(combine_scores_kernel, cgrid, dim3(256), 0, stream, p);
}

}  // namespace

bool score_tc_supported(const Ctx &ctx) {
    return ctx.cfg.dtype == FINCH_BF16 && (ctx.model.d == 64 || ctx.model.d == 128);
}

// The least scratch (float2 entries) the two-launch tensor-core path needs for this batch: one key split.
size_t score_tc_scratch_min(const Ctx &ctx, const BatchView &bv) {
    const ModelView &mv = ctx.model;
    const size_t rows = (size_t)mv.L * mv.Hq * (size_t)bv.total_q;
    const size_t cand = (size_t)mv.L * mv.Hkv * ((size_t)bv.total_cache + bv.total_chunk);
    return rows * (kGroups + 1) + (kGroups * cand + 1) / 2 + (size_t)bv.batch + 1 + kPlanBoundsInts / 2;
}

// `partial` holds partial_capacity float2 entries; the key-split count is limited so that one entry per prompt
// row, split and softmax group, one merged entry per row and the per-group partial scores fit.  Returns cudaErrorNotSupported (and launches nothing) when the tensors cannot be described
// to the TMA unit; the caller then uses the warp-level path for every request.
cudaError_t launch_score_tc(const Ctx &ctx, const TensorView &q, const TensorView &cache_k, const TensorView &chunk_k,
                            const BatchView &bv, float *scores, float2 *partial, size_t partial_capacity,
                            float *row_lse, cudaStream_t stream) {
    // Scoring works per KV head whatever the selection groups are: a query head only ever meets its own KV head's
    // keys.  With one selection group per layer the heads' column sums are added when the parts are combined.
    ModelView mv = ctx.model;
    mv.G = mv.Hkv;
    mv.hpg = mv.g;
    mv.kvpg = 1;
    if (mv.L * mv.G == 0 || bv.batch == 0 || bv.max_q == 0 || bv.max_cache + bv.max_chunk == 0) return cudaSuccess;
    const size_t rows = (size_t)mv.L * mv.Hq * (size_t)bv.total_q;
    // scratch layout (float2 units): per-split, per-group row statistics | merged row statistics | item plan |
    // per-group scores
    const size_t cand = (size_t)mv.L * mv.G * ((size_t)bv.total_cache + bv.total_chunk);
    const size_t parts_f2 = (kGroups * cand + 1) / 2;
    const size_t plan_f2 = (size_t)bv.batch + 1 + kPlanBoundsInts / 2;  // 64-bit work prefix, then the CTA bounds
    if (rows == 0 || partial_capacity < rows * (kGroups + 1) + parts_f2 + plan_f2) return cudaErrorNotSupported;
    CUtensorMap qm, cm, hm;
    if (!make_map(&qm, q, mv.d, bv.total_q, mv.Hq, mv.L, kSub)) return cudaErrorNotSupported;
    const bool have_cache = bv.max_cache > 0, have_chunk = bv.max_chunk > 0;
    if (have_cache && !make_map(&cm, cache_k, mv.d, bv.total_cache, mv.Hkv, mv.L, kRows)) return cudaErrorNotSupported;
    if (have_chunk && !make_map(&hm, chunk_k, mv.d, bv.total_chunk, mv.Hkv, mv.L, kRows)) return cudaErrorNotSupported;
    if (!have_cache) cm = hm;  // never dereferenced: no request has cache tiles
    if (!have_chunk) hm = cm;
    const int key_tiles = (bv.max_cache + kRows - 1) / kRows + (bv.max_chunk + kRows - 1) / kRows;
    const int max_splits =
        (int)min((size_t)kScoreMaxSplits, ((partial_capacity - parts_f2 - plan_f2) / rows - 1) / kGroups);
    TcParams p{mv, bv, partial, nullptr, row_lse, scores, nullptr, ctx.d_status, 1, 2, 1, 0, nullptr, nullptr,
               ctx.model.G, ctx.model.kvpg};
    p.splits = choose_splits(mv.L * mv.G * bv.batch, key_tiles, ctx.sm_count > 0 ? ctx.sm_count : 148, max_splits);
    p.merged = partial + (size_t)p.splits * kGroups * rows;
    p.work_prefix = (unsigned long long *)(p.merged + rows);
    p.score_parts = (float *)(p.merged + rows + plan_f2);
    if (bv.row_limit)  // causal query rows: the masked instantiation
        return mv.d == 64 ? launch_d<64, true>(ctx, qm, cm, hm, p, stream) : launch_d<128, true>(ctx, qm, cm, hm, p, stream);
    return mv.d == 64 ? launch_d<64, false>(ctx, qm, cm, hm, p, stream) : launch_d<128, false>(ctx, qm, cm, hm, p, stream);
}

}  // namespace finch

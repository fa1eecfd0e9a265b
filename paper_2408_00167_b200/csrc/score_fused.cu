// Prompt-guided scoring with both sweeps in ONE persistent kernel (single-request batches, bf16, head_dim 64/128,
// up to four 128-row query tiles per KV head, no per-row mask).
//
// The logits S = Q K^T of a unit (layer, KV head) are visited twice -- the row log-sum-exp must be known before any
// column sum can be formed -- but here the second visit follows the first closely enough that the keys come back
// from L2 instead of HBM, and nothing but a few bytes per prompt row leaves the SM in between:
//
//   * The key tiles of all units form one sequence (unit-major).  It is cut into ranges of W tiles; CTA i of the
//     persistent grid takes ranges i, i + P, i + 2P, ... (one "window" each), so the CTAs of a window work on
//     neighbouring tiles and the keys in flight between the two sweeps of a window are P x W tiles (tens of MB).
//   * Phase A of a window: D = Qtile x Ktile^T (one prompt row per TMEM lane), every softmax thread keeps the
//     (reference, sum exp2) of its rows over the window's tiles, publishes them to a small global array and bumps
//     the unit's ticket.  Nobody waits in phase A.
//   * Phase B: wait (bounded) until the ticket shows that every range of the unit has published -- the other
//     ranges belong to neighbouring CTAs that run phase A of the same window at the same time -- merge the parts
//     in a fixed order into (-R, w) per row, stage them in shared memory, then D = Ktile x Qtile^T (one key per
//     lane) and each thread sums exp2(s - R_r) w_r over the prompt rows: the column sums of its key.  The four
//     softmax groups see different query tiles; their partial sums meet through a per-group array and are added
//     in group order at the end of the range, by the same CTA.
//   * With `delay` = 1 a CTA runs phase A of window k + 1 before phase B of window k, so the tickets it waits for
//     are long complete.
//
// Roles and barriers are those of the two-launch kernels (score_tc.cu): TMA producer lane, MMA issuer lane, four
// softmax groups of four warps, accumulators dealt round-robin to the groups, every wait bounded.
#include "score_tc_common.cuh"

namespace finch {
namespace {

using namespace ptx;
using namespace tc;

// barriers, then the row statistics: 2 buffers x `tiles` query tiles
constexpr int fused_aux_bytes(int tiles) { return 1024 + 2 * tiles * kRows * 8; }
constexpr int kSoftmaxWarps = kGroups * 4;
// Waiters with time to spare poll rarely (their tests share the SM's memory-instruction queue with the softmax
// warps' special-function instructions): the producer is a ring ahead of the MMAs, the helpers a window ahead of
// anyone who needs what they publish.
constexpr uint32_t kProducerSleepNs = 500;
constexpr uint32_t kHelperSleepNs = 1000;
constexpr int kHelpers = 64;  // two helper warps: the exchange of row statistics and the sum over the groups
constexpr int kFusedThreads = kTcThreads + kHelpers;
constexpr int kMaxSegs = 8;  // ranges that may overlap one unit (bounds the partial-statistics array)

struct FusedParams {
    ModelView mv;  // the scoring view: one unit per KV head
    BatchView bv;
    float2 *partial;     // [units][seg_max][kGroups][rows_u] (reference base-2 logit, sum exp2) per row and part
    int *tickets;        // [units] ranges of the unit whose phase-A statistics are published
    float *row_lse;      // nullable
    float *unit_scores;  // [L][Hkv][cand]: the column sums of one KV head's query heads
    float *score_parts;  // [kGroups][L][Hkv][cand] per-group partial column sums
    int *status;
    int W;        // key tiles per range
    int seg_max;  // slots per unit in `partial`
    int rows_u;   // rows per unit in `partial` (query heads per KV head x longest prompt)
    int stages;   // key-tile ring depth
    int q_tiles;  // resident query tiles (= query tiles of a unit, at most kQTiles)
    int delay;    // 0: phase B of a window right after its phase A; 1: one window later
};

__device__ __forceinline__ int ld_acquire_gpu(const int *p) {
    int v;
    asm volatile("ld.acquire.gpu.global.s32 %0, [%1];" : "=r"(v) : "l"(p) : "memory");
    return v;
}

// Bounded wait for a global counter to reach `target` (about a second); gives up as soon as another thread of the
// CTA has, and then raises *abort_flag like the mbarrier waits.
constexpr uint32_t kTicketSpins = 1u << 21;
__device__ __forceinline__ bool ticket_wait(const int *ticket, int target, volatile int *abort_flag) {
    for (uint32_t it = 0; it < kTicketSpins; ++it) {
        if (ld_acquire_gpu(ticket) >= target) return true;
        if (*abort_flag) return false;
        __nanosleep(it < 256 ? 40 : 400);
    }
    *abort_flag = 1;
    return false;
}

// A counter in shared memory that some warps bump (after their writes) and another polls (before its reads).
__device__ __forceinline__ void count_arrive(int *counter) {
    __threadfence_block();
    atomicAdd_block(counter, 1);
}
__device__ __forceinline__ bool count_wait(int *counter, int target, volatile int *abort_flag) {
    for (uint32_t it = 0; it < kTicketSpins; ++it) {
        if (*(volatile int *)counter >= target) {
            __threadfence_block();
            return true;
        }
        if (*abort_flag) return false;
        __nanosleep(kHelperSleepNs);
    }
    *abort_flag = 1;
    return false;
}

// What is the same for every unit of a single-request batch.
struct Geo {
    UnitInfo u;  // l and G are filled in per segment
    bool run;
    int T;       // key tiles per unit
    int sbq, n_sb, n_qt;
    int total;   // key tiles of all units
    int n_win;   // windows of this CTA
};

// The part of one range that lies in one unit.
struct Seg {
    int unit, t0, t1;
    int slot, n_seg;  // this range's position among the ranges that overlap the unit, and their number
};

__device__ __forceinline__ bool next_seg(const Geo &g, int W, int rho, int &x, int x1, Seg &s) {
    if (x >= x1) return false;
    s.unit = x / g.T;
    s.t0 = x - s.unit * g.T;
    s.t1 = min(g.T, s.t0 + (x1 - x));
    const int first = (s.unit * g.T) / W, last = ((s.unit + 1) * g.T - 1) / W;
    s.slot = rho - first;
    s.n_seg = last - first + 1;
    x += s.t1 - s.t0;
    return true;
}

template <int D>
__global__ void __launch_bounds__(kFusedThreads, 1)
score_fused_kernel(const __grid_constant__ CUtensorMap q_map, const __grid_constant__ CUtensorMap cache_map,
                   const __grid_constant__ CUtensorMap chunk_map, FusedParams p) {
    constexpr int kSlabs = D / 64;
    constexpr int kTileBytes = kSlabs * kSlabBytes;
    constexpr int kSubBytes = kSub * 128;
    extern __shared__ uint8_t smem_raw[];
    uint8_t *smem = (uint8_t *)(((uintptr_t)smem_raw + 1023) & ~(uintptr_t)1023);
    uint8_t *q_res = smem;
    uint8_t *k_ring = smem + p.q_tiles * kTileBytes;
    uint8_t *aux = k_ring + p.stages * kTileBytes;
    uint64_t *q_full = (uint64_t *)aux;    // [kQTiles] a query tile of the segment's unit has landed
    uint64_t *q_free = q_full + kQTiles;   // [kQTiles] the segment's MMAs are through with a query tile
    uint64_t *full = q_free + kQTiles;
    uint64_t *empty = full + kMaxStages;
    uint64_t *acc_full = empty + kMaxStages;
    uint64_t *acc_empty = acc_full + kAccBufs;
    uint64_t *stats_ready = acc_empty + kAccBufs;  // [2] the helper warps have staged a segment's row statistics
    uint32_t *tmem_slot = (uint32_t *)(stats_ready + 2);
    volatile int *abort_flag = (volatile int *)(tmem_slot + 1);
    // Softmax warps -> helpers: plain counters (one count per warp and segment), not barrier phases, so that a helper
    // that falls behind by more than one segment still reads the right answer.
    int *a_count = (int *)(tmem_slot + 2);  // softmax warps that have written a phase-A segment's statistics
    int *b_count = a_count + 1;             // softmax warps that are through a phase-B segment
    float2 *stats_sm = (float2 *)(aux + 1024);  // [2][q_tiles * 128] row statistics of phase B, two segments in turn

    const ModelView &mv = p.mv;
    const BatchView &bv = p.bv;
    const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
    if (threadIdx.x == 0) {
        for (int b = 0; b < kQTiles; ++b) {
            mbar_init(&q_full[b], 1);
            mbar_init(&q_free[b], 1);
        }
        for (int s = 0; s < kMaxStages; ++s) {
            mbar_init(&full[s], 1);
            mbar_init(&empty[s], 1);
        }
        for (int b = 0; b < kAccBufs; ++b) {
            mbar_init(&acc_full[b], 1);
            mbar_init(&acc_empty[b], 4);  // one arrival per softmax warp of the owning group
        }
        for (int b = 0; b < 2; ++b) mbar_init(&stats_ready[b], kHelpers / 32);  // one arrival per helper warp
        *a_count = 0;
        *b_count = 0;
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
    // The tickets were cleared, and the inputs written, by what precedes this kernel.  The successor is NOT allowed
    // to launch early: its CTAs would take over the SMs of the CTAs that finish first and park there in their wait
    // (measured: + 20 us on the 0.5 ms step of 32 layers x 8 KV heads x 4096 candidates).
    dependency_wait();

    Geo g;
    g.u = unit_info(mv, bv, 0, 0);
    g.T = n_key_tiles(g.u);
    g.sbq = (g.u.n_q + kSub - 1) / kSub;
    g.n_sb = mv.hpg * g.sbq;
    g.n_qt = (g.n_sb + 1) / 2;
    g.run = g.u.ok && g.u.n_q > 0 && g.u.N > 0 && g.n_qt <= p.q_tiles;
    g.total = mv.L * mv.G * g.T;
    const int n_ranges = (g.total + p.W - 1) / p.W;
    g.n_win = g.run && (int)blockIdx.x < n_ranges ? (n_ranges - (int)blockIdx.x + (int)gridDim.x - 1) / (int)gridDim.x : 0;
    if (!g.u.ok && threadIdx.x == 0 && blockIdx.x == 0) atomicOr(p.status, FINCH_DEV_BAD_BATCH);
    const int n_steps = g.n_win ? g.n_win + p.delay : 0;

    // Every role walks the same sequence of (phase, range, segment) and keeps the same running counters (key
    // tiles loaded, query loads, accumulators), so barrier phases stay in step without any extra handshake.
#define FINCH_FOR_EACH_SEGMENT(...)                                                           \
    for (int step = 0; step < n_steps && ok; ++step)                                          \
        for (int ph = 0; ph < 2 && ok; ++ph) {                                                \
            const int win = ph == 0 ? step : step - p.delay;                                  \
            if (win < 0 || win >= g.n_win) continue;                                          \
            const int rho = win * (int)gridDim.x + (int)blockIdx.x;                           \
            int x = rho * p.W;                                                                \
            const int x1 = min(g.total, x + p.W);                                             \
            Seg sg;                                                                           \
            while (ok && next_seg(g, p.W, rho, x, x1, sg)) {                                  \
                UnitInfo u = g.u;                                                             \
                u.l = sg.unit / mv.G;                                                         \
                u.G = sg.unit % mv.G;                                                         \
                __VA_ARGS__                                                                   \
            }                                                                                 \
        }

    if (warp == 0) {
        // =================================================================== TMA producer
        if (lane == 0) {
            prefetch_tensormap(&q_map);
            prefetch_tensormap(&cache_map);
            prefetch_tensormap(&chunk_map);
            int kcnt = 0, qcnt = 0, nseg = 0, pst = 0, pph = 0, q_unit = -1;
            bool ok = true;
            auto load_key_tile = [&](const UnitInfo &u, int t) {
                const int stage = pst, sph = pph;
                if (++pst == p.stages) {
                    pst = 0;
                    pph ^= 1;
                }
                if (!mbar_wait_relaxed(&empty[stage], sph ^ 1, abort_flag, kProducerSleepNs)) {
                    ok = false;
                    return;
                }
                mbar_expect_tx(&full[stage], kTileBytes);
                const KeyTile kt = key_tile(u, t);
                const CUtensorMap *m = kt.is_chunk ? &chunk_map : &cache_map;
                for (int s = 0; s < kSlabs; ++s)
                    tma_load_4d(k_ring + stage * kTileBytes + s * kSlabBytes, m, &full[stage], s * 64, kt.row0, u.G, u.l);
                ++kcnt;
            };
            FINCH_FOR_EACH_SEGMENT({
                // the segment's first key tile goes first: its ring stage is free before the query tiles are
                load_key_tile(u, sg.t0);
                if (!ok) break;
                if (q_unit != sg.unit) {
                    // Another unit's query tiles, one tile at a time: tile qb may be overwritten once the previous
                    // segment's last MMAs on it are complete (its q_free phase), while the MMAs on the tiles behind it
                    // still run -- the reload hides behind the tail of the old segment instead of following it.
                    for (int qb = 0; qb < g.n_qt; ++qb) {
                        if (nseg > 0 && !mbar_wait(&q_free[qb], (nseg - 1) & 1, abort_flag)) { ok = false; break; }
                        const int nsb = min(2, g.n_sb - 2 * qb);
                        mbar_expect_tx(&q_full[qb], nsb * kSlabs * kSubBytes);
                        for (int sl = 2 * qb; sl < 2 * qb + nsb; ++sl) {
                            const SubBlock sb = sub_block(sl, g.sbq, g.n_sb, u.n_q);
                            uint8_t *dst = q_res + (sl / 2) * kTileBytes + (sl % 2) * kSubBytes;
                            for (int s = 0; s < kSlabs; ++s)
                                tma_load_4d(dst + s * kSlabBytes, &q_map, &q_full[qb], s * 64, u.q0 + sb.p0,
                                            u.G * mv.hpg + sb.hh, u.l);
                        }
                    }
                    if (!ok) break;
                    ++qcnt;
                    q_unit = sg.unit;
                }
                ++nseg;
                for (int t = sg.t0 + 1; t < sg.t1 && ok; ++t) load_key_tile(u, t);
            })
            // no copy may still be in flight when the CTA retires: wait (bounded) for the last loads issued
            for (int qb = 0; qcnt && qb < g.n_qt; ++qb) mbar_wait(&q_full[qb], (qcnt - 1) & 1, abort_flag);
            for (int i = max(0, kcnt - p.stages); i < kcnt; ++i)
                mbar_wait(&full[i % p.stages], (i / p.stages) & 1, abort_flag);
        }
    } else if (warp == 1) {
        // =================================================================== MMA issuer
        if (lane == 0) {
            constexpr uint32_t idesc = idesc_bf16_f32(kRows, kRows);
            const uint64_t q_desc = smem_desc_sw128(smem_u32(q_res)), ring_desc = smem_desc_sw128(smem_u32(k_ring));
            const uint32_t desc_hi = (uint32_t)(q_desc >> 32), q_lo = (uint32_t)q_desc, ring_lo = (uint32_t)ring_desc;
            bool ok = true;
            int A = 0, qcnt = 0, q_unit = -1, st = 0, sph = 0;
            FINCH_FOR_EACH_SEGMENT({
                const bool reloaded = q_unit != sg.unit;  // the producer has brought this unit's query tiles
                q_unit = sg.unit;
                // This thread is the kernel's pacemaker (it is held while its MMAs run and every barrier test costs
                // it some 200 cycles), so its loop carries as little as possible: descriptor bases and strides are
                // set per segment -- phase A: A operand = query tile qb, B = the key tile; phase B the other way
                // round -- and the MMAs' operands differ in their low words only (the 14-bit address field cannot
                // carry: shared memory ends below 2^18 bytes).
                const uint32_t q_step = (uint32_t)(kTileBytes >> 4), k_step = (uint32_t)(kTileBytes >> 4);
                const uint32_t a_q = ph == 0 ? q_step : 0u, a_k = ph == 0 ? 0u : k_step;  // strides of the A operand
                const uint32_t b_q = ph == 0 ? 0u : q_step, b_k = ph == 0 ? k_step : 0u;  // and of the B operand
                const uint32_t a_lo0 = ph == 0 ? q_lo : ring_lo, b_lo0 = ph == 0 ? ring_lo : q_lo;
                const bool wait_q = reloaded;
                for (int t = sg.t0; t < sg.t1 && ok; ++t) {
                    if (!mbar_wait(&full[st], sph, abort_flag)) { ok = false; break; }
                    const bool first = wait_q && t == sg.t0, last = t == sg.t1 - 1;
                    for (int qb = 0; qb < g.n_qt; ++qb, ++A) {
                        const int buf = A & 3;
                        if (!mbar_wait(&acc_empty[buf], ((A >> 2) & 1) ^ 1, abort_flag)) { ok = false; break; }
                        if (first && !mbar_wait(&q_full[qb], qcnt & 1, abort_flag)) { ok = false; break; }
                        tc_fence_after();
                        const uint32_t a_lo = a_lo0 + (uint32_t)qb * a_q + (uint32_t)st * a_k;
                        const uint32_t b_lo = b_lo0 + (uint32_t)qb * b_q + (uint32_t)st * b_k;
                        const uint32_t d_addr = tmem_base + buf * kRows;
#pragma unroll
                        for (int k = 0; k < D / 16; ++k) {
                            const uint32_t off = (uint32_t)(((k / 4) * kSlabBytes + (k % 4) * 32) >> 4);
                            const uint64_t a_desc = ((uint64_t)desc_hi << 32) | (a_lo + off);
                            const uint64_t b_desc = ((uint64_t)desc_hi << 32) | (b_lo + off);
                            if (k == 0)
                                umma_bf16_first(d_addr, a_desc, b_desc, idesc);
                            else
                                umma_bf16_acc(d_addr, a_desc, b_desc, idesc);
                        }
                        umma_commit(&acc_full[buf]);
                        if (last) umma_commit(&q_free[qb]);  // the segment is through with this query tile
                    }
                    if (ok) umma_commit(&empty[st]);  // the stage may be refilled once these MMAs have read it
                    if (++st == p.stages) {
                        st = 0;
                        sph ^= 1;
                    }
                }
                if (reloaded) ++qcnt;
            })
        }
    } else if (warp < 2 + kSoftmaxWarps) {
        // =================================================================== softmax warps (one TMEM lane per thread)
        // They only compute: what has to be exchanged with other CTAs, merged or summed across the groups is the
        // helper warps' business, and every barrier they wait on is normally complete when they get there.
        const int quarter = warp & 3;            // tcgen05.ld reaches lanes 32 * (warp % 4) ..
        const int sw = warp - 2;                 // softmax warp 0..15
        const int grp = sw >> 2;                 // softmax group = the accumulator buffer it owns
        const int my_row = quarter * 32 + lane;  // row of the A tile this thread owns
        const uint32_t t_acc = tmem_base + ((uint32_t)(quarter * 32) << 16) + grp * kRows;
        const float scale2 = mv.scale * kLog2e;
        const int64_t cand = (int64_t)bv.total_cache + bv.total_chunk;
        const int64_t units = (int64_t)mv.L * mv.G;
        int A = 0, mine = 0, segs_b = 0;
        bool ok = true;
        // What depends on the geometry only (the same for every unit of a single-request batch) is worked out once:
        // between two accumulators a softmax warp shares its scheduler's issue slots with three warps that compute,
        // so every instruction of bookkeeping there costs about four cycles.
        uint32_t live_mask = 0;   // bit qb: this thread's row of query tile qb holds a prompt row
        uint64_t valid_pack = 0;  // byte 2 qb / 2 qb + 1: prompt rows in the first / second 64-row half of tile qb
#pragma unroll
        for (int k = 0; k < kQTiles; ++k) {
            const SubBlock sb = sub_block(2 * k + my_row / kSub, g.sbq, g.n_sb, g.u.n_q);
            if (k < g.n_qt && my_row % kSub < sb.valid) live_mask |= 1u << k;
            valid_pack |= (uint64_t)sub_block(2 * k, g.sbq, g.n_sb, g.u.n_q).valid << (16 * k);
            valid_pack |= (uint64_t)sub_block(2 * k + 1, g.sbq, g.n_sb, g.u.n_q).valid << (16 * k + 8);
        }
        FINCH_FOR_EACH_SEGMENT({
            if (ph == 0) {
                // ---------------------------------------------------------------- phase A: row statistics
                float m_raw[kQTiles], z[kQTiles];
#pragma unroll
                for (int k = 0; k < kQTiles; ++k) {
                    m_raw[k] = -INFINITY;
                    z[k] = 0.f;
                }
                for (int t = sg.t0; t < sg.t1 && ok; ++t) {
                    const KeyTile kt = key_tile(u, t);
                    // the one accumulator of this key tile that belongs to the group, if any (accumulator A goes to
                    // group A % 4, a key tile has at most four)
                    const int qb = (grp - A) & 3;
                    A += g.n_qt;
                    if (qb < g.n_qt) {
                        // a wait's verdict is made warp-uniform so that a timeout takes the whole warp out
                        if (!__all_sync(0xffffffffu, mbar_wait(&acc_full[grp], mine & 1, abort_flag))) { ok = false; break; }
                        ++mine;
                        tc_fence_after();
                        float mc = 0.f, zc = 0.f;
#pragma unroll
                        for (int k = 0; k < kQTiles; ++k)
                            if (k == qb) {
                                mc = m_raw[k];
                                zc = z[k];
                            }
                        lse_accumulate<false>(t_acc, kt.valid, scale2, (live_mask >> qb) & 1u, mc, zc, 0);
#pragma unroll
                        for (int k = 0; k < kQTiles; ++k)
                            if (k == qb) {
                                m_raw[k] = mc;
                                z[k] = zc;
                            }
                        tc_fence_before();
                        __syncwarp();
                        if (lane == 0) mbar_arrive(&acc_empty[grp]);
                    }
                }
                if (!ok) break;
                // hand the statistics to the helper warps: every group reports every resident row, (-inf, 0) where
                // it saw no accumulator
                float2 *dst = p.partial + (((int64_t)sg.unit * p.seg_max + sg.slot) * kGroups + grp) * p.rows_u;
#pragma unroll
                for (int qb = 0; qb < kQTiles; ++qb) {
                    if (qb >= g.n_qt) continue;
                    const SubBlock sb = sub_block(2 * qb + my_row / kSub, g.sbq, g.n_sb, u.n_q);
                    const int r = my_row % kSub;
                    if (r < sb.valid) dst[sb.hh * bv.max_q + sb.p0 + r] = make_float2(m_raw[qb] * scale2, z[qb]);
                }
                __syncwarp();
                if (lane == 0) count_arrive(a_count);
            } else {
                // ---------------------------------------------------------------- phase B: column sums
                // The rows' merged statistics (-R, w) of this unit were staged by the helper warps while these warps ran
                // the phase A that came in between; the barrier is normally complete.  Two buffers and two barriers
                // in turn: the helpers cannot be two segments ahead, they wait for these warps' phase A in between.
                if (!__all_sync(0xffffffffu, mbar_wait(&stats_ready[segs_b & 1], (segs_b >> 1) & 1, abort_flag))) { ok = false; break; }
                const float2 *sm_seg = stats_sm + (segs_b & 1) * p.q_tiles * kRows;
                float *part = p.score_parts + ((int64_t)grp * units + sg.unit) * cand + u.cache0 + u.chunk0;
                for (int t = sg.t0; t < sg.t1 && ok; ++t) {
                    const KeyTile kt = key_tile(u, t);
                    float c0 = 0.f, c1 = 0.f;
                    const int qb = (grp - A) & 3;
                    A += g.n_qt;
                    if (qb < g.n_qt) {
                        if (!__all_sync(0xffffffffu, mbar_wait(&acc_full[grp], mine & 1, abort_flag))) { ok = false; break; }
                        ++mine;
                        tc_fence_after();
                        const int v0 = (int)(valid_pack >> (16 * qb)) & 0xff, v1 = (int)(valid_pack >> (16 * qb + 8)) & 0xff;
                        colsum_accumulate<false>(t_acc, v0, v1, scale2, sm_seg + qb * kRows, c0, c1, nullptr, 0);
                        tc_fence_before();
                        __syncwarp();
                        if (lane == 0) mbar_arrive(&acc_empty[grp]);
                    }
                    if (ok && my_row < kt.valid) part[kt.j0 + my_row] = c0 + c1;  // 0 if the group had no accumulator
                }
                if (!ok) break;
                // this warp's partial sums are written: the helper warps add the four groups' sums
                __syncwarp();
                if (lane == 0) count_arrive(b_count);
                ++segs_b;
            }
        })
    } else {
        // =================================================================== helper warps
        // What has to leave the CTA or cross the groups, off the softmax warps' path; they walk the same schedule
        // as everyone.  After a phase-A segment, once the softmax warps have written their statistics, one thread
        // makes them visible to the GPU and bumps the unit's ticket (neighbouring CTAs wait for it).  After a
        // phase-B segment the 64 threads add the four groups' partial column sums, in group order.
        const int tid = threadIdx.x - (2 + kSoftmaxWarps) * 32;
        const int64_t cand = (int64_t)bv.total_cache + bv.total_chunk;
        const int64_t units = (int64_t)mv.L * mv.G;
        const int gcd4 = (g.n_qt & 3) == 0 ? 4 : ((g.n_qt & 1) == 0 ? 2 : 1);  // gcd(query tiles, softmax groups)
        int segs_a = 0, segs_b = 0;
        bool ok = true;
        auto warp_agree = [&](bool good) -> bool { return __all_sync(0xffffffffu, good); };
        FINCH_FOR_EACH_SEGMENT({
            if (ph == 0) {
                ++segs_a;
                // every softmax warp has written the segment's statistics (and is through the phase B of two
                // segments ago, whose buffer is reused below)
                if (!warp_agree(lane != 0 || count_wait(a_count, kSoftmaxWarps * segs_a, abort_flag))) { ok = false; break; }
                if (tid == 0) {
                    __threadfence();  // cumulative: covers the softmax warps' stores this thread has synchronised with
                    atomicAdd(&p.tickets[sg.unit], 1);
                }
                // Stage the unit's statistics for the segment's phase B, which the softmax warps reach one phase A
                // later: wait (bounded) until every range of the unit has published -- the other ranges belong to
                // neighbouring CTAs that run the same window at the same time -- then merge the parts of each prompt
                // row in a fixed order (ranges, then groups) into (-R, w).
                int published = 1;
                if (lane == 0) published = ticket_wait(&p.tickets[sg.unit], sg.n_seg, abort_flag);
                if (!__shfl_sync(0xffffffffu, published, 0)) {
                    ok = false;
                    break;
                }
                float2 *sm_seg = stats_sm + ((segs_a - 1) & 1) * p.q_tiles * kRows;
                const float2 *part_stats = p.partial + ((int64_t)sg.unit * p.seg_max) * kGroups * p.rows_u;
                for (int i = tid; i < g.n_qt * kRows; i += kHelpers) {
                    const int qb = i / kRows, r = i % kRows;  // query tile, row of the tile
                    const SubBlock sb = sub_block(2 * qb + r / kSub, g.sbq, g.n_sb, u.n_q);
                    float2 out = make_float2(0.f, 0.f);
                    if (r % kSub < sb.valid) {
                        const int pr = sb.p0 + r % kSub;
                        const float2 *src = part_stats + sb.hh * bv.max_q + pr;
                        float M = -INFINITY, Z = 0.f;
                        // group g' has met tile qb only if g' - qb is a multiple of gcd(tiles, groups)
#pragma unroll 4
                        for (int sgi = 0; sgi < sg.n_seg; ++sgi) {
                            float2 part[kGroups];
#pragma unroll
                            for (int k = 0; k < kGroups; ++k)
                                part[k] = ((k - qb) & (gcd4 - 1)) == 0
                                              ? __ldcg(src + ((int64_t)sgi * kGroups + k) * p.rows_u)
                                              : make_float2(0.f, 0.f);
#pragma unroll
                            for (int k = 0; k < kGroups; ++k) merge_part(part[k], M, Z);
                        }
                        const int64_t row = ((int64_t)u.l * mv.Hq + u.G * mv.hpg + sb.hh) * bv.total_q + u.q0 + pr;
                        if (bv.self_lse) merge_self_term(bv.self_lse[row], M, Z);
                        float lse_nat;
                        out = merged_pair(M, Z, lse_nat);
                        if (p.row_lse && sg.slot == 0) p.row_lse[row] = lse_nat;  // once per unit: by its first range
                    }
                    // rows 2k and 2k+1 share one float4: (-ref_2k, -ref_2k+1, w_2k, w_2k+1)
                    float *smf = (float *)(sm_seg + qb * kRows) + (r >> 1) * 4 + (r & 1);
                    smf[0] = out.x;
                    smf[2] = out.y;
                }
                __syncwarp();
                if (lane == 0) mbar_arrive(&stats_ready[(segs_a - 1) & 1]);
            } else {
                ++segs_b;
                if (!warp_agree(lane != 0 || count_wait(b_count, kSoftmaxWarps * segs_b, abort_flag))) { ok = false; break; }
                const KeyTile first = key_tile(u, sg.t0), last = key_tile(u, sg.t1 - 1);
                const int j_end = last.j0 + last.valid;
                const float *parts0 = p.score_parts + (int64_t)sg.unit * cand + u.cache0 + u.chunk0;
                float *out = p.unit_scores + (int64_t)sg.unit * cand + u.cache0 + u.chunk0;
                for (int j = first.j0 + tid; j < j_end; j += kHelpers * 4) {  // four keys in flight per thread
                    float v[4][kGroups];
#pragma unroll
                    for (int i = 0; i < 4; ++i)
#pragma unroll
                        for (int k = 0; k < kGroups; ++k)
                            v[i][k] = j + kHelpers * i < j_end ? parts0[(int64_t)k * units * cand + j + kHelpers * i] : 0.f;
#pragma unroll
                    for (int i = 0; i < 4; ++i)
                        if (j + kHelpers * i < j_end) out[j + kHelpers * i] = ((v[i][0] + v[i][1]) + v[i][2]) + v[i][3];
                }
            }
        })
    }
#undef FINCH_FOR_EACH_SEGMENT

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

// Clears the unit tickets of the fused kernel (the scratch keeps whatever the previous call left there).
__global__ void __launch_bounds__(256)
clear_tickets_kernel(int *tickets, int n) {
    dependency_wait();
    dependents_may_launch();
    const int i = blockIdx.x * 256 + threadIdx.x;
    if (i < n) tickets[i] = 0;
}

// scores of a selection group that spans several KV heads (one group per layer): the heads' column sums, added in
// head order.
__global__ void __launch_bounds__(256)
sum_heads_kernel(ModelView mv, BatchView bv, const float *unit_scores, float *scores, int out_groups, int heads_per_group) {
    dependency_wait();
    const int64_t cand = (int64_t)bv.total_cache + bv.total_chunk;
    const int64_t j = (int64_t)blockIdx.x * 256 + threadIdx.x;
    const int l = blockIdx.y / out_groups, og = blockIdx.y % out_groups;
    const UnitInfo u = unit_info(mv, bv, 0, 0);
    if (!u.ok || j >= u.N) return;
    const int64_t at = (int64_t)u.cache0 + u.chunk0 + j;
    float s = 0.f;
    for (int k = 0; k < heads_per_group; ++k) s += unit_scores[((int64_t)l * mv.G + og * heads_per_group + k) * cand + at];
    scores[((int64_t)l * out_groups + og) * cand + at] = s;
}

// Key tiles per range, or 0 when the one-kernel path should leave the batch to the two-launch kernels.  A range
// divides the unit's tiles (otherwise ranges straddle units: the query tiles change inside a range and a unit's tiles
// are dealt unevenly), is long enough to amortise a window's fixed costs (query loads, the exchange of the row
// statistics: at least four tiles, or the whole unit), short enough that the keys in flight between a window's sweeps
// stay in L2, and fills the CTA x window slots of the persistent grid to at least 85 % (27 tiles per unit, 256 units:
// windows of 9 fill 86 % and the step takes 0.258 ms against 0.261 on the two-launch kernels, with K read once).
// Where no such length exists the batch goes to the two-launch kernels, whose key splits are chosen per launch.
int choose_window(long long units, int tiles_per_unit, int ctas, int tile_bytes) {
    const long long total = units * tiles_per_unit;
    const long long l2_budget = 40ll << 20;
    int best = 0;
    double best_score = 0.0;
    for (int W = 1; W <= tiles_per_unit; ++W) {
        if (tiles_per_unit % W) continue;
        if (W < 4 && W < tiles_per_unit) continue;  // a window of a tile or two is all hand-over
        if (tiles_per_unit / W > kMaxSegs) continue;  // the partial-statistics array has kMaxSegs slots per unit
        if (W > 1 && (long long)W * ctas * tile_bytes > l2_budget && best) break;
        const long long ranges = total / W, windows = (ranges + ctas - 1) / ctas;
        const double fill = (double)total / (double)(windows * W * (ranges < ctas ? ranges : ctas));
        if (fill < 0.85) continue;
        const double score = fill - 0.04 / W;
        if (score > best_score) {
            best_score = score;
            best = W;
        }
    }
    return best;
}

template <int D>
cudaError_t launch_fused_d(const Ctx &ctx, const CUtensorMap &qm, const CUtensorMap &cm, const CUtensorMap &hm,
                           FusedParams p, int n_ranges, int out_groups, int heads_per_group, float *scores,
                           cudaStream_t stream) {
    constexpr int kTileBytes = (D / 64) * kSlabBytes;
    const ModelView &mv = p.mv;
    const BatchView &bv = p.bv;
    const int aux = fused_aux_bytes(p.q_tiles);
    p.stages = min(kMaxStages, (kSmemLimit - 1024 - aux - p.q_tiles * kTileBytes) / kTileBytes);
    if (p.stages < 2) return cudaErrorNotSupported;
    const int smem = 1024 + (p.q_tiles + p.stages) * kTileBytes + aux;
    cudaError_t e = cudaFuncSetAttribute(score_fused_kernel<D>, cudaFuncAttributeMaxDynamicSharedMemorySize, smem);
    if (e != cudaSuccess) return e;
    const int units = mv.L * mv.G;
    e = launch_chained(clear_tickets_kernel, dim3((units + 255) / 256), dim3(256), 0, stream, p.tickets, units);
    if (e != cudaSuccess) return e;
    const int sms = ctx.sm_count > 0 ? ctx.sm_count : 148;
    dim3 grid(n_ranges < sms ? n_ranges : sms);  // persistent and resident at once: phase B waits for neighbours
    e = launch_chained(score_fused_kernel<D>, grid, dim3(kFusedThreads), smem, stream, qm, cm, hm, p);
    ctx.launches += 2;
    if (e != cudaSuccess || heads_per_group == 1) return e;
    dim3 sgrid((bv.max_cache + bv.max_chunk + 255) / 256, mv.L * out_groups);
    ctx.launches += 1;
    return launch_chained(sum_heads_kernel, sgrid, dim3(256), 0, stream, mv, bv, (const float *)p.unit_scores, scores,
                          out_groups, heads_per_group);
}

}  // namespace

// Key tiles per window the fused kernel would use for this batch; 0: the batch is not one it takes (several
// requests, causal rows, more than four query tiles per KV head, no window length that fits: see choose_window).
int score_fused_window(const Ctx &ctx, const BatchView &bv) {
    const ModelView &mv = ctx.model;
    if (!score_tc_supported(ctx) || bv.batch != 1 || bv.row_limit || bv.max_q == 0 || bv.max_cache + bv.max_chunk == 0)
        return 0;
    const int sub_blocks = mv.g * ((bv.max_q + kSub - 1) / kSub);
    if ((sub_blocks + 1) / 2 > kQTiles) return 0;
    const int tiles = (bv.max_cache + kRows - 1) / kRows + (bv.max_chunk + kRows - 1) / kRows;
    return choose_window((long long)mv.L * mv.Hkv, tiles, ctx.sm_count > 0 ? ctx.sm_count : 148, (mv.d / 64) * kSlabBytes);
}

// Float2 entries of scratch the fused kernel needs for this batch (0: the batch is not one it takes).
size_t score_fused_scratch(const Ctx &ctx, const BatchView &bv) {
    const ModelView &mv = ctx.model;
    if (score_fused_window(ctx, bv) == 0) return 0;
    const size_t rows = (size_t)mv.L * mv.Hq * (size_t)bv.max_q;
    const size_t units = (size_t)mv.L * mv.Hkv, cand = (size_t)bv.total_cache + bv.total_chunk;
    size_t n = rows * kMaxSegs * kGroups;      // partial row statistics
    n += (units + 1) / 2 + 1;                  // tickets
    n += (kGroups * units * cand + 1) / 2;     // per-group partial column sums
    if (mv.G != mv.Hkv) n += (units * cand + 1) / 2;  // per-KV-head sums of a selection group that spans several
    return n;
}

// Returns cudaErrorNotSupported (and launches nothing) when the batch is not one the fused kernel takes, the
// scratch is too small or the tensors cannot be described to the TMA unit.
cudaError_t launch_score_fused(const Ctx &ctx, const TensorView &q, const TensorView &cache_k, const TensorView &chunk_k,
                               const BatchView &bv, float *scores, float2 *scratch, size_t scratch_capacity,
                               float *row_lse, cudaStream_t stream) {
    const size_t need = score_fused_scratch(ctx, bv);
    if (need == 0 || scratch_capacity < need) return cudaErrorNotSupported;
    ModelView mv = ctx.model;  // the scoring view: a query head only ever meets its own KV head's keys
    mv.G = mv.Hkv;
    mv.hpg = mv.g;
    mv.kvpg = 1;
    CUtensorMap qm, cm, hm;
    if (!make_map(&qm, q, mv.d, bv.total_q, mv.Hq, mv.L, kSub)) return cudaErrorNotSupported;
    const bool have_cache = bv.max_cache > 0, have_chunk = bv.max_chunk > 0;
    if (have_cache && !make_map(&cm, cache_k, mv.d, bv.total_cache, mv.Hkv, mv.L, kRows)) return cudaErrorNotSupported;
    if (have_chunk && !make_map(&hm, chunk_k, mv.d, bv.total_chunk, mv.Hkv, mv.L, kRows)) return cudaErrorNotSupported;
    if (!have_cache) cm = hm;  // never dereferenced: the request has no cache tiles
    if (!have_chunk) hm = cm;
    const int tiles = (bv.max_cache + kRows - 1) / kRows + (bv.max_chunk + kRows - 1) / kRows;
    const int units = mv.L * mv.G;
    const int sms = ctx.sm_count > 0 ? ctx.sm_count : 148;
    const size_t rows = (size_t)mv.L * mv.Hq * (size_t)bv.max_q, cand = (size_t)bv.total_cache + bv.total_chunk;
    FusedParams p{};
    p.mv = mv;
    p.bv = bv;
    p.partial = scratch;
    p.tickets = (int *)(scratch + rows * kMaxSegs * kGroups);
    p.score_parts = (float *)(scratch + rows * kMaxSegs * kGroups + (units + 1) / 2 + 1);
    p.unit_scores = ctx.model.G == mv.Hkv ? scores : p.score_parts + (((size_t)kGroups * units * cand + 1) & ~(size_t)1);
    p.row_lse = row_lse;
    p.status = ctx.d_status;
    p.W = score_fused_window(ctx, bv);
    p.seg_max = kMaxSegs;
    p.rows_u = mv.g * bv.max_q;
    p.q_tiles = (mv.g * ((bv.max_q + kSub - 1) / kSub) + 1) / 2;
    p.delay = 1;
    if (p.W == 0) return cudaErrorNotSupported;
    const int n_ranges = (int)(((long long)units * tiles + p.W - 1) / p.W);
    return mv.d == 64 ? launch_fused_d<64>(ctx, qm, cm, hm, p, n_ranges, ctx.model.G, ctx.model.kvpg, scores, stream)
                      : launch_fused_d<128>(ctx, qm, cm, hm, p, n_ranges, ctx.model.G, ctx.model.kvpg, scores, stream);
}

}  // namespace finch

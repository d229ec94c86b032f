// Stage "scores", first pass, for bf16 caches: every candidate token against the observation queries (Eq. 2-3) and
// against the LAST key tile of its head (Eq. 5 and the start of Section 3.3's scan, which runs from the last position
// downwards).  tcgen05.mma with TMEM accumulators, fed by TMA, one persistent block per SM.
//
// The pass is a single sweep over the keys, so it is organised as a stream: the 128-row key tiles of a head flow
// through a ring of shared-memory stages as the A operand (one token per TMEM lane), while ONE B operand block of the
// head stays put: the rows of its last key tile, then its G * alpha query rows, then 16 rows that hold sum_j Kbar_j
// split into bf16 parts.  Per streamed tile the tensor cores form one product of N = 128 + query rows + 16 (a product
// with few columns costs nearly as much as one with 128), plus one K = 16 step on the key columns that folds the
// threshold test into the accumulator (slices of both operands written by the prep stage):
//
//   columns [0, 128)         h = k_i . k_j - T / (r_i r_j) for the 128 keys j of the last tile: S[j][i] > T exactly
//                            when h > 0.  The thread that owns token i scans them from the last position downwards,
//                            "the first beta hits" are Section 3.3's partners; a partner's value is T + h r_i r_j
//   columns [128, 128 + q)   k_i . q for every query row (a thread ends up with all logits of its key and takes the max,
//                            or the mean, over the group: Eq. 3), then k_i . s in three parts, which gives
//                            sum_j S[j][i] = Kbar_i . (sum_j Kbar_j) - Kbar_i . Kbar_i without forming the matrix
//
// Out, per token: the pooled logits, the column sum minus the removed entries (sbar), the partners still lacking (left).
//
// Work item = (head, range of row tiles); items are handed out by a global ticket counter, head-major.  The operands
// that stay put are double-buffered across items, so the next item's arrive while the current one is streamed, and
// the ring never drains at an item boundary.
// Warp roles (320 threads): warp 0 = tickets + TMA producer, warp 1 = MMA issuer and TMEM owner, warps 2..9 = epilogue
// in two groups of four (warp w may touch TMEM lanes 32 (w % 4) .. +31); group g drains accumulator buffer g, i.e.
// every second tile of the stream.  Every wait on an mbarrier is bounded; on expiry the block records
// RKV_ERR_TIMEOUT, stops issuing work and leaves through the common exit that frees TMEM.  No TMA multicast, no
// cluster launch.
#include "rkv_sm100.cuh"

namespace rkv {

namespace {

using namespace sm100;

constexpr int kThreadsP1 = 320;
constexpr int kHalfBytes = kTile * 64 * 2;       // one TMA box: 128 rows x 64 bf16 (128-byte swizzled rows)
constexpr int kTileBytes = 2 * kHalfBytes;       // 32 KB: a 128 x 128 bf16 operand tile
constexpr int kSliceBytes = kTile * 32;          // the extra K = 16 slice of an operand: 128 rows x 32 bytes (32-byte swizzle)
constexpr int kMaxStagesA = 6;
constexpr uint32_t kTmemColsP1 = 512;            // 2 buffers x (128 key columns + up to 128 query columns)
constexpr int kSmemLimit = 227 * 1024;

enum {
    kBarSlotFull = 0,                            // [2] item descriptor written and its resident operands landed
    kBarSlotEmpty = kBarSlotFull + 2,            // [2] ... no longer read: the MMA thread and the 8 epilogue warps
    kBarAFull = kBarSlotEmpty + 2,               // [kMaxStagesA] streamed tile landed
    kBarAEmpty = kBarAFull + kMaxStagesA,        // [kMaxStagesA] ... and consumed by the products
    kBarAccFull = kBarAEmpty + kMaxStagesA,      // [2] accumulator buffer written
    kBarAccEmpty = kBarAccFull + 2,              // [2] ... and drained by its 4 epilogue warps
    kNumBarsP1 = kBarAccEmpty + 2
};

// Shared-memory carve-up, offsets from a 1024-byte aligned base.
struct SmemPlan {
    int stages;          // ring depth
    int q_bytes;         // bytes of the query block: (q_rows_pad + 16) rows x 256 B
    int off_aug;         // stages x slice of a streamed tile
    int off_slot;        // 2 x [B block: rows [0, 128) the last key tile, then the query block; as two 64-column halves |
                         //      slice of the last key tile]
    int slot_bytes;      // (128 + q_rows_pad + 16) rows x 256 B; a half is slot_bytes / 2
    int slot_stride;     // slot_bytes + kSliceBytes
    int off_rj;          // 2 x 128 floats: r_j of the last key tile
    int off_bar, off_items, off_misc, total;
};

__host__ __device__ inline SmemPlan make_plan(int q_rows_pad)
{
    SmemPlan pl;
    pl.q_bytes = (q_rows_pad + 16) * 256;
    pl.slot_bytes = kTileBytes + pl.q_bytes;
    pl.slot_stride = pl.slot_bytes + kSliceBytes;
    const int fixed = 2 * pl.slot_stride + 2 * kTile * 4 + kNumBarsP1 * 8 + 2 * 16 + 16 + 1024;   // + alignment slack
    int stages = (kSmemLimit - fixed) / (kTileBytes + kSliceBytes);
    pl.stages = stages > kMaxStagesA ? kMaxStagesA : stages;
    pl.off_aug = pl.stages * kTileBytes;
    pl.off_slot = pl.off_aug + pl.stages * kSliceBytes;
    pl.off_rj = pl.off_slot + 2 * pl.slot_stride;
    pl.off_bar = pl.off_rj + 2 * kTile * 4;
    pl.off_items = pl.off_bar + kNumBarsP1 * 8;
    pl.off_misc = pl.off_items + 2 * 16;
    pl.total = pl.off_misc + 16 + 1024;
    return pl;
}

// Item descriptor (int4): {head, first row tile, one past the last row tile, n}.  x < 0: no more items.
__global__ void __launch_bounds__(kThreadsP1, 1)
scores_stream_sm100_kernel(Params p, const __grid_constant__ CUtensorMap map_k, const __grid_constant__ CUtensorMap map_q,
                           const __grid_constant__ CUtensorMap map_hs, const __grid_constant__ CUtensorMap map_ns,
                           const __grid_constant__ CUtensorMap map_ts, int splits, unsigned long long total_items,
                           int q_rows_pad)
{
    extern __shared__ uint8_t smem_raw[];
    uint8_t *smem = reinterpret_cast<uint8_t *>((reinterpret_cast<uintptr_t>(smem_raw) + 1023) & ~(uintptr_t)1023);
    const uint32_t sbase = smem_u32(smem);
    const SmemPlan pl = make_plan(q_rows_pad);
    int4 *items = reinterpret_cast<int4 *>(smem + pl.off_items);
    uint32_t *tmem_holder = reinterpret_cast<uint32_t *>(smem + pl.off_misc);
    volatile int *abort_flag = reinterpret_cast<volatile int *>(smem + pl.off_misc + 4);
    volatile int *bail = reinterpret_cast<volatile int *>(smem + pl.off_misc + 8);
    const uint32_t bar0 = sbase + pl.off_bar;
    auto bar = [bar0](int idx) -> uint32_t { return bar0 + 8u * (uint32_t)idx; };
    const int stages = pl.stages;

    // Once a bounded wait of this call has run out, the blocks still to start return at once.
    const ErrSink sink = make_sink(p);
    if (threadIdx.x == 0) *bail = call_aborted(p) ? 1 : 0;
    __syncthreads();
    if (*bail) return;

    const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
    const bool rule_on = p.beta > 0 && p.sim_threshold < 1.0f;

    if (threadIdx.x == 0) {
        for (int s = 0; s < 2; ++s) {
            mbar_init(bar(kBarSlotFull + s), 1);
            mbar_init(bar(kBarSlotEmpty + s), 9);
            mbar_init(bar(kBarAccFull + s), 1);
            mbar_init(bar(kBarAccEmpty + s), 4);
        }
        for (int s = 0; s < kMaxStagesA; ++s) {
            mbar_init(bar(kBarAFull + s), 1);
            mbar_init(bar(kBarAEmpty + s), 1);
        }
        *abort_flag = 0;
        asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory");
    }
    if (warp == 1) {
        asm volatile("tcgen05.alloc.cta_group::1.sync.aligned.shared::cta.b32 [%0], %1;"
                     ::"r"(smem_u32(tmem_holder)), "r"(kTmemColsP1) : "memory");
        asm volatile("tcgen05.relinquish_alloc_permit.cta_group::1.sync.aligned;" ::: "memory");
    }
    tc_fence_before();
    __syncthreads();
    tc_fence_after();
    const uint32_t tmem_base = *tmem_holder;
    unsigned long long tiles_done = 0ull;

    if (warp == 0) {
        // ------------------------------------------------------------------ tickets + TMA producer
        if (lane == 0) {
            uint32_t k_item = 0, acount = 0;
            bool ok = true;
            // the next ticket is drawn while the current item is set up (a block draws one ticket too many)
            unsigned long long next_ticket = atomicAdd(&p.counters[1], 1ull);
            while (ok) {
                const unsigned long long ticket = next_ticket;
                if (ticket >= total_items) break;
                next_ticket = atomicAdd(&p.counters[1], 1ull);
                const int head = (int)(ticket / (unsigned)splits);
                const int part = (int)(ticket % (unsigned)splits);
                const int n = seq_candidates(p, head / p.hkv);
                if (n == 0) continue;
                const int n_tiles = (n + kTile - 1) / kTile;
                const int t0 = (int)((long long)part * n_tiles / splits), t1 = (int)((long long)(part + 1) * n_tiles / splits);
                if (t0 >= t1) continue;                                        // more parts than tiles

                const uint32_t slot = k_item & 1;
                if (!mbar_wait(bar(kBarSlotEmpty + slot), ((k_item >> 1) & 1) ^ 1, abort_flag, sink)) break;
                items[slot] = make_int4(head, t0, t1, n);
                const uint32_t slot_addr = sbase + pl.off_slot + slot * pl.slot_stride;
                const uint32_t full = bar(kBarSlotFull + slot);
                // the descriptor is published by this arrival; the barrier completes when the operands have landed too
                mbar_expect_tx(full, (uint32_t)pl.q_bytes + (rule_on ? (uint32_t)(kTileBytes + kSliceBytes + kTile * 4) : 0u));
                {
                    const int b = head / p.hkv, h = head % p.hkv;
                    const int q_row = (b * p.hq + h * p.group) * p.alpha;
                    const uint32_t half = (uint32_t)pl.slot_bytes / 2, qdst = slot_addr + kTile * 128;
                    // behind the key tile's rows: the query rows, then 16 rows holding sum_j Kbar_j split into bf16
                    // parts; both 64-column halves
                    tma_load_2d(qdst, &map_q, 0, q_row, full);
                    tma_load_2d(qdst + half, &map_q, 64, q_row, full);
                    tma_load_2d(qdst + q_rows_pad * 128, &map_hs, 0, head * 16, full);
                    tma_load_2d(qdst + half + q_rows_pad * 128, &map_hs, 64, head * 16, full);
                }
                if (rule_on) {
                    const int y = (int)tile_row0(p, head, n_tiles - 1);
                    tma_load_2d(slot_addr, &map_k, 0, y, full);
                    tma_load_2d(slot_addr + (uint32_t)pl.slot_bytes / 2, &map_k, 64, y, full);
                    // the tile's extra slice: -T / r_j of its keys in three bf16 parts
                    tma_load_2d(slot_addr + (uint32_t)pl.slot_bytes, &map_ts, 0, head * kTile, full);
                    asm volatile("cp.async.bulk.shared::cluster.global.mbarrier::complete_tx::bytes [%0], [%1], %2, [%3];"
                                 ::"r"(sbase + pl.off_rj + slot * kTile * 4),
                                   "l"(p.inv_norm + (size_t)head * p.cap_pad + (size_t)(n_tiles - 1) * kTile),
                                   "r"((uint32_t)(kTile * 4)), "r"(full)
                                 : "memory");
                }
                for (int t = t0; t < t1; ++t) {
                    const uint32_t s = acount % (uint32_t)stages;
                    if (!mbar_wait(bar(kBarAEmpty + s), ((acount / (uint32_t)stages) & 1) ^ 1, abort_flag, sink)) {
                        ok = false;
                        break;
                    }
                    const uint32_t dst = sbase + s * kTileBytes;
                    const int y = (int)tile_row0(p, head, t);
                    mbar_expect_tx(bar(kBarAFull + s), kTileBytes + (rule_on ? kSliceBytes : 0));
                    tma_load_2d(dst, &map_k, 0, y, bar(kBarAFull + s));
                    tma_load_2d(dst + kHalfBytes, &map_k, 64, y, bar(kBarAFull + s));
                    if (rule_on)    // the tile's extra slice: 1 / r_i of its keys in three bf16 parts
                        tma_load_2d(sbase + pl.off_aug + s * kSliceBytes, &map_ns, 0, head * p.cap_pad + t * kTile,
                                    bar(kBarAFull + s));
                    ++acount;
                }
                ++k_item;
            }
            // terminator: tells the other roles that no item follows (skipped when the block is aborting)
            if (!*abort_flag) {
                const uint32_t slot = k_item & 1;
                if (mbar_wait(bar(kBarSlotEmpty + slot), ((k_item >> 1) & 1) ^ 1, abort_flag, sink)) {
                    items[slot] = make_int4(-1, 0, 0, 0);
                    mbar_arrive(bar(kBarSlotFull + slot));
                }
            }
        }
        __syncwarp();
    } else if (warp == 1) {
        // ------------------------------------------------------------------ MMA issuer
        if (lane == 0) {
            // one product per streamed tile: N = the 128 keys of the last tile + the query block (the query block alone
            // while the retention rule is off)
            const uint32_t idesc_kq = instr_desc(kTile, kTile + q_rows_pad + 16), idesc_q = instr_desc(kTile, q_rows_pad + 16);
            const uint32_t idesc_k = instr_desc(kTile, kTile);
            uint32_t k_item = 0, acount = 0;
            bool ok = true;
            while (ok) {
                const uint32_t slot = k_item & 1;
                if (!mbar_wait(bar(kBarSlotFull + slot), (k_item >> 1) & 1, abort_flag, sink)) break;
                const int4 d = items[slot];
                if (d.x < 0) break;
                const uint32_t b_block = sbase + pl.off_slot + slot * pl.slot_stride, b_half = (uint32_t)pl.slot_bytes / 2;
                for (int t = d.y; t < d.z; ++t) {
                    const uint32_t s = acount % (uint32_t)stages;
                    if (!mbar_wait(bar(kBarAFull + s), (acount / (uint32_t)stages) & 1, abort_flag, sink)) {
                        ok = false;
                        break;
                    }
                    const uint32_t a = acount & 1;                 // tile c of the stream uses accumulator buffer c & 1
                    if (!mbar_wait(bar(kBarAccEmpty + a), ((acount >> 1) & 1) ^ 1, abort_flag, sink)) {
                        ok = false;
                        break;
                    }
                    tc_fence_after();
                    const uint32_t tile = sbase + s * kTileBytes;
                    const uint32_t d_tmem = tmem_base + a * 256;
                    if (rule_on) {
                        umma_tile_k128_halves(d_tmem, tile, kHalfBytes, b_block, b_half, idesc_kq);
                        // ... - T / (r_i r_j) onto the key columns: the accumulator's sign is the threshold test
                        umma_k16_sw32(d_tmem, sbase + pl.off_aug + s * kSliceBytes, b_block + (uint32_t)pl.slot_bytes, idesc_k);
                        ++tiles_done;
                    } else {
                        umma_tile_k128_halves(d_tmem + 128, tile, kHalfBytes, b_block + kTile * 128, b_half, idesc_q);
                    }
                    umma_commit(bar(kBarAccFull + a));
                    umma_commit(bar(kBarAEmpty + s));              // the stage may be refilled once these products have read it
                    ++acount;
                }
                if (!ok) break;
                umma_commit(bar(kBarSlotEmpty + slot));            // so may the item's resident operands
                ++k_item;
            }
        }
        __syncwarp();
    } else {
        // ------------------------------------------------------------------ epilogue warps
        const int ew = warp - 2;                 // 0..7
        const int grp = ew >> 2;                 // accumulator buffer this warp drains
        const int quad = warp & 3;               // TMEM lane quadrant this warp may access
        const int lrow = quad * 32 + lane;       // row within the 128-row tile
        const uint32_t lane_base = tmem_base + ((uint32_t)(quad * 32) << 16) + (uint32_t)grp * 256;
        const float kInf = __int_as_float(0x7f800000);
        const float scale = p.logit_scale;                    // 1 / sqrt(d)
        const int G = p.group;
        uint32_t k_item = 0, ccount = 0;         // ccount: tiles of the stream so far (all of them, not only this group's)
        bool ok = true;

        while (ok) {
            const uint32_t slot = k_item & 1;
            if (!mbar_wait(bar(kBarSlotFull + slot), (k_item >> 1) & 1, abort_flag, sink)) break;
            const int4 d = items[slot];
            if (d.x < 0) break;
            const int head = d.x, n = d.w;
            const int last_tile = (n + kTile - 1) / kTile - 1;
            const int jbase = last_tile * kTile;
            const float *inv_norm = p.inv_norm + (size_t)head * p.cap_pad;
            const float4 *rj4 = reinterpret_cast<const float4 *>(smem + pl.off_rj + slot * kTile * 4);
            float *logits = p.logits + (size_t)head * p.alpha * p.cap_pad;

            const float *self_dot = p.self_dot + (size_t)head * p.cap_pad;
            float ri_next = 0.f, self_next = 0.f;
            int t_next = -1;                     // the tile ri_next / self_next were fetched for
            for (int t = d.y; t < d.z; ++t, ++ccount) {
                if ((int)(ccount & 1) != grp) continue;
                const int i = t * kTile + lrow;
                const bool row_ok = i < n;
                float ri, self;
                if (t_next == t) {
                    ri = ri_next;
                    self = self_next;
                } else {
                    ri = row_ok ? __ldg(inv_norm + i) : 0.f;
                    self = row_ok ? __ldg(self_dot + i) : 0.f;
                }
                if (t + 2 < d.z) {               // this group's next tile of the item: its factors arrive while this one is drained
                    const int i2 = i + 2 * kTile;
                    t_next = t + 2;
                    ri_next = i2 < n ? __ldg(inv_norm + i2) : 0.f;
                    self_next = i2 < n ? __ldg(self_dot + i2) : 0.f;
                }
                if (!mbar_wait(bar(kBarAccFull + grp), (ccount >> 1) & 1, abort_flag, sink)) {
                    ok = false;
                    break;
                }
                tc_fence_after();

                // ---- Eq. 2-3: all G * alpha logits of this key in its accumulator row, then k_i . s in three parts
                const uint32_t qbase = lane_base + 128;
                uint32_t sp[8];
                tmem_ld8(qbase + q_rows_pad, sp);
                float pooled[8];
                if (p.alpha == 8) {
#pragma unroll
                    for (int j = 0; j < 8; ++j) pooled[j] = p.gqa_mean_pool ? 0.f : -kInf;
                    for (int g0 = 0; g0 < G; g0 += 4) {       // four query heads per round trip to TMEM
                        uint32_t t0[8], t1[8], t2[8], t3[8];
                        tmem_ld8(qbase + g0 * 8, t0);
                        tmem_ld8(qbase + min(g0 + 1, G - 1) * 8, t1);     // heads beyond the group re-read its last one
                        tmem_ld8(qbase + min(g0 + 2, G - 1) * 8, t2);
                        tmem_ld8(qbase + min(g0 + 3, G - 1) * 8, t3);
                        tmem_wait8(t0);
                        tmem_wait8(t1);
                        tmem_wait8(t2);
                        tmem_wait8(t3);
                        if (p.gqa_mean_pool) {        // the variant: sum over the group (scaled to the mean below)
                            const bool h1 = g0 + 1 < G, h2 = g0 + 2 < G, h3 = g0 + 3 < G;
#pragma unroll
                            for (int j = 0; j < 8; ++j)
                                pooled[j] += (__uint_as_float(t0[j]) + (h1 ? __uint_as_float(t1[j]) : 0.f)) +
                                             ((h2 ? __uint_as_float(t2[j]) : 0.f) + (h3 ? __uint_as_float(t3[j]) : 0.f));
                            continue;
                        }
#pragma unroll
                        for (int j = 0; j < 8; ++j)
                            pooled[j] = fmaxf(fmaxf(pooled[j], __uint_as_float(t0[j])),
                                              max3(__uint_as_float(t1[j]), __uint_as_float(t2[j]), __uint_as_float(t3[j])));
                    }
                    const float scale_q = p.gqa_mean_pool ? scale / (float)G : scale;
#pragma unroll
                    for (int j = 0; j < 8; ++j) pooled[j] *= scale_q;
                } else {
                    for (int j = 0; j < p.alpha; ++j) {
                        float best = -kInf, sum = 0.f;
                        for (int g0 = 0; g0 < G; g0 += 4) {
                            uint32_t tq[4];
#pragma unroll
                            for (int u = 0; u < 4; ++u) tmem_ld1(qbase + min(g0 + u, G - 1) * p.alpha + j, tq[u]);
                            asm volatile("tcgen05.wait::ld.sync.aligned;"
                                         : "+r"(tq[0]), "+r"(tq[1]), "+r"(tq[2]), "+r"(tq[3]) :: "memory");
#pragma unroll
                            for (int u = 0; u < 4; ++u) {
                                best = fmaxf(best, __uint_as_float(tq[u]));
                                sum += (g0 + u < G) ? __uint_as_float(tq[u]) : 0.f;
                            }
                        }
                        if (row_ok)      // (written here: alpha is not known at compile time on this path)
                            logits[(size_t)j * p.cap_pad + i] = p.gqa_mean_pool ? sum * scale / (float)G : best * scale;
                    }
                }
                tmem_wait8(sp);
                // sum_j S[j][i] before the retention rule: Kbar_i . s - Kbar_i . Kbar_i
                const float total = ri * ((__uint_as_float(sp[0]) + __uint_as_float(sp[1])) + __uint_as_float(sp[2])) - self;

                // ---- the last key tile, last position first.  The accumulator holds h = k_i . k_j - T / (r_i r_j):
                // S[j][i] > T exactly when h > 0, so the screening is a sign test with nothing to load per column; a
                // partner's value is S = T + h r_i r_j, with the r_j of the tile in shared memory.
                float removed = 0.f;             // sum of h r_j over the partners found
                int nhit = 0;
                int left = row_ok ? p.beta : 0;
                if (rule_on) {
                    bool want = left > 0;
                    const int valid = n - jbase;                  // columns [0, valid) of the tile are candidates
                    const float *rj = reinterpret_cast<const float *>(rj4);
                    // 32-column chunks, last first.  The TMEM load of the next chunk is issued before the current one is
                    // looked at, so its latency passes under the work (two register sets, used alternately).
                    auto chunk = [&](const uint32_t (&g)[32], int ch) {
                        const int nv = valid - ch * 32;
                        uint32_t colmask = nv >= 32 ? 0xffffffffu : (nv <= 0 ? 0u : ((1u << nv) - 1u));
                        const unsigned own = (unsigned)(i - (jbase + ch * 32));           // zero diagonal (Eq. 5)
                        if (own < 32u) colmask &= ~(1u << own);
                        // bit c of `neg` = sign bit of entry c: one funnel shift per entry, four independent chains
                        uint32_t n0 = 0u, n1 = 0u, n2 = 0u, n3 = 0u;
#pragma unroll
                        for (int c = 7; c >= 0; --c) {
                            n0 = __funnelshift_l(g[c], n0, 1);
                            n1 = __funnelshift_l(g[8 + c], n1, 1);
                            n2 = __funnelshift_l(g[16 + c], n2, 1);
                            n3 = __funnelshift_l(g[24 + c], n3, 1);
                        }
                        const uint32_t neg = (n0 | (n1 << 8)) | ((n2 << 16) | (n3 << 24));
                        // entries with a clear sign bit (h > 0, but also +0 and some NaN patterns of rows that are not
                        // candidates: confirmed one by one below)
                        uint32_t pos = want ? (~neg & colmask) : 0u;
                        if (p.beta == 1) {
                            // one partner at most: the candidate at the highest set bit, its value picked by a select
                            // tree (nearly always a single turn)
                            while (pos != 0u) {
                                const int top = 31 - __clz(pos);
                                uint32_t t16[16], t8[8], t4[4];
#pragma unroll
                                for (int c = 0; c < 16; ++c) t16[c] = (top & 16) ? g[16 + c] : g[c];
#pragma unroll
                                for (int c = 0; c < 8; ++c) t8[c] = (top & 8) ? t16[8 + c] : t16[c];
#pragma unroll
                                for (int c = 0; c < 4; ++c) t4[c] = (top & 4) ? t8[4 + c] : t8[c];
                                const uint32_t u0 = (top & 2) ? t4[2] : t4[0], u1 = (top & 2) ? t4[3] : t4[1];
                                const float hv = __uint_as_float((top & 1) ? u1 : u0);
                                if (hv > 0.f) {
                                    removed = hv * rj[ch * 32 + top];
                                    nhit = 1;
                                    left = 0;
                                    want = false;
                                    break;
                                }
                                pos &= ~(1u << top);
                            }
                            return;
                        }
                        // several partners per token: the exact mask, cut down to the highest positions if they are more
                        // than the token still lacks, then the sum of their h r_j
                        if (!__any_sync(0xffffffffu, pos != 0u)) return;
                        uint32_t hits = 0u;
#pragma unroll
                        for (int c = 0; c < 32; ++c) hits |= (__uint_as_float(g[c]) > 0.f) ? (1u << c) : 0u;
                        hits &= pos;
                        int taken = __popc(hits);
                        for (; taken > left; --taken) hits &= hits - 1u;                   // drop the lowest positions
                        float s0 = 0.f, s1 = 0.f, s2 = 0.f, s3 = 0.f;
#pragma unroll
                        for (int q = 0; q < 8; ++q) {
                            const float4 R = rj4[ch * 8 + q];
                            s0 += (hits >> (4 * q) & 1u) ? __uint_as_float(g[4 * q]) * R.x : 0.f;
                            s1 += (hits >> (4 * q + 1) & 1u) ? __uint_as_float(g[4 * q + 1]) * R.y : 0.f;
                            s2 += (hits >> (4 * q + 2) & 1u) ? __uint_as_float(g[4 * q + 2]) * R.z : 0.f;
                            s3 += (hits >> (4 * q + 3) & 1u) ? __uint_as_float(g[4 * q + 3]) * R.w : 0.f;
                        }
                        removed += (s0 + s1) + (s2 + s3);
                        nhit += taken;
                        left -= taken;
                        if (left == 0) want = false;
                    };
                    if (__any_sync(0xffffffffu, want)) {
                        uint32_t ga[32], gb[32];
                        tmem_ld32(lane_base + 3 * 32, ga);
                        tmem_wait32(ga);
                        tmem_ld32(lane_base + 2 * 32, gb);
                        chunk(ga, 3);
                        tmem_wait32(gb);
                        if (__any_sync(0xffffffffu, want)) {                              // else every token of the warp is served
                            tmem_ld32(lane_base + 1 * 32, ga);
                            chunk(gb, 2);
                            tmem_wait32(ga);
                            if (__any_sync(0xffffffffu, want)) {
                                tmem_ld32(lane_base, gb);
                                chunk(ga, 1);
                                tmem_wait32(gb);
                                if (__any_sync(0xffffffffu, want)) chunk(gb, 0);
                            }
                        }
                    }
                }
                // the accumulator buffer is free again
                tc_fence_before();
                __syncwarp();
                if (lane == 0) mbar_arrive(bar(kBarAccEmpty + grp));

                if (row_ok) {
                    if (p.alpha == 8) {
#pragma unroll
                        for (int j = 0; j < 8; ++j) logits[(size_t)j * p.cap_pad + i] = pooled[j];
                    }
                    p.sbar[(size_t)head * p.cap_pad + i] = total - ((float)nhit * p.sim_threshold + removed * ri);
                    p.left[(size_t)head * p.cap_pad + i] = rule_on ? left : 0;
                }
            }
            if (!ok) break;
            // the item's r_j and descriptor are no longer read by this warp
            __syncwarp();
            if (lane == 0) mbar_arrive(bar(kBarSlotEmpty + slot));
            ++k_item;
        }
    }

    // ---------------------------------------------------------------------- common exit
    tc_fence_before();
    __syncthreads();
    if (warp == 1) {
        if (*abort_flag) __nanosleep(200000);      // error path only: let copies and MMAs in flight land
        tc_fence_after();
        asm volatile("tcgen05.dealloc.cta_group::1.sync.aligned.b32 %0, %1;" ::"r"(tmem_base), "r"(kTmemColsP1) : "memory");
    }
    if (warp == 1 && lane == 0 && !*abort_flag && tiles_done) atomicAdd(p.counters, tiles_done);
}

}  // namespace

cudaError_t launch_scores_pass1_sm100(const Params &p, cudaStream_t s, const CUtensorMap &map_k, const CUtensorMap &map_q,
                                      const CUtensorMap &map_hs, const CUtensorMap &map_ns, const CUtensorMap &map_ts,
                                      int q_rows_pad, int sms)
{
    const SmemPlan pl = make_plan(q_rows_pad);
    if (pl.stages < 2) return cudaErrorInvalidConfiguration;
    cudaError_t e;
    if ((e = cudaFuncSetAttribute(scores_stream_sm100_kernel, cudaFuncAttributeMaxDynamicSharedMemorySize, pl.total)) !=
        cudaSuccess)
        return e;
    const int heads = p.batch * p.hkv;
    // a head is cut into parts when there are too few heads to give every SM several items
    int splits = (4 * sms + heads - 1) / heads;
    splits = splits < 1 ? 1 : (splits > p.tiles ? p.tiles : splits);
    const unsigned long long total_items = (unsigned long long)splits * (unsigned long long)heads;
    const unsigned grid = (unsigned)(total_items < (unsigned long long)sms ? total_items : (unsigned long long)sms);
    scores_stream_sm100_kernel<<<grid, kThreadsP1, pl.total, s>>>(p, map_k, map_q, map_hs, map_ns, map_ts, splits, total_items,
                                                                  q_rows_pad);
    return cudaGetLastError();
}

}  // namespace rkv

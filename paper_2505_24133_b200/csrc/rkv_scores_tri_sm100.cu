// Stage "scores", tensor-core version for bf16 caches (the default): tcgen05.mma with TMEM accumulators, fed by
// TMA, one persistent block per SM.  Two passes over Eq. 5's similarity matrix that form only the part of it the
// result can depend on.
//
// Section 3.3's rule needs, per token i, the beta LARGEST positions j with S[j][i] > T.  S is symmetric before the
// rule, so token i's line can be read as row i.
//
//   pass 1  Every token against the LAST positions.  Work item = (head, pair of row tiles p): rows
//           [256 p, 256 p + 256) stay resident in shared memory as two 128 x 128 bf16 operand tiles
//           (double-buffered across items); the last kPass1Depth key tiles (for the last row tiles: down to their
//           own, diagonal tile) stream through a 3-stage ring.  One thread owns one token and scans its line from
//           the last position downwards, so the rule is "the first beta hits", kept in registers.  Before the key
//           tiles, the item multiplies its resident tiles with the head's G * alpha query rows (Eq. 2-3: a thread
//           ends up with all logits of its key and takes the max over the group).  Out: logits, the column sum
//           minus the removed entries, and `left` = partners still lacking.
//   compact The tokens with left > 0 (a few per cent when similar keys are common; all of them when nothing
//           exceeds T) are listed per head, ascending, in chunks of 256.
//   pass 2  Work item = (head, chunk of 256 listed tokens): their key rows are gathered into the resident tiles
//           by the epilogue warps; the key tiles from where pass 1 stopped down to tile 0 stream through the same
//           ring.  The removed entries are subtracted from what pass 1 stored.
//
// So the tensor cores form (tokens) x (the last positions) plus (listed tokens) x (the rest) entries per head
// instead of n^2; the n x n matrix never leaves TMEM, and no atomics or global flags are involved.
//
// Per element the epilogue costs one multiply (g r_j) and half a max; only a 32-column chunk whose maximum
// exceeds the token's threshold T / r_i is looked at entry by entry, last first.
// The plain column sum of Eq. 6 is not accumulated element by element:
// sum_j S[j][i] = Kbar_i . (sum_j Kbar_j) - Kbar_i . Kbar_i, with sum_j Kbar_j from the prep stage.
//
// Items are handed out by a global ticket counter, longest first within a head, so neighbouring blocks work on
// the same head while its keys are in L2.
// Warp roles (352 threads): warp 0 = ticket + TMA producer, warp 1 = MMA issuer of row tile 0 and TMEM owner,
// warp 10 = MMA issuer of row tile 1, warps 2..9 = epilogue (warp w may touch TMEM lanes 32 (w % 4) .. +31; warps 2-5 serve row tile 0, warps 6-9 row tile 1).
// TMEM: four 128-column fp32 accumulators, two per row tile, so the tensor pipe fills one while the epilogue
// drains the other.  Every wait on an mbarrier is bounded; on expiry the block records RKV_ERR_TIMEOUT, stops
// issuing work and leaves through the common exit that frees TMEM.  No TMA multicast and no cluster launch.
#include "rkv_sm100.cuh"

namespace rkv {

namespace {

using namespace sm100;

constexpr int kThreads = 352;                    // 11 warps: producer, 2 MMA issuers (warps 1 and 10), 8 epilogue
constexpr int kStagesB = 3;                      // ring depth of streamed tiles
constexpr int kItemSlots = 4;                    // ring depth of item descriptors
constexpr int kHalfBytes = kTile * 64 * 2;       // one TMA box: 128 rows x 64 bf16 (128-byte swizzled rows)
constexpr int kTileBytes = 2 * kHalfBytes;       // 32 KB: a 128 x 128 bf16 operand tile
constexpr int kRowsPerItem = 2 * kTile;
constexpr uint32_t kTmemCols = 512;
constexpr int kPass1Depth = 1;                   // key tiles every token is scanned against in pass 1 (measured: 1 beats 2 and 3)

// shared memory carve-up (offsets from a 1024-byte aligned base)
constexpr int kOffA = 0;                                   // 2 buffers x 2 resident tiles
constexpr int kOffB = kOffA + 2 * 2 * kTileBytes;          // kStagesB streamed tiles
constexpr int kOffBar = kOffB + kStagesB * kTileBytes;     // mbarriers
enum {
    kBarQFull = 0,                          // [kItemSlots] item descriptor written
    kBarQEmpty = kBarQFull + kItemSlots,    // [kItemSlots] read by the 2 MMA threads and the 8 epilogue warps
    kBarAFull = kBarQEmpty + kItemSlots,    // [2] resident tiles in place
    kBarAEmpty = kBarAFull + 2,             // [2] resident tiles no longer read
    kBarBFull = kBarAEmpty + 2,             // [kStagesB]
    kBarBEmpty = kBarBFull + kStagesB,      // [kStagesB]
    kBarAccFull = kBarBEmpty + kStagesB,    // [2 buffers][2 row tiles]
    kBarAccEmpty = kBarAccFull + 4,         // [2][2], 4 warps each
    kBarRFull = kBarAccEmpty + 4,           // [2] the r_j of the item's key tiles are in shared memory
    kBarREmpty = kBarRFull + 2,             // [2] ... and no longer read (8 epilogue warps)
    kNumBars = kBarREmpty + 2
};
// Pass 2 keeps one pair of resident tiles (its items are long) and uses the room of the second pair for the extra
// K = 16 slices of its operands: 128 rows x 32 bytes each (32-byte swizzle), one per resident tile and one per stage
// of the ring.
constexpr int kSliceBytes = kTile * 32;
constexpr int kOffAugA = kOffA + 2 * kTileBytes;           // 2 slices, beside the resident tiles
constexpr int kOffAugB = kOffAugA + 2 * kSliceBytes;       // kStagesB slices, beside the streamed tiles
// ... and, when beta > 1 (several partners per token: their values need the r_j of whole chunks), for the r_j of
// the head, one item at a time.
constexpr int kOffRHead = kOffAugB + kStagesB * kSliceBytes;
static_assert((2 + kStagesB) * kSliceBytes + RKV_MAX_CAP * 4 <= 2 * kTileBytes, "slices and r_j must fit the second resident pair");
constexpr int kOffItems = kOffBar + kNumBars * 8;          // kItemSlots x int4
constexpr int kOffMisc = kOffItems + kItemSlots * 16;      // tmem base, abort flag, bail flag
constexpr int kOffRj = kOffMisc + 16;                      // pass 1: [2 items][kPass1Depth * 128] r_j of the streamed tiles
constexpr int kSmemBytes = kOffRj + 2 * kPass1Depth * kTile * 4 + 1024;  // + slack for the manual 1024-byte alignment
static_assert(kOffItems % 16 == 0 && kOffRj % 16 == 0, "item descriptors are read as int4, r_j as float4");
static_assert(kSmemBytes <= 227 * 1024, "shared memory budget");

struct Bars {
    uint32_t bar0;
    __device__ __forceinline__ uint32_t at(int idx) const { return bar0 + 8 * idx; }
};

// Item descriptor (int4).  Pass 1: {head, pair p, n, -}.  Pass 2: {head, first listed token k0, tokens in the item
// (1..256), first streamed tile}.  x < 0: no more items.
//
// kPass2 = false: pass 1; true: pass 2 (see the top of the file).
template <bool kPass2>
__global__ void __launch_bounds__(kThreads, 1)
scores_tri_sm100_kernel(Params p, const __grid_constant__ CUtensorMap map_k, const __grid_constant__ CUtensorMap map_q,
                        const __grid_constant__ CUtensorMap map_hs, const __grid_constant__ CUtensorMap map_ns,
                        int items_per_head,
                        unsigned long long total_items_host, int q_rows_pad)
{
    extern __shared__ uint8_t smem_raw[];
    uint8_t *smem = reinterpret_cast<uint8_t *>((reinterpret_cast<uintptr_t>(smem_raw) + 1023) & ~(uintptr_t)1023);
    const uint32_t sbase = smem_u32(smem);
    int4 *items = reinterpret_cast<int4 *>(smem + kOffItems);
    uint32_t *tmem_holder = reinterpret_cast<uint32_t *>(smem + kOffMisc);
    volatile int *abort_flag = reinterpret_cast<volatile int *>(smem + kOffMisc + 4);
    volatile int *bail = reinterpret_cast<volatile int *>(smem + kOffMisc + 8);
    const Bars bar{sbase + kOffBar};

    // Once a bounded wait of this call has run out, the blocks still to start return at once (a sequence with an
    // invalid length does not stop the others: it just has no candidates).  Pass 2 has nothing to do when the list
    // is empty.
    const ErrSink sink = make_sink(p);
    if (threadIdx.x == 0) {
        int b = call_aborted(p) ? 1 : 0;
        if (kPass2 && p.counters[2] == 0ull) b = 1;
        *bail = b;
    }
    __syncthreads();
    if (*bail) return;

    const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
    const bool rule_on = p.beta > 0 && p.sim_threshold < 1.0f;
    const unsigned long long total_items = kPass2 ? p.counters[2] : total_items_host;

    if (threadIdx.x == 0) {
        for (int s = 0; s < kItemSlots; ++s) {
            mbar_init(bar.at(kBarQFull + s), 1);
            mbar_init(bar.at(kBarQEmpty + s), 10);
        }
        for (int s = 0; s < 2; ++s) {
            // pass 1: TMA fills the resident tiles; pass 2: the 8 epilogue warps do; the MMA thread reads them
            mbar_init(bar.at(kBarAFull + s), kPass2 ? 8 : 1);
            mbar_init(bar.at(kBarAEmpty + s), 2);              // both MMA issuers
        }
        for (int s = 0; s < kStagesB; ++s) {
            mbar_init(bar.at(kBarBFull + s), 1);
            mbar_init(bar.at(kBarBEmpty + s), 2);              // both MMA issuers
        }
        for (int s = 0; s < 4; ++s) {
            mbar_init(bar.at(kBarAccFull + s), 1);
            mbar_init(bar.at(kBarAccEmpty + s), 4);
        }
        for (int s = 0; s < 2; ++s) {
            mbar_init(bar.at(kBarRFull + s), 1);
            mbar_init(bar.at(kBarREmpty + s), 8);
        }
        *abort_flag = 0;
        asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory");
    }
    if (warp == 1) {
        asm volatile("tcgen05.alloc.cta_group::1.sync.aligned.shared::cta.b32 [%0], %1;"
                     ::"r"(smem_u32(tmem_holder)), "r"(kTmemCols) : "memory");
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
            uint32_t k_item = 0, bcount = 0;
            bool ok = true;
            // the next ticket is drawn while the current item is set up (a block draws one ticket too many)
            unsigned long long next_ticket = atomicAdd(&p.counters[kPass2 ? 3 : 1], 1ull);
            while (ok) {
                const unsigned long long ticket = next_ticket;
                if (ticket >= total_items) break;
                next_ticket = atomicAdd(&p.counters[kPass2 ? 3 : 1], 1ull);
                int4 desc;
                int n_iter, first_tile, head;
                if (!kPass2) {
                    head = (int)(ticket / (unsigned)items_per_head);
                    const int pi = (int)(ticket % (unsigned)items_per_head);
                    const int n = candidates_from_meta(p.meta[head / p.hkv], p.budget, p.alpha);
                    if (n == 0 || pi * kRowsPerItem >= n) continue;             // nothing to score in this item
                    const int n_tiles = (n + kTile - 1) / kTile;
                    desc = make_int4(head, pi, n, 0);
                    first_tile = n_tiles - 1;                  // streamed tiles: first_tile .. max(2 pi, n_tiles - depth)
                    n_iter = 1 + (rule_on ? n_tiles - max(2 * pi, n_tiles - kPass1Depth) : 0);   // + the query rows
                } else {
                    desc = p.strag_items[ticket];          // {head, first listed token, tokens, first streamed tile}
                    head = desc.x;
                    first_tile = desc.w;                   // streamed tiles: first_tile .. 0
                    n_iter = first_tile + 1;
                }
                const int key_row_base = head * p.cap;                         // first row of the head in the 2-D key view

                const uint32_t qs = k_item % kItemSlots;
                if (!mbar_wait(bar.at(kBarQEmpty + qs), ((k_item / kItemSlots) & 1) ^ 1, abort_flag, sink)) break;
                items[qs] = desc;
                mbar_arrive(bar.at(kBarQFull + qs));

                if (kPass2 && p.beta > 1) {
                    // r_j of the tiles this item streams (0 .. first_tile), straight into shared memory
                    if (!mbar_wait(bar.at(kBarREmpty), (k_item & 1) ^ 1, abort_flag, sink)) break;
                    const uint32_t bytes = (uint32_t)(first_tile + 1) * kTile * 4u;
                    mbar_expect_tx(bar.at(kBarRFull), bytes);
                    asm volatile("cp.async.bulk.shared::cluster.global.mbarrier::complete_tx::bytes [%0], [%1], %2, [%3];"
                                 ::"r"(sbase + kOffRHead), "l"(p.inv_norm + (size_t)head * p.cap_pad), "r"(bytes),
                                   "r"(bar.at(kBarRFull))
                                 : "memory");
                }
                if (!kPass2 && rule_on) {
                    // r_j of the key tiles this item streams (first_tile down to first_tile + 2 - n_iter)
                    const uint32_t rb = k_item & 1;
                    if (!mbar_wait(bar.at(kBarREmpty + rb), ((k_item >> 1) & 1) ^ 1, abort_flag, sink)) break;
                    const int low_tile = first_tile + 2 - n_iter;
                    const uint32_t bytes = (uint32_t)(n_iter - 1) * kTile * 4u;
                    mbar_expect_tx(bar.at(kBarRFull + rb), bytes);
                    asm volatile("cp.async.bulk.shared::cluster.global.mbarrier::complete_tx::bytes [%0], [%1], %2, [%3];"
                                 ::"r"(sbase + kOffRj + rb * kPass1Depth * kTile * 4),
                                   "l"(p.inv_norm + (size_t)head * p.cap_pad + (size_t)low_tile * kTile), "r"(bytes),
                                   "r"(bar.at(kBarRFull + rb))
                                 : "memory");
                }
                if (!kPass2) {
                    const int row0 = desc.y * kRowsPerItem;
                    const int num_m = (desc.z - row0 > kTile) ? 2 : 1;
                    const uint32_t ab = k_item & 1;
                    if (!mbar_wait(bar.at(kBarAEmpty + ab), ((k_item >> 1) & 1) ^ 1, abort_flag, sink)) break;
                    mbar_expect_tx(bar.at(kBarAFull + ab), (uint32_t)(num_m * kTileBytes));
                    for (int m = 0; m < num_m; ++m) {
                        const uint32_t dst = sbase + kOffA + (ab * 2 + m) * kTileBytes;
                        const int y = key_row_base + row0 + m * kTile;
                        tma_load_2d(dst, &map_k, 0, y, bar.at(kBarAFull + ab));
                        tma_load_2d(dst + kHalfBytes, &map_k, 64, y, bar.at(kBarAFull + ab));
                    }
                }
                for (int it = 0; it < n_iter; ++it) {
                    const uint32_t s = bcount % kStagesB;
                    if (!mbar_wait(bar.at(kBarBEmpty + s), ((bcount / kStagesB) & 1) ^ 1, abort_flag, sink)) {
                        ok = false;
                        break;
                    }
                    const uint32_t dst = sbase + kOffB + s * kTileBytes;
                    if (!kPass2 && it == 0) {
                        const int b = head / p.hkv, h = head % p.hkv;
                        const int q_row = (b * p.hq + h * p.group) * p.alpha;
                        // the query rows, then 16 rows holding sum_j Kbar_j split into bf16 parts
                        mbar_expect_tx(bar.at(kBarBFull + s), (uint32_t)(2 * (q_rows_pad + 16) * 128));
                        tma_load_2d(dst, &map_q, 0, q_row, bar.at(kBarBFull + s));
                        tma_load_2d(dst + kHalfBytes, &map_q, 64, q_row, bar.at(kBarBFull + s));
                        tma_load_2d(dst + q_rows_pad * 128, &map_hs, 0, head * 16, bar.at(kBarBFull + s));
                        tma_load_2d(dst + kHalfBytes + q_rows_pad * 128, &map_hs, 64, head * 16, bar.at(kBarBFull + s));
                    } else {
                        const int jt = first_tile - (kPass2 ? it : it - 1);
                        const int y = key_row_base + jt * kTile;
                        mbar_expect_tx(bar.at(kBarBFull + s), kTileBytes + (kPass2 ? kSliceBytes : 0));
                        tma_load_2d(dst, &map_k, 0, y, bar.at(kBarBFull + s));
                        tma_load_2d(dst + kHalfBytes, &map_k, 64, y, bar.at(kBarBFull + s));
                        if (kPass2)     // the tile's extra slice: the norms of its keys in three bf16 parts
                            tma_load_2d(sbase + kOffAugB + s * kSliceBytes, &map_ns, 0, head * p.cap_pad + jt * kTile,
                                        bar.at(kBarBFull + s));
                    }
                    ++bcount;
                }
                ++k_item;
            }
            // terminator: tells the other roles that no item follows (skipped when the block is aborting)
            if (!*abort_flag) {
                const uint32_t qs = k_item % kItemSlots;
                if (mbar_wait(bar.at(kBarQEmpty + qs), ((k_item / kItemSlots) & 1) ^ 1, abort_flag, sink)) {
                    items[qs] = make_int4(-1, 0, 0, 0);
                    mbar_arrive(bar.at(kBarQFull + qs));
                }
            }
        }
        __syncwarp();
    } else if (warp == 1 || warp == 10) {
        // ------------------------------------------------------------------ MMA issuers
        // One thread per row tile of the item (warp 1: row tile 0, warp 10: row tile 1).  With a single issuer the
        // tensor pipe ran dry between tiles while the thread went through its barrier waits; two threads keep each
        // other's products queued.  Both wait for every stage and every item (which keeps either from running a
        // whole barrier phase ahead) and both release them: by a commit after products of their own, by a plain
        // arrival otherwise.
        if (lane == 0) {
            const int m = warp == 1 ? 0 : 1;
            const uint32_t idesc_k = instr_desc(kTile, kTile), idesc_q = instr_desc(kTile, q_rows_pad + 16);
            uint32_t k_item = 0, bcount = 0, cnt = 0;
            bool ok = true;
            while (ok) {
                const uint32_t qs = k_item % kItemSlots;
                if (!mbar_wait(bar.at(kBarQFull + qs), (k_item / kItemSlots) & 1, abort_flag, sink)) break;
                const int4 d = items[qs];
                mbar_arrive(bar.at(kBarQEmpty + qs));
                if (d.x < 0) break;
                int num_m, n_iter, skip_it;       // skip_it: the iteration whose row tile 1 would mirror row tile 0's
                if (!kPass2) {
                    const int n_tiles = (d.z + kTile - 1) / kTile;
                    num_m = (d.z - d.y * kRowsPerItem > kTile) ? 2 : 1;
                    n_iter = 1 + (rule_on ? n_tiles - max(2 * d.y, n_tiles - kPass1Depth) : 0);
                    // row tile 2p + 1 stops at its diagonal tile: it skips tile 2p if the item gets that far
                    skip_it = (2 * d.y >= n_tiles - kPass1Depth) ? n_iter - 1 : -1;
                } else {
                    num_m = d.z > kTile ? 2 : 1;
                    n_iter = d.w + 1;
                    skip_it = -1;
                }
                const bool mine = m < num_m;
                const uint32_t ab = kPass2 ? 0u : (k_item & 1);                          // pass 2: one pair of tiles
                const uint32_t a_par = kPass2 ? (k_item & 1) : ((k_item >> 1) & 1);
                if (!mbar_wait(bar.at(kBarAFull + ab), a_par, abort_flag, sink)) break;
                if (kPass2) asm volatile("tcgen05.fence::after_thread_sync;" ::: "memory");
                const uint32_t resident = sbase + kOffA + (ab * 2 + m) * kTileBytes;
                for (int it = 0; it < n_iter; ++it) {
                    const uint32_t s = bcount % kStagesB;
                    if (!mbar_wait(bar.at(kBarBFull + s), (bcount / kStagesB) & 1, abort_flag, sink)) {
                        ok = false;
                        break;
                    }
                    const uint32_t stage = sbase + kOffB + s * kTileBytes;
                    const bool is_q = !kPass2 && it == 0;
                    if (mine && !(m == 1 && it == skip_it && it > 0)) {
                        const uint32_t a = cnt & 1;
                        if (!mbar_wait(bar.at(kBarAccEmpty + a * 2 + m), ((cnt >> 1) & 1) ^ 1, abort_flag, sink)) {
                            ok = false;
                            break;
                        }
                        tc_fence_after();
                        const uint32_t d_tmem = tmem_base + a * 256 + m * 128;
                        umma_tile_k128(d_tmem, resident, stage, is_q ? idesc_q : idesc_k);
                        if (kPass2)     // ... - (T / r_i) (||k_j|| + eps): the accumulator's sign is the threshold test
                            umma_k16_sw32(d_tmem, sbase + kOffAugA + m * kSliceBytes, sbase + kOffAugB + s * kSliceBytes, idesc_k);
                        umma_commit(bar.at(kBarAccFull + a * 2 + m));
                        ++cnt;
                        if (!is_q) ++tiles_done;
                        umma_commit(bar.at(kBarBEmpty + s));      // the stage may be refilled once these products have read it
                    } else {
                        mbar_arrive(bar.at(kBarBEmpty + s));
                    }
                    ++bcount;
                }
                if (!ok) break;
                if (mine) umma_commit(bar.at(kBarAEmpty + ab));   // so may the resident tiles
                else mbar_arrive(bar.at(kBarAEmpty + ab));
                ++k_item;
            }
        }
        __syncwarp();
    } else {
        // ------------------------------------------------------------------ epilogue warps
        const int ew = warp - 2;                 // 0..7
        const int m = ew >> 2;                   // row tile of the item this warp serves
        const int quad = warp & 3;               // TMEM lane quadrant this warp may access
        const int lrow = quad * 32 + lane;       // row within the 128-row tile
        const uint32_t lane_base = tmem_base + ((uint32_t)(quad * 32) << 16);
        const float kInf = __int_as_float(0x7f800000);
        const float scale = 0.08838834764831845f;             // 1 / sqrt(128)
        const int G = p.group;
        uint32_t k_item = 0, cnt = 0;

        while (true) {
            const uint32_t qs = k_item % kItemSlots;
            if (!mbar_wait(bar.at(kBarQFull + qs), (k_item / kItemSlots) & 1, abort_flag, sink)) break;
            const int4 d = items[qs];
            __syncwarp();
            if (lane == 0) mbar_arrive(bar.at(kBarQEmpty + qs));
            if (d.x < 0) break;
            const int head = d.x;
            const float *inv_norm = p.inv_norm + (size_t)head * p.cap_pad;
            const uint32_t ab = kPass2 ? 0u : (k_item & 1);
            const uint32_t a_par = kPass2 ? (k_item & 1) : ((k_item >> 1) & 1);

            // ---- per item: which token this thread owns, its threshold, where its scan starts and ends
            bool active, row_ok, item_ok = true;
            int i, first_tile, my_last_tile, own_tile;
            float ri, self = 0.f, total = 0.f;
            int left = 0;
            if (!kPass2) {
                const int pi = d.y, n = d.z;
                const int row0 = pi * kRowsPerItem;
                active = (m == 0) || (n - row0 > kTile);
                i = row0 + m * kTile + lrow;
                row_ok = active && i < n;
                ri = row_ok ? __ldg(inv_norm + i) : 0.f;
                self = row_ok ? __ldg(p.self_dot + (size_t)head * p.cap_pad + i) : 0.f;
                first_tile = (n + kTile - 1) / kTile - 1;                 // first streamed tile
                my_last_tile = max(2 * pi + m, first_tile + 1 - kPass1Depth);   // where this row tile's scan stops
                own_tile = 0x7fffffff;                                    // pass 1: every streamed tile takes part
                left = row_ok ? p.beta : 0;
            } else {
                const int k0 = d.y, rows = d.z;
                active = (m == 0) || (rows > kTile);
                const int k = k0 + m * kTile + lrow;
                row_ok = active && (m * kTile + lrow) < rows;
                i = row_ok ? p.strag[(size_t)head * p.cap_pad + k] : 0;
                ri = row_ok ? __ldg(inv_norm + i) : 0.f;
                {
                    const int n = candidates_from_meta(p.meta[head / p.hkv], p.budget, p.alpha);
                    // pass 1 scanned the token down to tile max(its own, n_tiles - depth): it takes part below that
                    own_tile = row_ok ? max(i / kTile, (n + kTile - 1) / kTile - kPass1Depth) : 0;
                }
                first_tile = d.w;
                my_last_tile = 0;
                left = row_ok ? p.left[(size_t)head * p.cap_pad + i] : 0;

                // gather this thread's key row into the resident tile (same swizzled layout as a TMA load); every
                // warp waits and arrives, also one without rows of its own, so that no arrival runs ahead
                item_ok = mbar_wait(bar.at(kBarAEmpty + ab), a_par ^ 1, abort_flag, sink);
                if (active && item_ok) {
                    uint8_t *tile = smem + kOffA + (ab * 2 + m) * kTileBytes;
                    const uint4 *src = reinterpret_cast<const uint4 *>(
                        static_cast<const __nv_bfloat16 *>(p.k_cache) + ((size_t)head * p.cap + i) * kHeadDim);
#pragma unroll
                    for (int hb = 0; hb < 2; ++hb) {
#pragma unroll
                        for (int c = 0; c < 8; ++c) {
                            const uint4 v = row_ok ? __ldg(src + hb * 8 + c) : make_uint4(0u, 0u, 0u, 0u);
                            *reinterpret_cast<uint4 *>(tile + hb * kHalfBytes + lrow * 128 + ((c ^ (lrow & 7)) << 4)) = v;
                        }
                    }
                    {
                        // the row's extra slice: -T / r_i in three bf16 parts as (-t1, -t1, -t1, -t2, -t2, -t3, 0 ...),
                        // which meets (n1, n2, n3, n1, n2, n1, 0 ...) of a key; 32-byte rows, 32-byte swizzle
                        float rest = (row_ok && ri > 0.f) ? -__fdiv_rn(p.sim_threshold, ri) : 0.f;
                        uint32_t part[3];
#pragma unroll
                        for (int c = 0; c < 3; ++c) {
                            const __nv_bfloat16 h16 = __float2bfloat16_rn(rest);
                            part[c] = (uint32_t)__bfloat16_as_ushort(h16);
                            rest -= __bfloat162float(h16);
                        }
                        uint8_t *slice = smem + kOffAugA + m * kSliceBytes + lrow * 32;
                        const int sw = (lrow >> 2) & 1;
                        *reinterpret_cast<uint4 *>(slice + (sw << 4)) =
                            make_uint4(part[0] | (part[0] << 16), part[0] | (part[1] << 16), part[1] | (part[2] << 16), 0u);
                        *reinterpret_cast<uint4 *>(slice + ((sw ^ 1) << 4)) = make_uint4(0u, 0u, 0u, 0u);
                    }
                    asm volatile("fence.proxy.async.shared::cta;" ::: "memory");   // generic writes -> tensor-core reads
                }
                __syncwarp();
                if (lane == 0) mbar_arrive(bar.at(kBarAFull + ab));
            }

            const bool scan = active && (kPass2 || rule_on);
            // r_j of the first key tile of the scan: loaded now, staged in shared memory when the tile is drained
            const bool has_r = kPass2 ? p.beta > 1 : rule_on;
            const uint32_t r_slot = kPass2 ? 0u : (k_item & 1), r_par = kPass2 ? (k_item & 1) : ((k_item >> 1) & 1);
            if (has_r) {        // every warp waits for the item's r_j, and hands them back at the item's end
                const bool r_ok = mbar_wait(bar.at(kBarRFull + r_slot), r_par, abort_flag, sink);
                item_ok = item_ok && r_ok;
            }

            if (!kPass2 && active) {
                const uint32_t a = cnt & 1;
                item_ok = mbar_wait(bar.at(kBarAccFull + a * 2 + m), (cnt >> 1) & 1, abort_flag, sink);
            }
            if (!kPass2 && active && item_ok) {
                // ---- iteration 0, Eq. 2-3: thread = key, all G * alpha logits of that key in its accumulator row,
                // followed by k_i . s in three parts
                const uint32_t a = cnt & 1;
                tc_fence_after();
                const uint32_t qbase = lane_base + a * 256 + m * 128;
                float *logits = p.logits + (size_t)head * p.alpha * p.cap_pad;
                uint32_t sp[8];
                tmem_ld8(qbase + q_rows_pad, sp);
                if (p.alpha == 8) {
                    float best[8];
#pragma unroll
                    for (int j = 0; j < 8; ++j) best[j] = p.gqa_mean_pool ? 0.f : -kInf;
                    for (int g0 = 0; g0 < G; g0 += 2) {
                        uint32_t t0[8], t1[8];
                        tmem_ld8(qbase + g0 * 8, t0);
                        tmem_ld8(qbase + min(g0 + 1, G - 1) * 8, t1);     // an odd G reads its last head twice
                        tmem_wait8(t0);
                        tmem_wait8(t1);
                        if (p.gqa_mean_pool) {        // the variant: sum over the group (scaled to the mean below)
                            const bool both = g0 + 1 < G;
#pragma unroll
                            for (int j = 0; j < 8; ++j)
                                best[j] += __uint_as_float(t0[j]) + (both ? __uint_as_float(t1[j]) : 0.f);
                            continue;
                        }
#pragma unroll
                        for (int j = 0; j < 8; ++j)
                            best[j] = fmaxf(best[j], fmaxf(__uint_as_float(t0[j]), __uint_as_float(t1[j])));
                    }
                    const float scale_q = p.gqa_mean_pool ? scale / (float)G : scale;
                    tmem_wait8(sp);
                    tc_fence_before();
                    __syncwarp();
                    if (lane == 0) mbar_arrive(bar.at(kBarAccEmpty + a * 2 + m));
                    if (row_ok) {
#pragma unroll
                        for (int j = 0; j < 8; ++j) logits[(size_t)j * p.cap_pad + i] = best[j] * scale_q;
                    }
                } else {
                    for (int j = 0; j < p.alpha; ++j) {
                        float best = -kInf, sum = 0.f;
                        for (int g0 = 0; g0 < G; g0 += 4) {
                            uint32_t t[4];
#pragma unroll
                            for (int u = 0; u < 4; ++u) tmem_ld1(qbase + min(g0 + u, G - 1) * p.alpha + j, t[u]);
                            asm volatile("tcgen05.wait::ld.sync.aligned;"
                                         : "+r"(t[0]), "+r"(t[1]), "+r"(t[2]), "+r"(t[3]) :: "memory");
#pragma unroll
                            for (int u = 0; u < 4; ++u) {
                                best = fmaxf(best, __uint_as_float(t[u]));
                                sum += (g0 + u < G) ? __uint_as_float(t[u]) : 0.f;
                            }
                        }
                        if (row_ok)
                            logits[(size_t)j * p.cap_pad + i] = p.gqa_mean_pool ? sum * scale / (float)G : best * scale;
                    }
                    tmem_wait8(sp);
                    tc_fence_before();
                    __syncwarp();
                    if (lane == 0) mbar_arrive(bar.at(kBarAccEmpty + a * 2 + m));
                }
                // sum_j S[j][i] before the retention rule: Kbar_i . s - Kbar_i . Kbar_i
                total = ri * ((__uint_as_float(sp[0]) + __uint_as_float(sp[1])) + __uint_as_float(sp[2])) - self;
                ++cnt;
            }

            float removed = 0.f;
            // pass 2: how many partners were found; with beta = 1 the one partner's position and accumulator value
            int nhit = 0, hit_j = -1;
            float hit_h = 0.f;
            if (scan) {
                // ---- key tiles, last to first; their r_j lie in shared memory
                const float thr = (row_ok && ri > 0.f) ? __fdiv_rn(p.sim_threshold, ri) : kInf;   // g r_j vs T / r_i
                // pass 2: the whole head from tile 0; pass 1: the item's tiles from its lowest one (that of row tile 0)
                // pass 1: the r_j of the item's tiles in shared memory; pass 2: the head's (there only with beta > 1,
                // and read for the chunks with partners only)
                const float *r_base = kPass2 ? reinterpret_cast<const float *>(smem + kOffRHead)
                                             : reinterpret_cast<const float *>(smem + kOffRj) + (k_item & 1) * kPass1Depth * kTile -
                                                   (size_t)max(2 * d.y, first_tile + 1 - kPass1Depth) * kTile;
                bool ok = item_ok;
                for (int jt = first_tile; jt >= my_last_tile; --jt) {
                    const int jbase = jt * kTile;
                    const float4 *rj4 = reinterpret_cast<const float4 *>(r_base + jbase);
                    const uint32_t a = cnt & 1;
                    if (ok) ok = mbar_wait(bar.at(kBarAccFull + a * 2 + m), (cnt >> 1) & 1, abort_flag, sink);
                    ++cnt;
                    if (!ok) continue;
                    tc_fence_after();
                    const uint32_t base = lane_base + a * 256 + m * 128;
                    // +inf once the token has its beta partners, and (pass 2) while the scan is still in pass 1's part
                    float thr_row = (left > 0 && jt < own_tile) ? thr : kInf;
                    if (__any_sync(0xffffffffu, thr_row < kInf)) {
                        // 32-column chunks, last first.  The loop is kept rolled on purpose: ten warps in three roles
                        // share the instruction cache, and one copy of this body is what fits.
#pragma unroll 1
                        for (int ch = 3; ch >= 0; --ch) {
                            uint32_t g[32];
                            tmem_ld32(base + ch * 32, g);
                            float v[32];
                            uint32_t hits = 0u;
                            if (kPass2) {
                                // The accumulator holds h = k_i . k_j - (T / r_i) (||k_j|| + eps): S[j][i] > T exactly
                                // when h > 0, so the screening is a maximum and a sign test, with nothing to load
                                // per column (the loads of the r_j were what this epilogue's time went into: every
                                // byte a thread receives, from TMEM or as a shared-memory broadcast, passes through
                                // the same return path).  The listed tokens rarely have a partner in a given chunk.
                                tmem_wait32(g);
#pragma unroll
                                for (int c = 0; c < 32; ++c) v[c] = __uint_as_float(g[c]);
                                float m0 = 0.f, m1 = 0.f;
#pragma unroll
                                for (int c = 0; c < 32; c += 4) {
                                    m0 = max3(m0, v[c], v[c + 1]);
                                    m1 = max3(m1, v[c + 2], v[c + 3]);
                                }
                                const float cut = thr_row < kInf ? 0.f : kInf;
                                if (!__any_sync(0xffffffffu, fmaxf(m0, m1) > cut)) continue;
#pragma unroll
                                for (int c = 0; c < 32; ++c) hits |= (v[c] > cut) ? (1u << c) : 0u;
                            } else {
                            float4 R[8];
#pragma unroll
                            for (int q = 0; q < 8; ++q) R[q] = rj4[ch * 8 + q];
                            tmem_wait32(g);
#pragma unroll
                            for (int q = 0; q < 8; ++q) {        // packed multiplies: two products per instruction
                                const float2 p0 = __fmul2_rn(make_float2(__uint_as_float(g[4 * q]), __uint_as_float(g[4 * q + 1])),
                                                             make_float2(R[q].x, R[q].y));
                                const float2 p1 = __fmul2_rn(make_float2(__uint_as_float(g[4 * q + 2]), __uint_as_float(g[4 * q + 3])),
                                                             make_float2(R[q].z, R[q].w));
                                v[4 * q] = p0.x;
                                v[4 * q + 1] = p0.y;
                                v[4 * q + 2] = p1.x;
                                v[4 * q + 3] = p1.y;
                            }
                            // some token of the warp has partners in this chunk: a bit mask of the entries above the
                            // threshold (no entry depends on another), cut down to the highest positions if they are
                            // more than the token still lacks, then their sum
#pragma unroll
                            for (int c = 0; c < 32; ++c) hits |= (v[c] > thr_row) ? (1u << c) : 0u;
                            }
                            const unsigned own = (unsigned)(i - (jbase + ch * 32));           // zero diagonal (Eq. 5)
                            if (own < 32u) hits &= ~(1u << own);
                            if (p.beta == 1) {
                                // one partner at most: the entry at the highest set bit, picked by a select tree
                                if (left > 0 && hits != 0u) {
                                    const int top = 31 - __clz(hits);
                                    float t16[16], t8[8], t4[4];
#pragma unroll
                                    for (int c = 0; c < 16; ++c) t16[c] = (top & 16) ? v[16 + c] : v[c];
#pragma unroll
                                    for (int c = 0; c < 8; ++c) t8[c] = (top & 8) ? t16[8 + c] : t16[c];
#pragma unroll
                                    for (int c = 0; c < 4; ++c) t4[c] = (top & 4) ? t8[4 + c] : t8[c];
                                    const float u0 = (top & 2) ? t4[2] : t4[0], u1 = (top & 2) ? t4[3] : t4[1];
                                    if (kPass2) {      // its r_j is fetched once, at the item's end
                                        hit_h = (top & 1) ? u1 : u0;
                                        hit_j = jbase + ch * 32 + top;
                                    } else {
                                        removed += (top & 1) ? u1 : u0;
                                    }
                                    left = 0;
                                    thr_row = kInf;
                                }
                                continue;
                            }
                            int taken = __popc(hits);
                            for (; taken > left; --taken) hits &= hits - 1u;                   // drop the lowest positions
                            if (kPass2) {
                                // S = T + h r_i r_j per partner
                                nhit += taken;
#pragma unroll
                                for (int q = 0; q < 8; ++q) {
                                    const float4 R = rj4[ch * 8 + q];
                                    v[4 * q] *= R.x;
                                    v[4 * q + 1] *= R.y;
                                    v[4 * q + 2] *= R.z;
                                    v[4 * q + 3] *= R.w;
                                }
                            }
                            float s0 = 0.f, s1 = 0.f, s2 = 0.f, s3 = 0.f;
#pragma unroll
                            for (int c = 0; c < 32; c += 4) {
                                s0 += (hits >> c & 1u) ? v[c] : 0.f;
                                s1 += (hits >> (c + 1) & 1u) ? v[c + 1] : 0.f;
                                s2 += (hits >> (c + 2) & 1u) ? v[c + 2] : 0.f;
                                s3 += (hits >> (c + 3) & 1u) ? v[c + 3] : 0.f;
                            }
                            removed += (s0 + s1) + (s2 + s3);
                            left -= taken;
                            if (left == 0) thr_row = kInf;
                        }
                        tc_fence_before();
                        __syncwarp();
                        if (lane == 0) mbar_arrive(bar.at(kBarAccEmpty + a * 2 + m));
                    } else {
                        tc_fence_before();
                        __syncwarp();
                        if (lane == 0) mbar_arrive(bar.at(kBarAccEmpty + a * 2 + m));
                    }
                }
                item_ok = ok;
            }
            if (has_r) {
                __syncwarp();
                if (lane == 0) mbar_arrive(bar.at(kBarREmpty + r_slot));
            }
            if (!item_ok) break;              // (the epilogue warps meet at no barrier of their own: each may leave alone)
            if (row_ok) {
                float *out = p.sbar + (size_t)head * p.cap_pad + i;
                if (!kPass2) {
                    *out = total - removed * ri;
                    p.left[(size_t)head * p.cap_pad + i] = rule_on ? left : 0;
                    if (rule_on) {
                        // for pass 2: 1 / r_i = ||k_i|| + eps as three bf16 parts (their sum has fp32 accuracy), laid
                        // out as the extra K = 16 slice of a key row, (n1, n2, n3, n1, n2, n1, 0 ...): its dot product
                        // with a token's (-t1, -t1, -t1, -t2, -t2, -t3, 0 ...) is -t / r_i up to terms of size 2^-24
                        float rest = ri > 0.f ? __fdiv_rn(1.0f, ri) : 0.f;
                        uint32_t part[3];
#pragma unroll
                        for (int c = 0; c < 3; ++c) {
                            const __nv_bfloat16 h16 = __float2bfloat16_rn(rest);
                            part[c] = (uint32_t)__bfloat16_as_ushort(h16);
                            rest -= __bfloat162float(h16);
                        }
                        uint4 *dst = reinterpret_cast<uint4 *>(p.norm_split + ((size_t)head * p.cap_pad + i) * 16);
                        dst[0] = make_uint4(part[0] | (part[1] << 16), part[2] | (part[0] << 16), part[1] | (part[0] << 16), 0u);
                        dst[1] = make_uint4(0u, 0u, 0u, 0u);
                    }
                } else {
                    // S = T + h r_i r_j for every partner found here
                    if (p.beta == 1 && hit_j >= 0) {
                        removed = hit_h * __ldg(inv_norm + hit_j);
                        nhit = 1;
                    }
                    *out -= (float)nhit * p.sim_threshold + removed * ri;
                }
            }
            ++k_item;
        }
    }

    // ---------------------------------------------------------------------- common exit
    tc_fence_before();
    __syncthreads();
    if (warp == 1) {
        if (*abort_flag) __nanosleep(200000);      // error path only: let copies and MMAs in flight land
        tc_fence_after();
        asm volatile("tcgen05.dealloc.cta_group::1.sync.aligned.b32 %0, %1;" ::"r"(tmem_base), "r"(kTmemCols) : "memory");
    }
    if ((warp == 1 || warp == 10) && lane == 0 && !*abort_flag && tiles_done) atomicAdd(p.counters, tiles_done);
}

// ---- between the passes: list, per head, the tokens still short of partners with positions not yet looked at -----
constexpr int kCompactThreads = 256;

__global__ void __launch_bounds__(kCompactThreads) strag_compact_kernel(Params p)
{
    __shared__ int warp_tot[kCompactThreads / 32];
    __shared__ int running;
    const int head = blockIdx.x;
    const int n = candidates_from_meta(p.meta[head / p.hkv], p.budget, p.alpha);
    const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
    const int32_t *left = p.left + (size_t)head * p.cap_pad;
    int32_t *list = p.strag + (size_t)head * p.cap_pad;
    if (threadIdx.x == 0) running = 0;
    __syncthreads();
    const int low = (n + kTile - 1) / kTile - kPass1Depth;    // pass 1 scanned every token down to this tile at least
    for (int i0 = 0; i0 < n; i0 += kCompactThreads) {
        const int i = i0 + threadIdx.x;
        const bool want = i < n && left[i] > 0 && max(i / kTile, low) >= 1;   // something is left below pass 1's part
        const unsigned bal = __ballot_sync(0xffffffffu, want);
        if (lane == 0) warp_tot[warp] = __popc(bal);
        __syncthreads();
        int before = running;
        for (int w = 0; w < warp; ++w) before += warp_tot[w];
        if (want) list[before + __popc(bal & ((1u << lane) - 1u))] = i;
        __syncthreads();
        if (threadIdx.x == 0) {
            int t = 0;
            for (int w = 0; w < kCompactThreads / 32; ++w) t += warp_tot[w];
            running += t;
        }
        __syncthreads();
    }
    if (threadIdx.x == 0) {
        const int count = running;
        p.strag_count[head] = count;
        const int chunks = (count + kRowsPerItem - 1) / kRowsPerItem;
        if (chunks > 0) {
            const unsigned long long at = atomicAdd(&p.counters[2], (unsigned long long)chunks);
            // complete item descriptors, longest scans (largest positions) first: pass 1 took the chunk's last token
            // down to tile max(its own, n_tiles - depth), so the chunk's scan starts one tile below that
            unsigned long long pairs = 0ull;
            for (int q = 0; q < chunks; ++q) {
                const int c = chunks - 1 - q, k0 = c * kRowsPerItem, rows = min(count - k0, kRowsPerItem);
                const int first_tile = max(list[k0 + rows - 1] / kTile, low) - 1;     // >= 0 for every listed token
                p.strag_items[at + q] = make_int4(head, k0, rows, first_tile);
                pairs += (unsigned long long)rows * (unsigned long long)(first_tile + 1);
            }
            atomicAdd(&p.counters[kPairsWord], pairs);      // listed tokens x key tiles: the work pass 2 cannot avoid
        }
    }
}

}  // namespace

cudaError_t launch_scores_tri_sm100(const Params &p, cudaStream_t s)
{
    const int q_rows = p.group * p.alpha;
    const int q_rows_pad = (q_rows + 15) / 16 * 16;
    CUtensorMap map_k, map_q, map_hs, map_ns;
    if (!make_map(&map_k, p.k_cache, (uint64_t)p.batch * p.hkv * p.cap, kTile) ||
        !make_map(&map_q, p.q_window, (uint64_t)p.batch * p.hq * p.alpha, (uint32_t)q_rows_pad) ||
        !make_map(&map_hs, p.head_sum_bf16, (uint64_t)p.batch * p.hkv * 16, 16u) ||
        !make_map_k16(&map_ns, p.norm_split, (uint64_t)p.batch * p.hkv * p.cap_pad))
        return cudaErrorInvalidValue;
    cudaError_t e;
    if ((e = cudaFuncSetAttribute(scores_tri_sm100_kernel<false>, cudaFuncAttributeMaxDynamicSharedMemorySize,
                                  kSmemBytes)) != cudaSuccess ||
        (e = cudaFuncSetAttribute(scores_tri_sm100_kernel<true>, cudaFuncAttributeMaxDynamicSharedMemorySize,
                                  kSmemBytes)) != cudaSuccess)
        return e;
    int dev = 0, sms = 0;
    if ((e = cudaGetDevice(&dev)) != cudaSuccess) return e;
    if ((e = cudaDeviceGetAttribute(&sms, cudaDevAttrMultiProcessorCount, dev)) != cudaSuccess) return e;
    const int heads = p.batch * p.hkv;
    const int items_per_head = (p.tiles + 1) / 2;
    const unsigned long long total_items = (unsigned long long)items_per_head * (unsigned long long)heads;
    const unsigned grid1 = (unsigned)(total_items < (unsigned long long)sms ? total_items : (unsigned long long)sms);
    (void)grid1;
    if ((e = launch_scores_pass1_sm100(p, s, map_k, map_q, map_hs, q_rows_pad, sms)) != cudaSuccess) return e;
    if ((e = mark_kernel(p, 0, s)) != cudaSuccess) return e;
    const bool rule_on = p.beta > 0 && p.sim_threshold < 1.0f;
    if (!rule_on || p.tiles < 2) return mark_kernel(p, 1, s);       // nobody can lack partners / pass 1 has seen everything
    strag_compact_kernel<<<(unsigned)heads, kCompactThreads, 0, s>>>(p);
    if ((e = cudaGetLastError()) != cudaSuccess) return e;
    if ((e = mark_kernel(p, 1, s)) != cudaSuccess) return e;
    const unsigned long long max_items2 = (unsigned long long)heads * (unsigned long long)(p.cap_pad / kRowsPerItem + 1);
    const unsigned grid2 = (unsigned)(max_items2 < (unsigned long long)sms ? max_items2 : (unsigned long long)sms);
    scores_tri_sm100_kernel<true><<<grid2, kThreads, kSmemBytes, s>>>(p, map_k, map_q, map_hs, map_ns, 0, 0ull, q_rows_pad);
    return cudaGetLastError();
}

}  // namespace rkv

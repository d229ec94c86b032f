// Stage "scores", second pass, for bf16 caches: the tokens that the first pass (rkv_scores_p1_sm100.cu) left short
// of partners against the key tiles BELOW the last one, last to first.  tcgen05.mma with TMEM accumulators, fed by
// TMA, one persistent block per SM.
//
// Section 3.3's rule needs, per token i, the beta LARGEST positions j with S[j][i] > T.  S is symmetric before the
// rule, so token i's line can be read as row i, and a scan from the last position downwards turns the rule into "the
// first beta hits".  The first pass scans every token against the last key tile; where similar keys are common that
// settles most tokens.  The rest is done here, in ROUNDS:
//
//   list    The tokens with left > 0 are listed per head, ascending, in chunks of 256 (strag_compact_kernel).
//   scan    Work item = (head, chunk of 256 listed tokens, window of key tiles): the chunk's key rows are gathered
//           into two resident operand tiles by the epilogue warps; the window's key tiles stream through a ring, last
//           to first.  The removed entries are subtracted from what the first pass stored, `left` is updated.
//
// The first round's window is a few tiles only (kRoundTiles); the tokens that found their partners in it drop out of the next
// round's list, so the long scan down to tile 0 is paid only by the few tokens that have no partner at all (a
// single-round scan would drag every listed token of a chunk along with them).  The last round's window reaches
// tile 0.  Worst case (no pair above T): the rounds together form the whole matrix below the last tile.
//
// Every tile product carries one extra K = 16 step that folds the threshold test into the accumulator (see the
// epilogue): the screening is a maximum and a sign test with nothing to load per column.  The n x n matrix never
// leaves TMEM, and no atomics or global flags are involved in the scores.
//
// Items are handed out by a global ticket counter, longest first within a head, so neighbouring blocks work on
// the same head while its keys are in L2.
// Warp roles (512 threads): warp 15 = tickets (publishes item descriptors up to three items ahead), warps 11..14 =
// gather (fill the resident tiles of the NEXT item while the current one is scanned: two buffers), warp 0 = TMA
// producer of the streamed key tiles, warp 1 = MMA issuer of row tile 0 and TMEM owner, warp 10 = MMA issuer of row
// tile 1, warps 2..9 = epilogue (warp w may touch TMEM lanes 32 (w % 4) .. +31; warps 2-5 serve row tile 0, warps 6-9
// row tile 1).
// TMEM: four 128-column fp32 accumulators, two per row tile, so the tensor pipe fills one while the epilogue
// drains the other.  Every wait on an mbarrier is bounded; on expiry the block records RKV_ERR_TIMEOUT, stops
// issuing work and leaves through the common exit that frees TMEM.  No TMA multicast and no cluster launch.
#include "rkv_sm100.cuh"

namespace rkv {

namespace {

using namespace sm100;

constexpr int kThreads = 512;                    // 16 warps: producer, 2 MMA issuers (warps 1 and 10), 8 epilogue, 4 gather, tickets
constexpr int kGatherWarp0 = 11;                 // first of the 4 gather warps
constexpr int kTicketWarp = 15;                  // draws the items and publishes their descriptors, up to three items ahead
constexpr int kStagesB = 2;                      // ring depth of streamed tiles
constexpr int kItemSlots = 4;                    // ring depth of item descriptors
constexpr int kHalfBytes = kTile * 64 * 2;       // one TMA box: 128 rows x 64 bf16 (128-byte swizzled rows)
constexpr int kTileBytes = 2 * kHalfBytes;       // 32 KB: a 128 x 128 bf16 operand tile
constexpr int kRowsPerItem = 2 * kTile;
constexpr uint32_t kTmemCols = 512;
constexpr int kPass1Depth = 1;                   // key tiles every token is scanned against in the first pass
constexpr int kRoundWords = 8;                   // Params::counters[kRoundWords + 2 r], [.. + 1]: items and ticket of round r

// shared memory carve-up (offsets from a 1024-byte aligned base)
constexpr int kOffA = 0;                                   // 2 buffers x 2 resident tiles (the gathered rows of an item)
constexpr int kOffB = kOffA + 2 * 2 * kTileBytes;          // kStagesB streamed tiles
// The extra K = 16 slices of the operands: 128 rows x 32 bytes each (32-byte swizzle), one per resident tile and one
// per stage of the ring.
constexpr int kSliceBytes = kTile * 32;
constexpr int kOffAugA = kOffB + kStagesB * kTileBytes;    // 2 buffers x 2 slices
constexpr int kOffAugB = kOffAugA + 2 * 2 * kSliceBytes;   // kStagesB slices
// what the epilogue needs to know about an item's tokens, left by the gather warps: position, r_i, partners lacking
constexpr int kOffStash = kOffAugB + kStagesB * kSliceBytes;            // 2 buffers x 3 arrays x kRowsPerItem words
constexpr int kOffBar = kOffStash + 2 * 3 * kRowsPerItem * 4;           // mbarriers
enum {
    kBarQFull = 0,                          // [kItemSlots] item descriptor written
    kBarQEmpty = kBarQFull + kItemSlots,    // [kItemSlots] read by the producer, the 2 MMA threads, the 8 epilogue and the 4 gather warps
    kBarAFull = kBarQEmpty + kItemSlots,    // [2] resident tiles, slices and stash of the item in place (4 gather warps)
    kBarAEmpty = kBarAFull + 2,             // [2] ... no longer read (2 MMA threads, 8 epilogue warps)
    kBarBFull = kBarAEmpty + 2,             // [kStagesB]
    kBarBEmpty = kBarBFull + kStagesB,      // [kStagesB]
    kBarAccFull = kBarBEmpty + kStagesB,    // [2 buffers][2 row tiles]
    kBarAccEmpty = kBarAccFull + 4,         // [2][2], 4 warps each
    kNumBars = kBarAccEmpty + 4
};
constexpr int kOffItems = kOffBar + kNumBars * 8;          // kItemSlots x int4
constexpr int kOffMisc = kOffItems + kItemSlots * 16;      // tmem base, abort flag, bail flag
constexpr int kSmemBytes = kOffMisc + 16 + 1024;           // + slack for the manual 1024-byte alignment
static_assert(kOffItems % 16 == 0, "item descriptors are read as int4");
static_assert(kSmemBytes <= 227 * 1024, "shared memory budget");

struct Bars {
    uint32_t bar0;
    __device__ __forceinline__ uint32_t at(int idx) const { return bar0 + 8 * idx; }
};

// Item descriptor (int4): {head, first listed token k0, tokens in the item (1..256) | key tiles of the window << 16,
// first (highest) streamed tile}.  x < 0: no more items.  `round` selects the round's counters.
__global__ void __launch_bounds__(kThreads, 1)
scores_pass2_sm100_kernel(Params p, const __grid_constant__ CUtensorMap map_k, const __grid_constant__ CUtensorMap map_ns,
                          int round)
{
    unsigned long long *const item_count = p.counters + kRoundWords + 2 * round, *const ticket = item_count + 1;
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
        if (*item_count == 0ull) b = 1;
        *bail = b;
    }
    __syncthreads();
    if (*bail) return;

    const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
    const unsigned long long total_items = *item_count;

    if (threadIdx.x == 0) {
        for (int s = 0; s < kItemSlots; ++s) {
            mbar_init(bar.at(kBarQFull + s), 1);
            mbar_init(bar.at(kBarQEmpty + s), 15);
        }
        for (int s = 0; s < 2; ++s) {
            // the 4 gather warps fill the resident tiles; the MMA threads and the epilogue warps read them and the stash
            mbar_init(bar.at(kBarAFull + s), 4);
            mbar_init(bar.at(kBarAEmpty + s), 10);
        }
        for (int s = 0; s < kStagesB; ++s) {
            mbar_init(bar.at(kBarBFull + s), 1);
            mbar_init(bar.at(kBarBEmpty + s), 2);              // both MMA issuers
        }
        for (int s = 0; s < 4; ++s) {
            mbar_init(bar.at(kBarAccFull + s), 1);
            mbar_init(bar.at(kBarAccEmpty + s), 4);
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
        // ------------------------------------------------------------------ TMA producer
        if (lane == 0) {
            uint32_t k_item = 0, bcount = 0;
            bool ok = true;
            while (ok) {
                const uint32_t qs = k_item % kItemSlots;
                if (!mbar_wait(bar.at(kBarQFull + qs), (k_item / kItemSlots) & 1, abort_flag, sink)) break;
                const int4 desc = items[qs];            // {head, first listed token, tokens | window, first streamed tile}
                mbar_arrive(bar.at(kBarQEmpty + qs));
                if (desc.x < 0) break;
                const int head = desc.x;
                const int first_tile = desc.w;             // streamed tiles: first_tile .. first_tile - n_iter + 1
                const int n_iter = desc.z >> 16;
                for (int it = 0; it < n_iter; ++it) {
                    const uint32_t s = bcount % kStagesB;
                    if (!mbar_wait(bar.at(kBarBEmpty + s), ((bcount / kStagesB) & 1) ^ 1, abort_flag, sink)) {
                        ok = false;
                        break;
                    }
                    const uint32_t dst = sbase + kOffB + s * kTileBytes;
                    const int jt = first_tile - it;
                    const int y = (int)tile_row0(p, head, jt);
                    mbar_expect_tx(bar.at(kBarBFull + s), kTileBytes + kSliceBytes);
                    tma_load_2d(dst, &map_k, 0, y, bar.at(kBarBFull + s));
                    tma_load_2d(dst + kHalfBytes, &map_k, 64, y, bar.at(kBarBFull + s));
                    // the tile's extra slice: the norms of its keys in three bf16 parts
                    tma_load_2d(sbase + kOffAugB + s * kSliceBytes, &map_ns, 0, head * p.cap_pad + jt * kTile,
                                bar.at(kBarBFull + s));
                    ++bcount;
                }
                ++k_item;
            }
        }
        __syncwarp();
    } else if (warp == kTicketWarp) {
        // ------------------------------------------------------------------ tickets
        // Items are published as soon as a descriptor slot is free, so the gather warps learn of the next item while
        // the producer is still streaming the key tiles of the current one.
        if (lane == 0) {
            uint32_t k_item = 0;
            while (true) {
                const unsigned long long cur = atomicAdd(ticket, 1ull);
                if (cur >= total_items) break;
                const int4 desc = p.strag_items[cur];
                const uint32_t qs = k_item % kItemSlots;
                if (!mbar_wait(bar.at(kBarQEmpty + qs), ((k_item / kItemSlots) & 1) ^ 1, abort_flag, sink)) break;
                items[qs] = desc;
                mbar_arrive(bar.at(kBarQFull + qs));
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
            const uint32_t idesc_k = instr_desc(kTile, kTile);
            uint32_t k_item = 0, bcount = 0, cnt = 0;
            bool ok = true;
            while (ok) {
                const uint32_t qs = k_item % kItemSlots;
                if (!mbar_wait(bar.at(kBarQFull + qs), (k_item / kItemSlots) & 1, abort_flag, sink)) break;
                const int4 d = items[qs];
                mbar_arrive(bar.at(kBarQEmpty + qs));
                if (d.x < 0) break;
                const int num_m = (d.z & 0xffff) > kTile ? 2 : 1;
                const int n_iter = d.z >> 16;
                const bool mine = m < num_m;
                const uint32_t ab = k_item & 1;                  // resident buffer of this item
                if (!mbar_wait(bar.at(kBarAFull + ab), (k_item >> 1) & 1, abort_flag, sink)) break;     // the gathered rows are in place
                asm volatile("tcgen05.fence::after_thread_sync;" ::: "memory");
                const uint32_t resident = sbase + kOffA + (ab * 2 + m) * kTileBytes;
                const uint32_t res_slice = sbase + kOffAugA + (ab * 2 + m) * kSliceBytes;
                for (int it = 0; it < n_iter; ++it) {
                    const uint32_t s = bcount % kStagesB;
                    if (!mbar_wait(bar.at(kBarBFull + s), (bcount / kStagesB) & 1, abort_flag, sink)) {
                        ok = false;
                        break;
                    }
                    const uint32_t stage = sbase + kOffB + s * kTileBytes;
                    if (mine) {
                        const uint32_t a = cnt & 1;
                        if (!mbar_wait(bar.at(kBarAccEmpty + a * 2 + m), ((cnt >> 1) & 1) ^ 1, abort_flag, sink)) {
                            ok = false;
                            break;
                        }
                        tc_fence_after();
                        const uint32_t d_tmem = tmem_base + a * 256 + m * 128;
                        umma_tile_k128(d_tmem, resident, stage, idesc_k);
                        // ... - (T / r_i) (||k_j|| + eps): the accumulator's sign is the threshold test
                        umma_k16_sw32(d_tmem, res_slice, sbase + kOffAugB + s * kSliceBytes, idesc_k);
                        umma_commit(bar.at(kBarAccFull + a * 2 + m));
                        ++cnt;
                        ++tiles_done;
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
    } else if (warp >= kGatherWarp0) {
        // ------------------------------------------------------------------ gather warps
        // They run one item ahead of the scan: the listed tokens' key rows go into the resident tiles of the buffer
        // the scan is not using (same swizzled layout as a TMA load), each row's extra slice beside them, and what the
        // epilogue needs to know about the token into the stash.  Thread g serves rows g and g + 128 of the item.
        const int gt = (warp - kGatherWarp0) * 32 + lane;      // 0..127
        uint32_t k_item = 0;
        while (true) {
            const uint32_t qs = k_item % kItemSlots;
            if (!mbar_wait(bar.at(kBarQFull + qs), (k_item / kItemSlots) & 1, abort_flag, sink)) break;
            const int4 d = items[qs];
            __syncwarp();
            if (lane == 0) mbar_arrive(bar.at(kBarQEmpty + qs));
            if (d.x < 0) break;
            const int head = d.x, k0 = d.y, rows = d.z & 0xffff;
            const uint32_t ab = k_item & 1;
            if (!mbar_wait(bar.at(kBarAEmpty + ab), ((k_item >> 1) & 1) ^ 1, abort_flag, sink)) break;
            const int num_m = rows > kTile ? 2 : 1;
            const size_t hoff = (size_t)head * p.cap_pad;
            int pos[2];
            float rr[2];
            int lf[2];
#pragma unroll
            for (int m = 0; m < 2; ++m) pos[m] = (m * kTile + gt < rows) ? p.strag[hoff + k0 + m * kTile + gt] : -1;
#pragma unroll
            for (int m = 0; m < 2; ++m) {
                rr[m] = pos[m] >= 0 ? __ldg(p.inv_norm + hoff + pos[m]) : 0.f;
                lf[m] = pos[m] >= 0 ? p.left[hoff + pos[m]] : 0;
            }
            int32_t *stash_i = reinterpret_cast<int32_t *>(smem + kOffStash + ab * 3 * kRowsPerItem * 4);
            float *stash_r = reinterpret_cast<float *>(stash_i + kRowsPerItem);
            int32_t *stash_left = stash_i + 2 * kRowsPerItem;
#pragma unroll
            for (int m = 0; m < 2; ++m) {
                if (m >= num_m) break;
                const bool row_ok = pos[m] >= 0;
                uint8_t *tile = smem + kOffA + (ab * 2 + m) * kTileBytes;
                const uint4 *src = reinterpret_cast<const uint4 *>(
                    static_cast<const __nv_bfloat16 *>(p.k_cache) + (size_t)row_index(p, head, row_ok ? pos[m] : 0) * kHeadDim);
                uint4 v[16];
#pragma unroll
                for (int c = 0; c < 16; ++c) v[c] = row_ok ? __ldg(src + c) : make_uint4(0u, 0u, 0u, 0u);
#pragma unroll
                for (int hb = 0; hb < 2; ++hb) {
#pragma unroll
                    for (int c = 0; c < 8; ++c)
                        *reinterpret_cast<uint4 *>(tile + hb * kHalfBytes + gt * 128 + ((c ^ (gt & 7)) << 4)) = v[hb * 8 + c];
                }
                // the row's extra slice: -T / r_i in three bf16 parts as (-t1, -t1, -t1, -t2, -t2, -t3, 0 ...),
                // which meets (n1, n2, n3, n1, n2, n1, 0 ...) of a key; 32-byte rows, 32-byte swizzle
                float rest = (row_ok && rr[m] > 0.f) ? -__fdiv_rn(p.sim_threshold, rr[m]) : 0.f;
                uint32_t part[3];
#pragma unroll
                for (int c = 0; c < 3; ++c) {
                    const __nv_bfloat16 h16 = __float2bfloat16_rn(rest);
                    part[c] = (uint32_t)__bfloat16_as_ushort(h16);
                    rest -= __bfloat162float(h16);
                }
                uint8_t *slice = smem + kOffAugA + (ab * 2 + m) * kSliceBytes + gt * 32;
                const int sw = (gt >> 2) & 1;
                *reinterpret_cast<uint4 *>(slice + (sw << 4)) =
                    make_uint4(part[0] | (part[0] << 16), part[0] | (part[1] << 16), part[1] | (part[2] << 16), 0u);
                *reinterpret_cast<uint4 *>(slice + ((sw ^ 1) << 4)) = make_uint4(0u, 0u, 0u, 0u);
                stash_i[m * kTile + gt] = row_ok ? pos[m] : 0;
                stash_r[m * kTile + gt] = rr[m];
                stash_left[m * kTile + gt] = lf[m];
            }
            asm volatile("fence.proxy.async.shared::cta;" ::: "memory");   // generic writes -> tensor-core reads
            __syncwarp();
            if (lane == 0) mbar_arrive(bar.at(kBarAFull + ab));
            ++k_item;
        }
    } else {
        // ------------------------------------------------------------------ epilogue warps
        const int ew = warp - 2;                 // 0..7
        const int m = ew >> 2;                   // row tile of the item this warp serves
        const int quad = warp & 3;               // TMEM lane quadrant this warp may access
        const int lrow = quad * 32 + lane;       // row within the 128-row tile
        const uint32_t lane_base = tmem_base + ((uint32_t)(quad * 32) << 16);
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
            const uint32_t ab = k_item & 1;          // resident buffer (and stash) of this item

            // ---- per item: which token this thread owns (left in the stash by the gather warps), where the scan
            // starts and ends
            const int rows = d.z & 0xffff, first_tile = d.w, last_tile = d.w - (d.z >> 16) + 1;
            const bool active = (m == 0) || (rows > kTile);
            const bool row_ok = active && (m * kTile + lrow) < rows;
            bool item_ok = mbar_wait(bar.at(kBarAFull + ab), (k_item >> 1) & 1, abort_flag, sink);
            int i = 0, left = 0;
            float ri = 0.f;
            if (row_ok && item_ok) {
                const int32_t *stash_i = reinterpret_cast<const int32_t *>(smem + kOffStash + ab * 3 * kRowsPerItem * 4);
                i = stash_i[m * kTile + lrow];
                ri = reinterpret_cast<const float *>(stash_i + kRowsPerItem)[m * kTile + lrow];
                left = stash_i[2 * kRowsPerItem + m * kTile + lrow];
            }

            float removed = 0.f;
            // how many partners were found; with beta = 1 the one partner's position and accumulator value
            int nhit = 0, hit_j = -1;
            float hit_h = 0.f;
            if (active) {
                // ---- key tiles of the window, last to first
                bool ok = item_ok;
                for (int jt = first_tile; jt >= last_tile; --jt) {
                    const int jbase = jt * kTile;
                    // (with beta > 1 the partners' values need the r_j of whole chunks: read through the L1 cache, and only
                    // for the chunks that hold partners)
                    const float4 *rj4 = reinterpret_cast<const float4 *>(inv_norm + jbase);
                    const uint32_t a = cnt & 1;
                    if (ok) ok = mbar_wait(bar.at(kBarAccFull + a * 2 + m), (cnt >> 1) & 1, abort_flag, sink);
                    ++cnt;
                    if (!ok) continue;
                    tc_fence_after();
                    const uint32_t base = lane_base + a * 256 + m * 128;
                    // a token that has its beta partners screens nothing any more
                    bool want = left > 0;
                    // The accumulator holds h = k_i . k_j - (T / r_i) (||k_j|| + eps): S[j][i] > T exactly when h > 0, so
                    // the screening is a sign test, with nothing to load per column (loads of the r_j were what this
                    // epilogue's time went into: every byte a thread receives, from TMEM or as a shared-memory
                    // broadcast, passes through the same return path).  32-column chunks, last first; the TMEM load of
                    // the next chunk is issued before the current one is looked at (two register sets, used alternately).
                    // (beta = 1, the default: one partner per token)
                    auto chunk = [&](const uint32_t (&g)[32], int ch) {
                        uint32_t colmask = 0xffffffffu;
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
                        // entries with a clear sign bit (h > 0, but also +0: confirmed one by one below)
                        uint32_t pos = want ? (~neg & colmask) : 0u;
                        {
                            // one partner at most: the candidate at the highest set bit, its value picked by a select
                            // tree (nearly always a single turn); its r_j is fetched once, at the item's end
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
                                    hit_h = hv;
                                    hit_j = jbase + ch * 32 + top;
                                    left = 0;
                                    want = false;
                                    break;
                                }
                                pos &= ~(1u << top);
                            }
                        }
                    };
                    if (p.beta == 1) {
                        if (__any_sync(0xffffffffu, want)) {
                            uint32_t ga[32], gb[32];
                            tmem_ld32(base + 96, ga);
                            tmem_wait32(ga);
                            tmem_ld32(base + 64, gb);
                            chunk(ga, 3);
                            tmem_wait32(gb);
                            tmem_ld32(base + 32, ga);
                            chunk(gb, 2);
                            tmem_wait32(ga);
                            tmem_ld32(base, gb);
                            chunk(ga, 1);
                            tmem_wait32(gb);
                            chunk(gb, 0);
                        }
                    } else if (__any_sync(0xffffffffu, want)) {
                        // Several partners per token.  This loop is kept rolled on purpose: the warps of three roles
                        // share the instruction cache, and one copy of this body is what fits (unrolled like the
                        // path above it ran a third slower).
#pragma unroll 1
                        for (int ch = 3; ch >= 0; --ch) {
                            uint32_t g[32];
                            tmem_ld32(base + ch * 32, g);
                            float v[32];
                            uint32_t hits = 0u;
                            tmem_wait32(g);
#pragma unroll
                            for (int c = 0; c < 32; ++c) v[c] = __uint_as_float(g[c]);
                            float m0 = 0.f, m1 = 0.f;
#pragma unroll
                            for (int c = 0; c < 32; c += 4) {
                                m0 = max3(m0, v[c], v[c + 1]);
                                m1 = max3(m1, v[c + 2], v[c + 3]);
                            }
                            const float cut = want ? 0.f : __int_as_float(0x7f800000);
                            if (!__any_sync(0xffffffffu, fmaxf(m0, m1) > cut)) continue;
#pragma unroll
                            for (int c = 0; c < 32; ++c) hits |= (v[c] > cut) ? (1u << c) : 0u;
                            const unsigned own = (unsigned)(i - (jbase + ch * 32));           // zero diagonal (Eq. 5)
                            if (own < 32u) hits &= ~(1u << own);
                            // the exact mask, cut down to the highest positions if they are more than the token still
                            // lacks, then the sum of their h r_j (S = T + h r_i r_j per partner)
                            int taken = __popc(hits);
                            for (; taken > left; --taken) hits &= hits - 1u;                   // drop the lowest positions
                            nhit += taken;
#pragma unroll
                            for (int q = 0; q < 8; ++q) {
                                const float4 R = __ldg(rj4 + ch * 8 + q);
                                v[4 * q] *= R.x;
                                v[4 * q + 1] *= R.y;
                                v[4 * q + 2] *= R.z;
                                v[4 * q + 3] *= R.w;
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
                            if (left == 0) want = false;
                        }
                    }
                    tc_fence_before();
                    __syncwarp();
                    if (lane == 0) mbar_arrive(bar.at(kBarAccEmpty + a * 2 + m));
                }
                item_ok = ok;
            }
            // the item's resident buffer and stash are no longer read by this warp
            __syncwarp();
            if (lane == 0 && item_ok) mbar_arrive(bar.at(kBarAEmpty + ab));
            if (!item_ok) break;              // (the epilogue warps meet at no barrier of their own: each may leave alone)
            if (row_ok) {
                // S = T + h r_i r_j for every partner found here
                if (p.beta == 1 && hit_j >= 0) {
                    removed = hit_h * __ldg(inv_norm + hit_j);
                    nhit = 1;
                }
                if (nhit > 0) {
                    p.sbar[(size_t)head * p.cap_pad + i] -= (float)nhit * p.sim_threshold + removed * ri;
                    p.left[(size_t)head * p.cap_pad + i] = left;       // the next round lists the tokens still short
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

// ---- before every round: list, per head, the tokens still short of partners, and cut the list into work items ----
constexpr int kCompactThreads = 256;
constexpr int kDenseMinTiles = 12;       // caches of fewer key tiles never take the symmetric route (two more launches)

// `below`: key tiles under the first pass's part that earlier rounds have covered; `width`: tiles of this round's
// window (the last round passes a width that reaches tile 0 whatever the cache size).
__global__ void __launch_bounds__(kCompactThreads) strag_compact_kernel(Params p, int round, int below, int width)
{
    __shared__ int warp_tot[kCompactThreads / 32];
    __shared__ int running;
    const int head = blockIdx.x;
    const int n = seq_candidates(p, head / p.hkv);
    const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
    const int32_t *left = p.left + (size_t)head * p.cap_pad;
    int32_t *list = p.strag + (size_t)head * p.cap_pad;
    // the first pass scanned every token against the last kPass1Depth key tiles; this round starts `below` tiles
    // under that
    const int n_tiles = (n + kTile - 1) / kTile;
    const int first_tile = n_tiles - kPass1Depth - 1 - below;
    if (first_tile < 0 || call_aborted(p) || (round > 0 && p.dense[head])) {
        // nothing left to scan for this head, the call has given up, or the head went to the symmetric route
        if (threadIdx.x == 0) {
            p.strag_count[head] = 0;
            if (round == 0) p.dense[head] = 0;
        }
        return;
    }
    if (threadIdx.x == 0) running = 0;
    __syncthreads();
    for (int i0 = 0; i0 < n; i0 += kCompactThreads) {
        const int i = i0 + threadIdx.x;
        const bool want = i < n && left[i] > 0;
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
    if (round == 0) {
        // Most tokens still lack a partner (few pairs exceed T): the rounds would form nearly the whole matrix for this
        // head.  It goes to the symmetric route instead, which forms each tile pair once.
        const bool dense = p.dense_ok && n_tiles >= kDenseMinTiles && 5 * running > 4 * n;
        if (dense) {
            uint32_t *best = p.best + (size_t)head * p.cap_pad;
            for (int i = threadIdx.x; i < p.cap_pad; i += kCompactThreads) best[i] = 0u;
            if (threadIdx.x == 0) {
                p.dense[head] = 1;
                p.strag_count[head] = 0;
                const int pairs_of_tiles = (n_tiles + 1) / 2;
                const unsigned long long at = atomicAdd(&p.counters[kDenseWords], (unsigned long long)pairs_of_tiles);
                for (int q = 0; q < pairs_of_tiles; ++q) p.dense_items[at + q] = make_int4(head, q, n, 0);   // longest first
                // useful work: every unordered pair of the listed tokens' tiles once
                atomicAdd(&p.counters[kPairsWord], (unsigned long long)running * (unsigned long long)(n_tiles + 1) / 2ull);
            }
            return;
        }
        if (threadIdx.x == 0) p.dense[head] = 0;
    }
    if (threadIdx.x == 0) {
        const int count = running;
        p.strag_count[head] = count;
        const int chunks = (count + kRowsPerItem - 1) / kRowsPerItem;
        if (chunks > 0) {
            const int n_iter = min(width, first_tile + 1);
            const unsigned long long at = atomicAdd(&p.counters[kRoundWords + 2 * round], (unsigned long long)chunks);
            for (int q = 0; q < chunks; ++q) {
                const int k0 = q * kRowsPerItem, rows = min(count - k0, kRowsPerItem);
                p.strag_items[at + q] = make_int4(head, k0, rows | (n_iter << 16), first_tile);
            }
            atomicAdd(&p.counters[2], (unsigned long long)chunks);
            // listed tokens x key tiles: the work the round cannot avoid
            atomicAdd(&p.counters[kPairsWord], (unsigned long long)count * (unsigned long long)n_iter);
        }
    }
}

}  // namespace

bool scores_dense_possible(int tiles, int beta) { return beta == 1 && tiles >= kDenseMinTiles; }

int scores_pass2_rounds(int tiles)
{
    const int below = tiles - kPass1Depth;      // key tiles under the first pass's part, at most
    return below <= 8 ? 1 : 2;
}

cudaError_t launch_scores_tri_sm100(const Params &p, cudaStream_t s)
{
    const int q_rows = p.group * p.alpha;
    const int q_rows_pad = (q_rows + 15) / 16 * 16;
    CUtensorMap map_k, map_q, map_hs, map_ns, map_ts;
    if (!make_map(&map_k, p.k_cache, key_rows_total(p), kTile) ||
        !make_map(&map_q, p.q_window, (uint64_t)p.batch * p.hq * p.alpha, (uint32_t)q_rows_pad) ||
        !make_map(&map_hs, p.head_sum_bf16, (uint64_t)p.batch * p.hkv * 16, 16u) ||
        !make_map_k16(&map_ns, p.norm_split, (uint64_t)p.batch * p.hkv * p.cap_pad) ||
        !make_map_k16(&map_ts, p.thr_split, (uint64_t)p.batch * p.hkv * kTile))
        return cudaErrorInvalidValue;
    cudaError_t e;
    if ((e = cudaFuncSetAttribute(scores_pass2_sm100_kernel, cudaFuncAttributeMaxDynamicSharedMemorySize, kSmemBytes)) !=
        cudaSuccess)
        return e;
    int dev = 0, sms = 0;
    if ((e = cudaGetDevice(&dev)) != cudaSuccess) return e;
    if ((e = cudaDeviceGetAttribute(&sms, cudaDevAttrMultiProcessorCount, dev)) != cudaSuccess) return e;
    const int heads = p.batch * p.hkv;
    if ((e = launch_scores_pass1_sm100(p, s, map_k, map_q, map_hs, map_ns, map_ts, q_rows_pad, sms)) != cudaSuccess) return e;
    if ((e = mark_kernel(p, 0, s)) != cudaSuccess) return e;
    const bool rule_on = p.beta > 0 && p.sim_threshold < 1.0f;
    if (!rule_on || p.tiles < 2) return mark_kernel(p, 1, s);       // nobody can lack partners / the first pass has seen everything
    const unsigned long long max_items2 = (unsigned long long)heads * (unsigned long long)(p.cap_pad / kRowsPerItem + 1);
    const unsigned grid2 = (unsigned)(max_items2 < (unsigned long long)sms ? max_items2 : (unsigned long long)sms);
    // rounds of the second pass: short windows first, so that the tokens that find their partners soon drop out
    // before the long scan down to tile 0
    const int rounds = scores_pass2_rounds(p.tiles);
    static const int kRoundTiles[2] = {6, 1 << 20};      // (measured: 6 + rest beats 4 + 8 + rest and 8 + rest by a little)
    const bool dense_possible = p.dense_ok && p.tiles >= kDenseMinTiles;
    int below = 0;
    for (int r = 0; r < rounds; ++r) {
        const int width = r == rounds - 1 ? (1 << 20) : kRoundTiles[r];
        strag_compact_kernel<<<(unsigned)heads, kCompactThreads, 0, s>>>(p, r, below, width);
        if ((e = cudaGetLastError()) != cudaSuccess) return e;
        if (r == 0 && (e = mark_kernel(p, 1, s)) != cudaSuccess) return e;
        scores_pass2_sm100_kernel<<<grid2, kThreads, kSmemBytes, s>>>(p, map_k, map_ns, r);
        if ((e = cudaGetLastError()) != cudaSuccess) return e;
        // the heads the first listing sent to the symmetric route (none on inputs where similar keys are common:
        // the kernel then returns at once)
        if (r == 0 && dense_possible && (e = launch_scores_dense_sm100(p, s, map_k, map_ns, sms)) != cudaSuccess) return e;
        below += width;
    }
    return dense_possible ? launch_dense_finish(p, s, sms) : cudaSuccess;
}

}  // namespace rkv

// Stage "scores", symmetric route of the second pass, for heads in which most tokens are still short of a partner
// after the first pass (few pairs above the threshold T: the two-pass shortcut does not pay there and the rounds of
// rkv_scores_p2_sm100.cu would form nearly the whole similarity matrix).  Only with beta = 1.
//
// Eq. 5's matrix is symmetric before the retention rule, so one tile product serves both of its index sets.  Per head
// the tile pairs (I, J) with J >= I are formed once (the upper triangle: T (T + 1) / 2 products instead of T^2):
//
//   row direction     thread = token i of row tile I scans the tile's 128 columns j: a partner LATER than i (or in i's
//                     own tile).  Key tiles stream from the last one downwards, so the first hit is the largest j.
//   column direction  (J > I only) every entry above the threshold also makes token i a candidate EARLIER partner of
//                     token j of key tile J.
//
// Section 3.3's rule with beta = 1 keeps, per token, the LARGEST position j with S[j][i] > T: a maximum, which does not
// depend on the order in which candidates turn up.  Both directions therefore just raise best[token] = position + 1
// with atomicMax (row direction once per item, column direction per entry above the threshold: rare on the inputs
// this route is chosen for).  The partner's similarity is recomputed afterwards, once per token, from the two key
// rows (dense_finish_kernel).  The threshold test is the sign of the accumulator, as in the other two scoring kernels
// (one extra K = 16 step per tile product).
//
// Work item = (head, pair of row tiles p): rows [256 p, 256 p + 256) resident (TMA), key tiles T - 1 .. 2 p streamed;
// row tile 2 p + 1 skips key tile 2 p (the lower triangle).  Items are drawn longest first.  Warp roles and barriers
// as in rkv_scores_p2_sm100.cu (512 threads: ticket warp, TMA producer, two MMA issuers, eight epilogue warps, four
// warps that prepare the next item's threshold slices and per-token data while the current one is scanned).  Every
// wait is bounded; no TMA multicast, no clusters.
#include "rkv_sm100.cuh"

namespace rkv {

namespace {

using namespace sm100;

constexpr int kThreadsD = 512;
constexpr int kPrepWarp0 = 11;                   // first of the 4 warps that prepare slices and stash
constexpr int kTicketWarpD = 15;
constexpr int kStagesD = 2;                      // ring depth of streamed tiles
constexpr int kItemSlotsD = 4;
constexpr int kHalfBytes = kTile * 64 * 2;
constexpr int kTileBytes = 2 * kHalfBytes;
constexpr int kRowsPerItem = 2 * kTile;
constexpr uint32_t kTmemColsD = 512;
constexpr int kSliceBytes = kTile * 32;

constexpr int kOffA = 0;                                   // 2 buffers x 2 resident tiles
constexpr int kOffB = kOffA + 2 * 2 * kTileBytes;          // kStagesD streamed tiles
constexpr int kOffAugA = kOffB + kStagesD * kTileBytes;    // 2 buffers x 2 slices (rows: -T / r_i)
constexpr int kOffAugB = kOffAugA + 2 * 2 * kSliceBytes;   // kStagesD slices (keys: 1 / r_j)
constexpr int kOffStash = kOffAugB + kStagesD * kSliceBytes;            // 2 buffers x kRowsPerItem x left
constexpr int kOffBar = kOffStash + 2 * kRowsPerItem * 4;
enum {
    kBarQFull = 0,
    kBarQEmpty = kBarQFull + kItemSlotsD,   // producer, 2 MMA threads, 8 epilogue warps, 4 preparing warps
    kBarAFull = kBarQEmpty + kItemSlotsD,   // [2] resident tiles landed (producer + bytes) and slices / stash written (4 warps)
    kBarAEmpty = kBarAFull + 2,             // [2] ... no longer read (2 MMA threads, 8 epilogue warps)
    kBarBFull = kBarAEmpty + 2,
    kBarBEmpty = kBarBFull + kStagesD,
    kBarAccFull = kBarBEmpty + kStagesD,    // [2 buffers][2 row tiles]
    kBarAccEmpty = kBarAccFull + 4,
    kNumBarsD = kBarAccEmpty + 4
};
constexpr int kOffItems = kOffBar + kNumBarsD * 8;
constexpr int kOffMisc = kOffItems + kItemSlotsD * 16;
constexpr int kSmemBytesD = kOffMisc + 16 + 1024;
static_assert(kOffItems % 16 == 0, "item descriptors are read as int4");
static_assert(kSmemBytesD <= 227 * 1024, "shared memory budget");

// Item descriptor (int4): {head, pair of row tiles p, n, -}.  x < 0: no more items.
__global__ void __launch_bounds__(kThreadsD, 1)
scores_dense_sm100_kernel(Params p, const __grid_constant__ CUtensorMap map_k, const __grid_constant__ CUtensorMap map_ns)
{
    unsigned long long *const item_count = p.counters + kDenseWords, *const ticket = item_count + 1;
    extern __shared__ uint8_t smem_raw[];
    uint8_t *smem = reinterpret_cast<uint8_t *>((reinterpret_cast<uintptr_t>(smem_raw) + 1023) & ~(uintptr_t)1023);
    const uint32_t sbase = smem_u32(smem);
    int4 *items = reinterpret_cast<int4 *>(smem + kOffItems);
    uint32_t *tmem_holder = reinterpret_cast<uint32_t *>(smem + kOffMisc);
    volatile int *abort_flag = reinterpret_cast<volatile int *>(smem + kOffMisc + 4);
    volatile int *bail = reinterpret_cast<volatile int *>(smem + kOffMisc + 8);
    const uint32_t bar0 = sbase + kOffBar;
    auto bar = [bar0](int idx) -> uint32_t { return bar0 + 8u * (uint32_t)idx; };

    const ErrSink sink = make_sink(p);
    if (threadIdx.x == 0) *bail = (call_aborted(p) || *item_count == 0ull) ? 1 : 0;     // nothing listed for this route
    __syncthreads();
    if (*bail) return;

    const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
    const unsigned long long total_items = *item_count;

    if (threadIdx.x == 0) {
        for (int s = 0; s < kItemSlotsD; ++s) {
            mbar_init(bar(kBarQFull + s), 1);
            mbar_init(bar(kBarQEmpty + s), 15);
        }
        for (int s = 0; s < 2; ++s) {
            mbar_init(bar(kBarAFull + s), 5);
            mbar_init(bar(kBarAEmpty + s), 10);
        }
        for (int s = 0; s < kStagesD; ++s) {
            mbar_init(bar(kBarBFull + s), 1);
            mbar_init(bar(kBarBEmpty + s), 2);
        }
        for (int s = 0; s < 4; ++s) {
            mbar_init(bar(kBarAccFull + s), 1);
            mbar_init(bar(kBarAccEmpty + s), 4);
        }
        *abort_flag = 0;
        asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory");
    }
    if (warp == 1) {
        asm volatile("tcgen05.alloc.cta_group::1.sync.aligned.shared::cta.b32 [%0], %1;"
                     ::"r"(smem_u32(tmem_holder)), "r"(kTmemColsD) : "memory");
        asm volatile("tcgen05.relinquish_alloc_permit.cta_group::1.sync.aligned;" ::: "memory");
    }
    tc_fence_before();
    __syncthreads();
    tc_fence_after();
    const uint32_t tmem_base = *tmem_holder;
    unsigned long long tiles_done = 0ull;

    if (warp == kTicketWarpD) {
        // ------------------------------------------------------------------ tickets: descriptors up to three items ahead
        if (lane == 0) {
            uint32_t k_item = 0;
            while (true) {
                const unsigned long long cur = atomicAdd(ticket, 1ull);
                if (cur >= total_items) break;
                const int4 desc = p.dense_items[cur];
                const uint32_t qs = k_item % kItemSlotsD;
                if (!mbar_wait(bar(kBarQEmpty + qs), ((k_item / kItemSlotsD) & 1) ^ 1, abort_flag, sink)) break;
                items[qs] = desc;
                mbar_arrive(bar(kBarQFull + qs));
                ++k_item;
            }
            if (!*abort_flag) {             // terminator (skipped when the block is aborting)
                const uint32_t qs = k_item % kItemSlotsD;
                if (mbar_wait(bar(kBarQEmpty + qs), ((k_item / kItemSlotsD) & 1) ^ 1, abort_flag, sink)) {
                    items[qs] = make_int4(-1, 0, 0, 0);
                    mbar_arrive(bar(kBarQFull + qs));
                }
            }
        }
        __syncwarp();
    } else if (warp == 0) {
        // ------------------------------------------------------------------ TMA producer: resident row tiles, then key tiles
        if (lane == 0) {
            uint32_t k_item = 0, bcount = 0;
            bool ok = true;
            while (ok) {
                const uint32_t qs = k_item % kItemSlotsD;
                if (!mbar_wait(bar(kBarQFull + qs), (k_item / kItemSlotsD) & 1, abort_flag, sink)) break;
                const int4 d = items[qs];
                mbar_arrive(bar(kBarQEmpty + qs));
                if (d.x < 0) break;
                const int head = d.x, pi = d.y, n = d.z;
                const int n_tiles = (n + kTile - 1) / kTile;
                const int num_m = (n - pi * kRowsPerItem > kTile) ? 2 : 1;
                const uint32_t ab = k_item & 1;
                if (!mbar_wait(bar(kBarAEmpty + ab), ((k_item >> 1) & 1) ^ 1, abort_flag, sink)) break;
                mbar_expect_tx(bar(kBarAFull + ab), (uint32_t)(num_m * kTileBytes));
                for (int m = 0; m < num_m; ++m) {
                    const uint32_t dst = sbase + kOffA + (ab * 2 + m) * kTileBytes;
                    const int y = (int)tile_row0(p, head, 2 * pi + m);
                    tma_load_2d(dst, &map_k, 0, y, bar(kBarAFull + ab));
                    tma_load_2d(dst + kHalfBytes, &map_k, 64, y, bar(kBarAFull + ab));
                }
                for (int jt = n_tiles - 1; jt >= 2 * pi; --jt) {
                    const uint32_t s = bcount % kStagesD;
                    if (!mbar_wait(bar(kBarBEmpty + s), ((bcount / kStagesD) & 1) ^ 1, abort_flag, sink)) {
                        ok = false;
                        break;
                    }
                    const uint32_t dst = sbase + kOffB + s * kTileBytes;
                    const int y = (int)tile_row0(p, head, jt);
                    mbar_expect_tx(bar(kBarBFull + s), kTileBytes + kSliceBytes);
                    tma_load_2d(dst, &map_k, 0, y, bar(kBarBFull + s));
                    tma_load_2d(dst + kHalfBytes, &map_k, 64, y, bar(kBarBFull + s));
                    tma_load_2d(sbase + kOffAugB + s * kSliceBytes, &map_ns, 0, head * p.cap_pad + jt * kTile, bar(kBarBFull + s));
                    ++bcount;
                }
                ++k_item;
            }
        }
        __syncwarp();
    } else if (warp == 1 || warp == 10) {
        // ------------------------------------------------------------------ MMA issuers (one per row tile of the item)
        if (lane == 0) {
            const int m = warp == 1 ? 0 : 1;
            const uint32_t idesc_k = instr_desc(kTile, kTile);
            uint32_t k_item = 0, bcount = 0, cnt = 0;
            bool ok = true;
            while (ok) {
                const uint32_t qs = k_item % kItemSlotsD;
                if (!mbar_wait(bar(kBarQFull + qs), (k_item / kItemSlotsD) & 1, abort_flag, sink)) break;
                const int4 d = items[qs];
                mbar_arrive(bar(kBarQEmpty + qs));
                if (d.x < 0) break;
                const int pi = d.y, n = d.z;
                const int n_tiles = (n + kTile - 1) / kTile;
                const bool mine = m == 0 || (n - pi * kRowsPerItem > kTile);
                const uint32_t ab = k_item & 1;
                if (!mbar_wait(bar(kBarAFull + ab), (k_item >> 1) & 1, abort_flag, sink)) break;
                asm volatile("tcgen05.fence::after_thread_sync;" ::: "memory");
                const uint32_t resident = sbase + kOffA + (ab * 2 + m) * kTileBytes;
                const uint32_t res_slice = sbase + kOffAugA + (ab * 2 + m) * kSliceBytes;
                for (int jt = n_tiles - 1; jt >= 2 * pi; --jt) {
                    const uint32_t s = bcount % kStagesD;
                    if (!mbar_wait(bar(kBarBFull + s), (bcount / kStagesD) & 1, abort_flag, sink)) {
                        ok = false;
                        break;
                    }
                    const uint32_t stage = sbase + kOffB + s * kTileBytes;
                    if (mine && jt >= 2 * pi + m) {           // row tile 2 p + 1 leaves key tile 2 p to the column direction
                        const uint32_t a = cnt & 1;
                        if (!mbar_wait(bar(kBarAccEmpty + a * 2 + m), ((cnt >> 1) & 1) ^ 1, abort_flag, sink)) {
                            ok = false;
                            break;
                        }
                        tc_fence_after();
                        const uint32_t d_tmem = tmem_base + a * 256 + m * 128;
                        umma_tile_k128(d_tmem, resident, stage, idesc_k);
                        umma_k16_sw32(d_tmem, res_slice, sbase + kOffAugB + s * kSliceBytes, idesc_k);
                        umma_commit(bar(kBarAccFull + a * 2 + m));
                        ++cnt;
                        ++tiles_done;
                        umma_commit(bar(kBarBEmpty + s));
                    } else {
                        mbar_arrive(bar(kBarBEmpty + s));
                    }
                    ++bcount;
                }
                if (!ok) break;
                if (mine) umma_commit(bar(kBarAEmpty + ab));
                else mbar_arrive(bar(kBarAEmpty + ab));
                ++k_item;
            }
        }
        __syncwarp();
    } else if (warp >= kPrepWarp0) {
        // ------------------------------------------------------------------ preparing warps, one item ahead of the scan
        // Thread g serves rows g and g + 128 of the item: the row's extra slice, -T / r_i in three bf16 parts as
        // (-t1, -t1, -t1, -t2, -t2, -t3, 0 ...) (32-byte rows, 32-byte swizzle), and whether the token still lacks
        // its partner.
        const int gt = (warp - kPrepWarp0) * 32 + lane;
        uint32_t k_item = 0;
        while (true) {
            const uint32_t qs = k_item % kItemSlotsD;
            if (!mbar_wait(bar(kBarQFull + qs), (k_item / kItemSlotsD) & 1, abort_flag, sink)) break;
            const int4 d = items[qs];
            __syncwarp();
            if (lane == 0) mbar_arrive(bar(kBarQEmpty + qs));
            if (d.x < 0) break;
            const int head = d.x, pi = d.y, n = d.z;
            const uint32_t ab = k_item & 1;
            if (!mbar_wait(bar(kBarAEmpty + ab), ((k_item >> 1) & 1) ^ 1, abort_flag, sink)) break;
            const size_t hoff = (size_t)head * p.cap_pad;
            int32_t *stash_left = reinterpret_cast<int32_t *>(smem + kOffStash + ab * kRowsPerItem * 4);
#pragma unroll
            for (int m = 0; m < 2; ++m) {
                const int i = pi * kRowsPerItem + m * kTile + gt;
                const bool row_ok = i < n;
                const float ri = row_ok ? __ldg(p.inv_norm + hoff + i) : 0.f;
                const int lf = row_ok ? p.left[hoff + i] : 0;
                float rest = (row_ok && ri > 0.f) ? -__fdiv_rn(p.sim_threshold, ri) : 0.f;
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
                stash_left[m * kTile + gt] = lf;
            }
            asm volatile("fence.proxy.async.shared::cta;" ::: "memory");   // generic writes -> tensor-core reads
            __syncwarp();
            if (lane == 0) mbar_arrive(bar(kBarAFull + ab));
            ++k_item;
        }
    } else {
        // ------------------------------------------------------------------ epilogue warps
        const int ew = warp - 2;                 // 0..7
        const int m = ew >> 2;                   // row tile of the item this warp serves
        const int quad = warp & 3;               // TMEM lane quadrant this warp may access
        const int lrow = quad * 32 + lane;
        const uint32_t lane_base = tmem_base + ((uint32_t)(quad * 32) << 16);
        const float kInf = __int_as_float(0x7f800000);
        uint32_t k_item = 0, cnt = 0;

        while (true) {
            const uint32_t qs = k_item % kItemSlotsD;
            if (!mbar_wait(bar(kBarQFull + qs), (k_item / kItemSlotsD) & 1, abort_flag, sink)) break;
            const int4 d = items[qs];
            __syncwarp();
            if (lane == 0) mbar_arrive(bar(kBarQEmpty + qs));
            if (d.x < 0) break;
            const int head = d.x, pi = d.y, n = d.z;
            const int n_tiles = (n + kTile - 1) / kTile;
            const uint32_t ab = k_item & 1;
            const bool active = (m == 0) || (n - pi * kRowsPerItem > kTile);
            const int own_tile = 2 * pi + m;
            const int i = own_tile * kTile + lrow;
            const bool row_ok = active && i < n;
            bool ok = mbar_wait(bar(kBarAFull + ab), (k_item >> 1) & 1, abort_flag, sink);
            bool want = false;                   // the token still lacks its partner
            if (row_ok && ok) want = reinterpret_cast<const int32_t *>(smem + kOffStash + ab * kRowsPerItem * 4)[m * kTile + lrow] > 0;
            uint32_t *best = p.best + (size_t)head * p.cap_pad;
            int hit_j = -1;                      // row direction: the largest position above the threshold found by this scan

            if (active) {
                for (int jt = n_tiles - 1; jt >= own_tile; --jt) {     // (row tile 2 p + 1 has no product with key tile 2 p)
                    const int jbase = jt * kTile;
                    const uint32_t a = cnt & 1;
                    if (ok) ok = mbar_wait(bar(kBarAccFull + a * 2 + m), (cnt >> 1) & 1, abort_flag, sink);
                    ++cnt;
                    if (!ok) continue;
                    tc_fence_after();
                    const uint32_t base = lane_base + a * 256 + m * 128;
                    const bool col_dir = jt > own_tile;           // entries also make token i a candidate for token j
                    const int valid = n - jbase;                  // columns [0, valid) of the tile are candidates
                    const float cut = row_ok ? 0.f : kInf;
#pragma unroll 1
                    for (int ch = 3; ch >= 0; --ch) {
                        uint32_t g[32];
                        tmem_ld32(base + ch * 32, g);
                        float v[32];
                        tmem_wait32(g);
#pragma unroll
                        for (int c = 0; c < 32; ++c) v[c] = __uint_as_float(g[c]);
                        float m0 = 0.f, m1 = 0.f;
#pragma unroll
                        for (int c = 0; c < 32; c += 4) {
                            m0 = max3(m0, v[c], v[c + 1]);
                            m1 = max3(m1, v[c + 2], v[c + 3]);
                        }
                        if (!__any_sync(0xffffffffu, fmaxf(m0, m1) > cut)) continue;       // nothing above the threshold here
                        uint32_t hits = 0u;
#pragma unroll
                        for (int c = 0; c < 32; ++c) hits |= (v[c] > cut) ? (1u << c) : 0u;
                        const int nv = valid - ch * 32;
                        hits &= nv >= 32 ? 0xffffffffu : (nv <= 0 ? 0u : ((1u << nv) - 1u));
                        const unsigned own = (unsigned)(i - (jbase + ch * 32));           // zero diagonal (Eq. 5)
                        if (own < 32u) hits &= ~(1u << own);
                        if (want && hits != 0u) {                 // the scan runs from the last position downwards
                            hit_j = jbase + ch * 32 + (31 - __clz(hits));
                            want = false;
                        }
                        if (col_dir) {
                            while (hits != 0u) {
                                const int c = __ffs(hits) - 1;
                                atomicMax(best + jbase + ch * 32 + c, (uint32_t)(i + 1));
                                hits &= hits - 1u;
                            }
                        }
                    }
                    tc_fence_before();
                    __syncwarp();
                    if (lane == 0) mbar_arrive(bar(kBarAccEmpty + a * 2 + m));
                }
            }
            if (ok && row_ok && hit_j >= 0) atomicMax(best + i, (uint32_t)(hit_j + 1));
            __syncwarp();
            if (lane == 0 && ok) mbar_arrive(bar(kBarAEmpty + ab));
            if (!ok) break;
            ++k_item;
        }
    }

    // ---------------------------------------------------------------------- common exit
    tc_fence_before();
    __syncthreads();
    if (warp == 1) {
        if (*abort_flag) __nanosleep(200000);      // error path only: let copies and MMAs in flight land
        tc_fence_after();
        asm volatile("tcgen05.dealloc.cta_group::1.sync.aligned.b32 %0, %1;" ::"r"(tmem_base), "r"(kTmemColsD) : "memory");
    }
    if ((warp == 1 || warp == 10) && lane == 0 && !*abort_flag && tiles_done) atomicAdd(p.counters, tiles_done);
}

// After the symmetric scan: every token of a head on this route that still lacks its partner and was given one takes
// the partner's similarity off its column sum, S = Kbar_i . Kbar_j, recomputed from the two key rows in fp32.
constexpr int kFinishThreads = 256;

__global__ void __launch_bounds__(kFinishThreads) dense_finish_kernel(Params p)
{
    // work unit = (head, chunk of 256 tokens), handed out with the grid as stride.  When no head took the route (the
    // common case: no work item of the symmetric scan was ever listed) the blocks return at once.
    const int chunks = (p.cap + kFinishThreads - 1) / kFinishThreads;
    const long long units = (long long)p.batch * p.hkv * chunks;
    if (call_aborted(p) || p.counters[kDenseWords] == 0ull) return;
    for (long long u = blockIdx.x; u < units; u += gridDim.x) {
    const int head = (int)(u / chunks);
    if (!p.dense[head]) continue;
    const int i = (int)(u % chunks) * kFinishThreads + threadIdx.x;
    const int n = seq_candidates(p, head / p.hkv);
    if (i >= n) continue;
    const size_t hoff = (size_t)head * p.cap_pad;
    if (p.left[hoff + i] <= 0) continue;
    const uint32_t b = p.best[hoff + i];
    if (b == 0u) continue;
    const int j = (int)b - 1;
    const uint4 *ki = reinterpret_cast<const uint4 *>(static_cast<const __nv_bfloat16 *>(p.k_cache) + (size_t)row_index(p, head, i) * kHeadDim);
    const uint4 *kj = reinterpret_cast<const uint4 *>(static_cast<const __nv_bfloat16 *>(p.k_cache) + (size_t)row_index(p, head, j) * kHeadDim);
    float dot = 0.f;
#pragma unroll 4
    for (int c = 0; c < kHeadDim / 8; ++c) {
        float a[8], bb[8];
        Elem<__nv_bfloat16>::unpack(__ldg(ki + c), a);
        Elem<__nv_bfloat16>::unpack(__ldg(kj + c), bb);
#pragma unroll
        for (int e = 0; e < 8; ++e) dot = fmaf(a[e], bb[e], dot);
    }
    p.sbar[hoff + i] -= dot * p.inv_norm[hoff + i] * p.inv_norm[hoff + j];
    p.left[hoff + i] = 0;
    }
}

}  // namespace

cudaError_t launch_scores_dense_sm100(const Params &p, cudaStream_t s, const CUtensorMap &map_k, const CUtensorMap &map_ns, int sms)
{
    cudaError_t e = cudaFuncSetAttribute(scores_dense_sm100_kernel, cudaFuncAttributeMaxDynamicSharedMemorySize, kSmemBytesD);
    if (e != cudaSuccess) return e;
    const unsigned long long max_items = (unsigned long long)(p.batch * p.hkv) * (unsigned long long)((p.tiles + 1) / 2);
    const unsigned grid = (unsigned)(max_items < (unsigned long long)sms ? max_items : (unsigned long long)sms);
    scores_dense_sm100_kernel<<<grid, kThreadsD, kSmemBytesD, s>>>(p, map_k, map_ns);
    return cudaGetLastError();
}

cudaError_t launch_dense_finish(const Params &p, cudaStream_t s, int sms)
{
    const unsigned long long units = (unsigned long long)(p.batch * p.hkv) * (unsigned long long)((p.cap + kFinishThreads - 1) / kFinishThreads);
    const unsigned long long wave = 8ull * (unsigned long long)sms;             // resident blocks of this size
    dense_finish_kernel<<<(unsigned)(units < wave ? units : wave), kFinishThreads, 0, s>>>(p);
    return cudaGetLastError();
}

}  // namespace rkv

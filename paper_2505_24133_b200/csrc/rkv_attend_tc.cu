// Decode-step attention over the compressed cache (Section 3.1, Eq. 1 with one query row per head), tensor-core form
// for bf16 and 8-bit caches with d = 128:
//
//   out[b][q] = sum_j softmax_j( q_new[b][q] . K[b][q / G][j] / sqrt(d) ) V[b][q / G][j],   j < seq_lens[b]
//
// The work is HBM-bound (every cached K and V row is read once), but with G query heads per KV head a CUDA-core
// kernel spends 4 G d fp32 operations per 512 bytes and runs out of issue slots from G = 5 on.  Here the two
// contractions go to the tensor cores, with the keys -- not the G <= 8 queries -- as the 128-row M dimension:
//
//   scores   S^T [128 keys x 16] = K_tile [128 x d] . Q^T [d x 16]     (K-major operands; the group's queries, padded to
//            N = 16, are the B operand; one accumulator of 16 TMEM columns PER key tile of the block)
//   values   O^T [d x 16] += V_tile^T [d x 128 keys] . P [128 keys x 16]   (the V tile as TMA leaves it, used transposed:
//            MN-major A operand; P = the softmax weights in bf16, written to shared memory by the softmax threads)
//
// A block owns one (KV head, split of the key tiles) with at most 15 tiles.  First all its K tiles stream through the
// ring and leave their scores in TMEM (16 columns each, 240 at most, beside the 16 output columns); then the exact
// maximum per query over the whole split is taken, so the weights need no running rescale; then the V tiles stream
// through the same ring while the softmax threads turn score columns into P tiles (double-buffered).  Every weight
// is split into two bf16 parts (rows g and 8 + g of P: N = 16 has the room), so the products carry fp32-accurate
// weights; the sum of the weights is taken from the same parts.  Splits are merged by attend_merge_kernel.
//
// Warps 0..3: softmax (thread = TMEM lane = key row of a tile, later = output dimension), warp 4: TMA producer,
// warp 5: MMA issuer and TMEM owner.
//
// 8-bit caches (E4M3 codes, kFp8): the tiles arrive as 128 rows of 128 bytes (a ring of two 16 KB stages) and are
// widened into one of two bf16 operand tiles by the softmax threads, one row each, on their way to the tensor cores
// (four raw stages and a single operand tile were measured slower: the chain widen -> product must not serialise); everything else is the same, at half the bytes per cached
// row.  Rows beyond the length are written as zeros there.
//
// Every mbarrier wait is bounded; on expiry the block records RKV_ERR_TIMEOUT,
// writes zeros and leaves through the common exit that frees TMEM.  No TMA multicast, no cluster launch.
#include "rkv_sm100.cuh"

namespace rkv {

namespace {

using namespace sm100;

constexpr int kTcThreads = 192;
constexpr int kTcStages = 3;                         // ring of key / value tiles
constexpr int kTcMaxTiles = 15;                      // key tiles per block
constexpr int kTcHalf = kTile * 64 * 2;              // one TMA box: 128 rows x 64 bf16
constexpr int kTcTileBytes = 2 * kTcHalf;            // 32 KB
constexpr int kTcSmall = 16 * kHeadDim * 2;          // a [16 x 128] bf16 operand (Q^T or P): two [16 x 64] halves of 2 KB
constexpr uint32_t kTcTmemCols = 256;                // 16 (output) + 16 per key tile

constexpr int kOffRing = 0;                          // bf16 caches: kTcStages tiles.  8-bit caches: kConvBufs widened tiles,
constexpr int kConvBufs = 2;
constexpr int kRawStages = 2;
constexpr int kOffRaw = kConvBufs * kTcTileBytes;    // then kRawStages raw stages of 16 KB
constexpr int kRawBytes = kTile * kHeadDim;          // a tile of E4M3 codes
constexpr int kOffQ = kOffRing + kTcStages * kTcTileBytes;
static_assert(kOffRaw + kRawStages * kRawBytes <= kOffQ, "the 8-bit layout fits the room of the ring");
constexpr int kOffP = kOffQ + kTcSmall;              // two buffers
constexpr int kOffRed = kOffP + 2 * kTcSmall;        // [4 warps][8] floats: reductions over the softmax threads
constexpr int kOffBars = kOffRed + 4 * 8 * 4;
enum {
    kBarFull = 0,                        // [kTcStages] tile landed
    kBarEmpty = kBarFull + kTcStages,    // [kTcStages] tile read by the tensor cores
    kBarQ = kBarEmpty + kTcStages,       // queries landed
    kBarScores,                          // every score column of the split is in TMEM
    kBarPFull,                           // [2] P tile written (128 softmax threads)
    kBarPEmpty = kBarPFull + 2,          // [2] ... read by the tensor cores
    kBarOut = kBarPEmpty + 2,            // the output columns are final
    kBarRawFull,                                 // [kRawStages] 8-bit caches: codes landed
    kBarRawEmpty = kBarRawFull + kRawStages,     // [kRawStages] ... widened (128 softmax threads)
    kTcNumBars = kBarRawEmpty + kRawStages
};
constexpr int kOffMisc = kOffBars + kTcNumBars * 8;  // TMEM base, abort flag
constexpr int kTcSmem = kOffMisc + 16 + 1024;        // + slack for the 1024-byte alignment
static_assert(2 * (kTcSmem + 1024) <= 227 * 1024, "two blocks per SM");
static_assert(16 + 16 * kTcMaxTiles <= (int)kTcTmemCols, "TMEM columns");

struct AttendTcParams {
    const int32_t *seq_lens;
    float *out;                 // [batch][hq][d]
    float *partial;             // [P][splits][G][d + 2]: unnormalised output, maximum (base-2 domain), sum of weights
    int batch, hkv, hq, cap, splits, tiles_per_split;
    int32_t *status;
    long long wait_cycles;
    const int32_t *block_table; // paged caches: [P][cap / 128] page ids, else null
};

__device__ __forceinline__ void tmem_ld16(uint32_t taddr, uint32_t (&r)[16])
{
    asm volatile(
        "tcgen05.ld.sync.aligned.32x32b.x16.b32 {%0, %1, %2, %3, %4, %5, %6, %7, %8, %9, %10, %11, %12, %13, %14, %15}, [%16];"
        : "=r"(r[0]), "=r"(r[1]), "=r"(r[2]), "=r"(r[3]), "=r"(r[4]), "=r"(r[5]), "=r"(r[6]), "=r"(r[7]), "=r"(r[8]),
          "=r"(r[9]), "=r"(r[10]), "=r"(r[11]), "=r"(r[12]), "=r"(r[13]), "=r"(r[14]), "=r"(r[15])
        : "r"(taddr)
        : "memory");
}
__device__ __forceinline__ void tmem_wait16(uint32_t (&r)[16])
{
    asm volatile("tcgen05.wait::ld.sync.aligned;"
                 : "+r"(r[0]), "+r"(r[1]), "+r"(r[2]), "+r"(r[3]), "+r"(r[4]), "+r"(r[5]), "+r"(r[6]), "+r"(r[7]), "+r"(r[8]),
                   "+r"(r[9]), "+r"(r[10]), "+r"(r[11]), "+r"(r[12]), "+r"(r[13]), "+r"(r[14]), "+r"(r[15])
                 :: "memory");
}
// barrier among the 128 softmax threads only
__device__ __forceinline__ void softmax_sync() { asm volatile("bar.sync 1, 128;" ::: "memory"); }

// Byte offset of element (row g, column k) of a [16 x 128] bf16 operand kept as two K-major halves of 64 columns,
// 128-byte rows, 128-byte swizzle (the 16-byte chunk index of a row is XORed with the row's low three bits).
__device__ __forceinline__ uint32_t small_off(int g, int k)
{
    const int half = k >> 6, kk = k & 63;
    return (uint32_t)(half * (kTcSmall / 2) + g * 128 + ((((kk >> 3) ^ (g & 7)) << 4) | ((kk & 7) << 1)));
}

// With kFp8, kBarFull / kBarEmpty [0 .. kConvBufs) stand for the widened tiles (filled by the softmax threads, 128 arrivals).
// kSrc: 0 = bf16 caches of 128 dimensions (tiles go to the tensor cores as they land), 1 = E4M3 codes of 128 dimensions,
// 2 = bf16 caches of 64 dimensions (both: rows of 128 bytes, widened / padded with zeros into bf16 operand tiles of
// 128 dimensions; the queries of the 64-dimension case fill the first half of their operand, the rest stays zero).
template <int G, int kSrc>
__global__ void __launch_bounds__(kTcThreads, 2)
attend_tc_kernel(AttendTcParams p, const __grid_constant__ CUtensorMap map_k, const __grid_constant__ CUtensorMap map_v,
                 const __grid_constant__ CUtensorMap map_q)
{
    constexpr bool kFp8 = kSrc != 0;            // the tiles pass through the softmax threads on their way to the tensor cores
    constexpr int kDim = kSrc == 2 ? 64 : kHeadDim;          // head dimension of the caches, the queries and the output
    extern __shared__ uint8_t att_tc_raw[];
    uint8_t *smem = reinterpret_cast<uint8_t *>((reinterpret_cast<uintptr_t>(att_tc_raw) + 1023) & ~(uintptr_t)1023);
    const uint32_t sbase = smem_u32(smem);
    uint32_t *tmem_holder = reinterpret_cast<uint32_t *>(smem + kOffMisc);
    volatile int *abort_flag = reinterpret_cast<volatile int *>(smem + kOffMisc + 4);
    float *red = reinterpret_cast<float *>(smem + kOffRed);
    auto bar = [&](int i) { return sbase + kOffBars + 8 * i; };
    const ErrSink sink{p.status, nullptr, p.wait_cycles};

    const int head = blockIdx.x / p.splits, split = blockIdx.x % p.splits;
    const int b = head / p.hkv, h = head % p.hkv;
    const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
    int L = p.seq_lens[b];
    if (L < 0 || L > p.cap) {               // reported, and treated as an empty cache
        report(p.status, RKV_ERR_INVALID_ARG);
        L = 0;
    }
    const int t0 = split * p.tiles_per_split;                       // first key tile of this block
    const int T = min(min(p.tiles_per_split, kTcMaxTiles), (L + kTile - 1) / kTile - t0);      // its tiles (<= 0: none)
    constexpr int kStride = kHeadDim + 2;
    float *part = p.partial + ((size_t)head * p.splits + split) * G * kStride;
    float *out = p.out + ((size_t)b * p.hq + (size_t)h * G) * kDim;

    if (T <= 0) {       // no cached row falls into this split (uniform for the block: nothing was allocated yet)
        for (int x = threadIdx.x; x < G * kDim; x += kTcThreads) {
            const int g = x / kDim, c = x % kDim;
            if (p.splits == 1) {
                out[(size_t)g * kDim + c] = 0.f;
            } else {
                part[g * kStride + c] = 0.f;
                if (c == 0) {
                    part[g * kStride + kHeadDim] = -INFINITY;
                    part[g * kStride + kHeadDim + 1] = 0.f;
                }
            }
        }
        return;
    }

    if (threadIdx.x == 0) {
        for (int s = 0; s < kTcStages; ++s) {
            mbar_init(bar(kBarFull + s), kFp8 ? 128 : 1);
            mbar_init(bar(kBarEmpty + s), 1);
        }
        for (int s = 0; s < kRawStages; ++s) {
            mbar_init(bar(kBarRawFull + s), 1);
            mbar_init(bar(kBarRawEmpty + s), 128);
        }
        mbar_init(bar(kBarQ), 1);
        mbar_init(bar(kBarScores), 1);
        for (int s = 0; s < 2; ++s) {
            mbar_init(bar(kBarPFull + s), 128);
            mbar_init(bar(kBarPEmpty + s), 1);
        }
        mbar_init(bar(kBarOut), 1);
        *abort_flag = 0;
        asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory");
    }
    if (warp == 5) {
        asm volatile("tcgen05.alloc.cta_group::1.sync.aligned.shared::cta.b32 [%0], %1;"
                     ::"r"(smem_u32(tmem_holder)), "r"(kTcTmemCols) : "memory");
        asm volatile("tcgen05.relinquish_alloc_permit.cta_group::1.sync.aligned;" ::: "memory");
    }
    // the P buffers start as zeros: rows of queries the group does not have are never written (and so does the query
    // operand: with 64 dimensions only its first half is loaded)
    for (int x = threadIdx.x; x < 3 * kTcSmall / 16; x += kTcThreads)
        reinterpret_cast<uint4 *>(smem + kOffQ)[x] = make_uint4(0u, 0u, 0u, 0u);
    asm volatile("fence.proxy.async.shared::cta;" ::: "memory");
    tc_fence_before();
    __syncthreads();
    tc_fence_after();
    const uint32_t tmem = *tmem_holder;

    // where key tile t of the head starts, in rows of the 2-D [rows][d] view of the caches
    auto tile_y = [&](int t) -> int {
        return p.block_table ? p.block_table[(size_t)head * (p.cap / kTile) + t] * kTile : head * p.cap + t * kTile;
    };

    if (warp == 4) {
        // ------------------------------------------------------------------ TMA producer
        if (lane == 0) {
            mbar_expect_tx(bar(kBarQ), kSrc == 2 ? kTcSmall / 2 : kTcSmall);
            const int qy = b * p.hq + h * G;                 // the group's G query rows (the rows after them are not used)
            tma_load_2d(sbase + kOffQ, &map_q, 0, qy, bar(kBarQ));
            if (kSrc != 2) tma_load_2d(sbase + kOffQ + kTcSmall / 2, &map_q, 64, qy, bar(kBarQ));
            for (int i = 0; i < 2 * T; ++i) {                // the K tiles, then the V tiles
                const CUtensorMap *map = i < T ? &map_k : &map_v;
                const int y = tile_y(t0 + (i < T ? i : i - T));
                if (kFp8) {
                    const int s = i % kRawStages;
                    if (!mbar_wait(bar(kBarRawEmpty + s), ((i / kRawStages) & 1) ^ 1, abort_flag, sink)) break;
                    mbar_expect_tx(bar(kBarRawFull + s), kRawBytes);
                    tma_load_2d(sbase + kOffRaw + s * kRawBytes, map, 0, y, bar(kBarRawFull + s));
                } else {
                    const int s = i % kTcStages;
                    if (!mbar_wait(bar(kBarEmpty + s), ((i / kTcStages) & 1) ^ 1, abort_flag, sink)) break;
                    const uint32_t dst = sbase + kOffRing + s * kTcTileBytes;
                    mbar_expect_tx(bar(kBarFull + s), kTcTileBytes);
                    tma_load_2d(dst, map, 0, y, bar(kBarFull + s));
                    tma_load_2d(dst + kTcHalf, map, 64, y, bar(kBarFull + s));
                }
            }
        }
        __syncwarp();
    } else if (warp == 5) {
        // ------------------------------------------------------------------ MMA issuer
        if (lane == 0) {
            bool ok = mbar_wait(bar(kBarQ), 0, abort_flag, sink);
            const uint32_t idesc_s = instr_desc(kTile, 16);
            constexpr int kBufs = kFp8 ? kConvBufs : kTcStages;      // operand tiles the tensor cores read from
            for (int t = 0; t < T && ok; ++t) {              // scores of key tile t into its own 16 columns
                const int s = t % kBufs;
                ok = mbar_wait(bar(kBarFull + s), (t / kBufs) & 1, abort_flag, sink);
                if (!ok) break;
                tc_fence_after();
                umma_tile_k128_halves(tmem + 16 + 16 * t, sbase + kOffRing + s * kTcTileBytes, kTcHalf, sbase + kOffQ,
                                      kTcSmall / 2, idesc_s);
                umma_commit(bar(kBarEmpty + s));
            }
            if (ok) umma_commit(bar(kBarScores));
            // f32 accumulate, bf16 x bf16, A MN-major (bit 15), B K-major, M = 128, N = 16
            const uint32_t idesc_o = (1u << 4) | (1u << 7) | (1u << 10) | (1u << 15) | ((16u >> 3) << 17) | ((128u >> 4) << 24);
            for (int t = 0; t < T && ok; ++t) {              // O^T += V_t^T . P_t
                const int i = T + t, s = i % kBufs, pb = t & 1;
                ok = mbar_wait(bar(kBarFull + s), (i / kBufs) & 1, abort_flag, sink) &&
                     mbar_wait(bar(kBarPFull + pb), (t >> 1) & 1, abort_flag, sink);
                if (!ok) break;
                tc_fence_after();
                const uint32_t v_tile = sbase + kOffRing + s * kTcTileBytes, p_tile = sbase + kOffP + pb * kTcSmall;
#pragma unroll
                for (int ks = 0; ks < 8; ++ks) {             // 16 keys per step
                    const uint32_t a_addr = v_tile + ks * 2048;             // 16 rows of 128 bytes further
                    const uint32_t b_addr = p_tile + (ks >> 2) * (kTcSmall / 2) + (ks & 3) * 32;
                    // A: 64-element (128-byte) atoms along M 16 KB apart (the second TMA box), 8-row groups along K 1 KB apart
                    const uint64_t da = (uint64_t)((a_addr & 0x3FFFFu) >> 4) | ((uint64_t)(16384u >> 4) << 16) |
                                        ((uint64_t)(1024u >> 4) << 32) | ((uint64_t)1 << 46) | ((uint64_t)2 << 61);
                    umma(tmem, da, smem_desc(b_addr), idesc_o, (t > 0 || ks > 0) ? 1u : 0u);
                }
                umma_commit(bar(kBarEmpty + s));
                umma_commit(bar(kBarPEmpty + pb));
            }
            if (ok) umma_commit(bar(kBarOut));
        }
        __syncwarp();
    } else {
        // ------------------------------------------------------------------ softmax threads (warps 0..3)
        const int r = threadIdx.x;                                   // TMEM lane: key row of a tile, later output dimension
        const uint32_t lane_base = tmem + ((uint32_t)(warp * 32) << 16);
        const float c2 = 1.4426950408889634f * rsqrtf((float)kDim);          // scores in the base-2 domain
        // 8-bit caches: source tile i (the K tiles, then the V tiles) from its raw stage into a bf16 operand buffer, this
        // thread's row; a row beyond the length becomes zeros
        auto widen_tile = [&](int i) -> bool {
            const int s = i % kRawStages, cb = i % kConvBufs;
            if (!mbar_wait(bar(kBarRawFull + s), (i / kRawStages) & 1, abort_flag, sink)) return false;
            if (!mbar_wait(bar(kBarEmpty + cb), ((i / kConvBufs) & 1) ^ 1, abort_flag, sink)) return false;
            const bool row_valid = (t0 + (i < T ? i : i - T)) * kTile + r < L;
            const uint8_t *raw = smem + kOffRaw + s * kRawBytes + r * 128;
            uint8_t *dst = smem + kOffRing + cb * kTcTileBytes + r * 128;
            uint4 codes[8];                                  // the whole row first: the loads must not wait for the stores
#pragma unroll
            for (int c = 0; c < 8; ++c) codes[c] = *reinterpret_cast<const uint4 *>(raw + ((c ^ (r & 7)) << 4));
#pragma unroll
            for (int c = 0; c < 8; ++c) {                    // codes 16 c .. 16 c + 15 -> the row's bf16 chunks 2 c and 2 c + 1
                if (kSrc == 2) {                             // 64 dimensions: the row is the first half, the second half zeros
                    *reinterpret_cast<uint4 *>(dst + ((c ^ (r & 7)) << 4)) = row_valid ? codes[c] : make_uint4(0u, 0u, 0u, 0u);
                    *reinterpret_cast<uint4 *>(dst + kTcHalf + ((c ^ (r & 7)) << 4)) = make_uint4(0u, 0u, 0u, 0u);
                    continue;
                }
                uint4 lo = make_uint4(0u, 0u, 0u, 0u), hi = lo;
                if (row_valid) widen16(codes[c], &lo, &hi);
                const int half = c >> 2, pos = (2 * c) & 7;
                *reinterpret_cast<uint4 *>(dst + half * kTcHalf + ((pos ^ (r & 7)) << 4)) = lo;
                *reinterpret_cast<uint4 *>(dst + half * kTcHalf + (((pos + 1) ^ (r & 7)) << 4)) = hi;
            }
            asm volatile("fence.proxy.async.shared::cta;" ::: "memory");       // generic writes -> tensor-core reads
            mbar_arrive(bar(kBarFull + cb));
            mbar_arrive(bar(kBarRawEmpty + s));
            return true;
        };
        bool ok = true;
        if (kFp8)
            for (int t = 0; t < T && ok; ++t) ok = widen_tile(t);
        if (ok) ok = mbar_wait(bar(kBarScores), 0, abort_flag, sink);
        float m[G], l[G];
#pragma unroll
        for (int g = 0; g < G; ++g) m[g] = -INFINITY, l[g] = 0.f;
        if (ok) {
            tc_fence_after();
            for (int t = 0; t < T; ++t) {
                uint32_t acc[16];
                tmem_ld16(lane_base + 16 + 16 * t, acc);
                tmem_wait16(acc);
                const bool valid = (t0 + t) * kTile + r < L;
#pragma unroll
                for (int g = 0; g < G; ++g)
                    if (valid) m[g] = fmaxf(m[g], __uint_as_float(acc[g]) * c2);
            }
        }
#pragma unroll
        for (int g = 0; g < G; ++g) {
#pragma unroll
            for (int off = 16; off > 0; off >>= 1) m[g] = fmaxf(m[g], __shfl_xor_sync(0xffffffffu, m[g], off));
            if (lane == 0) red[warp * 8 + g] = m[g];
        }
        softmax_sync();
#pragma unroll
        for (int g = 0; g < G; ++g) m[g] = fmaxf(fmaxf(red[g], red[8 + g]), fmaxf(red[16 + g], red[24 + g]));
        softmax_sync();                                  // `red` is used again for the sums

        for (int t = 0; t < T && ok; ++t) {
            const int pb = t & 1;
            if (kFp8) ok = widen_tile(T + t);
            if (ok) ok = mbar_wait(bar(kBarPEmpty + pb), ((t >> 1) & 1) ^ 1, abort_flag, sink);
            if (!ok) break;
            uint32_t acc[16];
            tmem_ld16(lane_base + 16 + 16 * t, acc);
            tmem_wait16(acc);
            const bool valid = (t0 + t) * kTile + r < L;
            uint8_t *pt = smem + kOffP + pb * kTcSmall;
#pragma unroll
            for (int g = 0; g < G; ++g) {
                // (a NaN or infinite score of a row that is not cached never gets here: `valid` decides)
                const float w = valid ? exp2f(__uint_as_float(acc[g]) * c2 - m[g]) : 0.f;
                const __nv_bfloat16 hi = __float2bfloat16_rn(w);
                const __nv_bfloat16 lo = __float2bfloat16_rn(w - __bfloat162float(hi));
                l[g] += __bfloat162float(hi) + __bfloat162float(lo);
                *reinterpret_cast<__nv_bfloat16 *>(pt + small_off(g, r)) = hi;
                *reinterpret_cast<__nv_bfloat16 *>(pt + small_off(8 + g, r)) = lo;
            }
            if (!kFp8 && !valid) {
                // a row beyond the sequence's length may hold anything, and 0 x NaN would spoil the product: its V row
                // is cleared in shared memory (only the split's last tile has such rows)
                const int i = T + t, s = i % kTcStages;
                ok = mbar_wait(bar(kBarFull + s), (i / kTcStages) & 1, abort_flag, sink);
                if (ok) {
                    uint8_t *vt = smem + kOffRing + s * kTcTileBytes;
#pragma unroll
                    for (int c = 0; c < 8; ++c) {
                        *reinterpret_cast<uint4 *>(vt + r * 128 + c * 16) = make_uint4(0u, 0u, 0u, 0u);
                        *reinterpret_cast<uint4 *>(vt + kTcHalf + r * 128 + c * 16) = make_uint4(0u, 0u, 0u, 0u);
                    }
                }
            }
            asm volatile("fence.proxy.async.shared::cta;" ::: "memory");       // generic writes -> tensor-core reads
            mbar_arrive(bar(kBarPFull + pb));
        }

        // ---- the sums of the weights over the 128 key rows, then the output columns
#pragma unroll
        for (int g = 0; g < G; ++g) {
#pragma unroll
            for (int off = 16; off > 0; off >>= 1) l[g] += __shfl_xor_sync(0xffffffffu, l[g], off);
            if (lane == 0) red[warp * 8 + g] = l[g];
        }
        softmax_sync();
        if (ok) ok = mbar_wait(bar(kBarOut), 0, abort_flag, sink);
        uint32_t o[16];
#pragma unroll
        for (int c = 0; c < 16; ++c) o[c] = 0u;
        if (ok) {
            tc_fence_after();
            tmem_ld16(lane_base, o);
            tmem_wait16(o);
        }
#pragma unroll
        for (int g = 0; g < G; ++g) {
            const float den = ok ? (red[g] + red[8 + g]) + (red[16 + g] + red[24 + g]) : 0.f;     // error path: zeros
            const float num = __uint_as_float(o[g]) + __uint_as_float(o[8 + g]);
            if (r >= kDim) continue;                          // (64 dimensions: the padded half of the output)
            if (p.splits == 1) {
                out[(size_t)g * kDim + r] = den > 0.f ? num / den : 0.f;
            } else {
                part[g * kStride + r] = num;
                if (r == 0) {
                    part[g * kStride + kHeadDim] = ok ? m[g] : -INFINITY;
                    part[g * kStride + kHeadDim + 1] = den;
                }
            }
        }
    }

    // ---------------------------------------------------------------------- common exit
    tc_fence_before();
    __syncthreads();
    if (warp == 5) {
        if (*abort_flag) __nanosleep(200000);      // error path only: let copies and products in flight land
        tc_fence_after();
        asm volatile("tcgen05.dealloc.cta_group::1.sync.aligned.b32 %0, %1;" ::"r"(tmem), "r"(kTcTmemCols) : "memory");
    }
}

template <int G, int kSrc>
cudaError_t launch_tc_one(const AttendTcParams &p, const CUtensorMap &mk, const CUtensorMap &mv, const CUtensorMap &mq,
                          cudaStream_t s)
{
    cudaError_t e = cudaFuncSetAttribute(attend_tc_kernel<G, kSrc>, cudaFuncAttributeMaxDynamicSharedMemorySize, kTcSmem);
    if (e != cudaSuccess) return e;
    attend_tc_kernel<G, kSrc><<<(unsigned)(p.batch * p.hkv * p.splits), kTcThreads, kTcSmem, s>>>(p, mk, mv, mq);
    return cudaGetLastError();
}
template <int G>
cudaError_t launch_tc_for(const AttendTcParams &p, int src, const CUtensorMap &mk, const CUtensorMap &mv, const CUtensorMap &mq,
                          cudaStream_t s)
{
    return src == 1 ? launch_tc_one<G, 1>(p, mk, mv, mq, s) : src == 2 ? launch_tc_one<G, 2>(p, mk, mv, mq, s)
                                                                          : launch_tc_one<G, 0>(p, mk, mv, mq, s);
}

}  // namespace

// Splits of a head's key tiles for the tensor-core kernel: enough blocks for two waves of resident blocks (2 per SM),
// never more than kTcMaxTiles tiles per block, never finer than a tile.
int attend_tc_splits(int heads, int cap, int sms)
{
    const int tiles = (cap + kTile - 1) / kTile;
    int splits = (4 * sms + heads - 1) / heads;
    const int least = (tiles + kTcMaxTiles - 1) / kTcMaxTiles;
    splits = splits < least ? least : splits;
    return splits > tiles ? tiles : splits;
}

cudaError_t launch_attend_tc(const void *k_cache, const void *v_cache, const void *q_new, const int32_t *seq_lens, float *out,
                             float *partial, int batch, int hkv, int hq, int cap, int splits, int32_t *status,
                             long long wait_cycles, const int32_t *block_table, long long pool_pages, int src, cudaStream_t s)
{
    const int tiles = (cap + kTile - 1) / kTile;
    AttendTcParams p;
    p.seq_lens = seq_lens;
    p.out = out;
    p.partial = partial;
    p.batch = batch;
    p.hkv = hkv;
    p.hq = hq;
    p.cap = cap;
    p.splits = splits;
    p.tiles_per_split = (tiles + splits - 1) / splits;
    p.status = status;
    p.wait_cycles = wait_cycles;
    p.block_table = block_table;
    if (p.tiles_per_split > kTcMaxTiles) return cudaErrorInvalidValue;
    const uint64_t rows = block_table ? (uint64_t)pool_pages * kTile : (uint64_t)batch * hkv * cap;
    CUtensorMap mk, mv, mq;
    // src: 0 = bf16 caches of 128 dimensions, 1 = E4M3 codes of 128 dimensions, 2 = bf16 caches of 64 dimensions
    const bool maps_ok = src != 0 ? (sm100::make_map_row128(&mk, k_cache, rows, src == 1) && sm100::make_map_row128(&mv, v_cache, rows, src == 1))
                                  : (sm100::make_map(&mk, k_cache, rows, kTile) && sm100::make_map(&mv, v_cache, rows, kTile));
    const bool q_ok = src == 2 ? sm100::make_map_q64(&mq, q_new, (uint64_t)batch * hq) : sm100::make_map(&mq, q_new, (uint64_t)batch * hq, 16);
    if (!maps_ok || !q_ok) return cudaErrorInvalidValue;
    switch (hq / hkv) {
        case 1: return launch_tc_for<1>(p, src, mk, mv, mq, s);
        case 2: return launch_tc_for<2>(p, src, mk, mv, mq, s);
        case 3: return launch_tc_for<3>(p, src, mk, mv, mq, s);
        case 4: return launch_tc_for<4>(p, src, mk, mv, mq, s);
        case 5: return launch_tc_for<5>(p, src, mk, mv, mq, s);
        case 6: return launch_tc_for<6>(p, src, mk, mv, mq, s);
        case 7: return launch_tc_for<7>(p, src, mk, mv, mq, s);
        case 8: return launch_tc_for<8>(p, src, mk, mv, mq, s);
        default: return cudaErrorInvalidValue;
    }
}

}  // namespace rkv

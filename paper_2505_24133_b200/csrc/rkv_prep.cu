// Stage "prep": one streaming pass over the candidate keys.
//
// For every key row i of every head it produces r_i = 1 / (||k_i||_2 + eps), the normalisation
// factor of Eq. 5, and per 128-row tile the vector sum_i r_i * k_i.  The tile sums let the
// scoring stage obtain sum_j S[j][i] = Kbar_i . (sum_j Kbar_j) - Kbar_i . Kbar_i (Eq. 6 before the
// retention rule) without accumulating the n x n matrix element by element.
// Rows i >= n (observation tokens, unused capacity) get r_i = 0 and contribute nothing.
// The last block to finish a head also leaves sum_i r_i * k_i over the whole head (head_sum).
// Kbar_i . Kbar_i is kept per row as well (self_dot).
//
// HBM-bound: each block brings its tile of K into shared memory with one bulk copy (cp.async.bulk, bounded wait
// on its mbarrier) and reads it from there; the row norm is reduced with warp shuffles.  Outputs are 8 bytes per
// 256-byte row.
#include <algorithm>

#include "rkv_sm100.cuh"

namespace rkv {

namespace {

constexpr int kPrepThreads = 256;
constexpr int kPrepWarps = kPrepThreads / 32;

template <typename T, int D>
__global__ void __launch_bounds__(kPrepThreads, D <= 128 ? 5 : 2) prep_kernel(Params p)
{
    using namespace sm100;
    extern __shared__ __align__(128) uint8_t prep_smem[];       // the tile's candidate rows, then one mbarrier
    constexpr int kTileBytesT = kTile * D * (int)sizeof(T);
    __shared__ int abort_flag;
    const ErrSink sink = make_sink(p);
    constexpr int kPerVec = Elem<T>::kPerVec;            // elements per 16-byte vector
    constexpr int kVecPerLane = 2;                       // 16-byte vectors of a row held by one lane
    constexpr int kLanesPerRow = D / (kPerVec * kVecPerLane);     // 8 (bf16) or 16 (fp32)
    constexpr int kVecPerRow = D / kPerVec;
    constexpr int kRowsPerPass = 32 / kLanesPerRow;      // rows a warp covers with one load
    constexpr int kRowsPerWarp = kTile / kPrepWarps;     // 16
    constexpr int kPasses = kRowsPerWarp / kRowsPerPass;

    const int tile = blockIdx.x % p.tiles;
    const int head = blockIdx.x / p.tiles;               // head-problem index b * hkv + h
    const int b = head / p.hkv;
    const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;

    int L = p.seq_lens[b];
    int budget_b = p.budgets ? p.budgets[b] : p.budget;             // Section 4.2's per-sequence (ratio) budgets
    if (L < 0 || L > p.cap || budget_b <= p.alpha || budget_b > p.budget) {
        report(p.status, RKV_ERR_INVALID_ARG);
        L = kMetaInvalid;
        budget_b = p.budget;
    }
    if (tile == 0 && head % p.hkv == 0 && threadIdx.x == 0) {
        p.meta[b] = L;
        p.meta[p.batch + b] = budget_b;
    }
    const int n = candidates_from_meta(L, budget_b, p.alpha);

    const T *K_tile = static_cast<const T *>(p.k_cache) + (size_t)tile_row0(p, head, tile) * D;      // the tile's first row
    float *inv_norm = p.inv_norm + (size_t)head * p.cap_pad;

    const int sub = lane / kLanesPerRow;                 // which of the rows of this pass
    const int lane_in_row = lane % kLanesPerRow;         // vector u of the lane = vector lane_in_row + u * kLanesPerRow
                                                         // of the row: a warp's load covers whole 128-byte lines

    // One bulk copy brings the tile's candidate rows (contiguous in memory) into shared memory: the bytes in
    // flight cost no registers, so several blocks per SM keep HBM busy.
    const int rows_here = min(max(n - tile * kTile, 0), kTile);
    const uint32_t bar = smem_u32(prep_smem + kTileBytesT);
    if (threadIdx.x == 0) {
        abort_flag = 0;
        mbar_init(bar, 1);
        asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory");
        if (rows_here > 0) {
            const uint32_t bytes = (uint32_t)rows_here * D * (uint32_t)sizeof(T);
            mbar_expect_tx(bar, bytes);
            asm volatile("cp.async.bulk.shared::cluster.global.mbarrier::complete_tx::bytes [%0], [%1], %2, [%3];"
                         ::"r"(smem_u32(prep_smem)), "l"(K_tile), "r"(bytes), "r"(bar)
                         : "memory");
        }
    }
    __syncthreads();
    const bool landed = rows_here == 0 || mbar_wait(bar, 0, &abort_flag, sink);
    if (!__syncthreads_and(landed)) {      // the block leaves as a whole, or not at all
        __nanosleep(200000);               // error path only: let the copy land before the block's memory is reused
        return;
    }
    const uint4 *tile_s = reinterpret_cast<const uint4 *>(prep_smem);
    // packed fp32 arithmetic (two values per instruction), few lanes per row (short shuffle trees): this kernel is
    // bound by its instruction count
    constexpr int kHeld = kPerVec * kVecPerLane;         // elements of a row per lane
    float2 acc2[kHeld / 2];
#pragma unroll
    for (int e = 0; e < kHeld / 2; ++e) acc2[e] = make_float2(0.f, 0.f);

    float r_keep[kPasses];               // r of this lane's row in every pass (for the slices written after the loop)
#pragma unroll
    for (int q = 0; q < kPasses; ++q) {
        const int lr = warp * kRowsPerWarp + q * kRowsPerPass + sub;       // row within the tile
        const int row = tile * kTile + lr;
        float f[kHeld];
#pragma unroll
        for (int u = 0; u < kVecPerLane; ++u) {
            uint4 vec = make_uint4(0u, 0u, 0u, 0u);
            if (lr < rows_here) vec = tile_s[lr * kVecPerRow + lane_in_row + u * kLanesPerRow];
            Elem<T>::unpack(vec, f + u * kPerVec);
        }
        float2 sq2 = make_float2(0.f, 0.f);
#pragma unroll
        for (int e = 0; e < kHeld / 2; ++e) {
            const float2 f2 = make_float2(f[2 * e], f[2 * e + 1]);
            sq2 = __ffma2_rn(f2, f2, sq2);
        }
        float sq = sq2.x + sq2.y;
#pragma unroll
        for (int off = kLanesPerRow / 2; off > 0; off >>= 1) sq += __shfl_xor_sync(0xffffffffu, sq, off);
        // 1 / (sqrt(sq) + eps) from the hardware's approximate rsqrt and divide (a few ulp: far inside the score
        // tolerances, and every scoring kernel uses these same r); sq = 0 (an all-zero key) gives 1 / eps
        const float nrm = sq > 0.f ? sq * rsqrtf(sq) : 0.f;
        const float r = (row < n) ? __fdividef(1.0f, nrm + p.eps) : 0.f;
        if (lane_in_row == 0) {
            inv_norm[row] = r;                       // row < cap_pad: the grid covers exactly cap_pad rows per head
            p.self_dot[(size_t)head * p.cap_pad + row] = (r * r) * sq;     // Kbar_i . Kbar_i
        }
        r_keep[q] = r;
        const float2 r2 = make_float2(r, r);
#pragma unroll
        for (int e = 0; e < kHeld / 2; ++e) acc2[e] = __ffma2_rn(r2, make_float2(f[2 * e], f[2 * e + 1]), acc2[e]);
    }

    if (p.tri) {
        // The threshold test of Section 3.3, S[j][i] > T, as the sign of k_i . k_j - T / (r_i r_j): the tensor-core kernels
        // append one K = 16 step to a tile product whose operands are these slices.  1 / r = ||k|| + eps in three bf16
        // parts (their sum has fp32 accuracy) as (n1, n2, n3, n1, n2, n1, 0 ...) for a key row; its dot product with a
        // row's (-t1, -t1, -t1, -t2, -t2, -t3, 0 ...), the parts of T / r, is -T / (r_i r_j) up to terms of size 2^-24.
        // One lane per row of the warp's 16 rows: lane l takes row l, whose r sits with the first lane of its group.
        float r_mine = 0.f;
#pragma unroll
        for (int q = 0; q < kPasses; ++q) {
            const float v = __shfl_sync(0xffffffffu, r_keep[q], (lane % kRowsPerPass) * kLanesPerRow);
            if (lane / kRowsPerPass == q) r_mine = v;
        }
        if (lane < kRowsPerWarp) {
            const int lr = warp * kRowsPerWarp + lane, row = tile * kTile + lr;
            float rest = r_mine > 0.f ? __fdiv_rn(1.0f, r_mine) : 0.f;
            uint32_t part[3];
#pragma unroll
            for (int c = 0; c < 3; ++c) {
                const __nv_bfloat16 h16 = __float2bfloat16_rn(rest);
                part[c] = (uint32_t)__bfloat16_as_ushort(h16);
                rest -= __bfloat162float(h16);
            }
            uint4 *dst = reinterpret_cast<uint4 *>(p.norm_split + ((size_t)head * p.cap_pad + row) * 16);
            dst[0] = make_uint4(part[0] | (part[1] << 16), part[2] | (part[0] << 16), part[1] | (part[0] << 16), 0u);
            dst[1] = make_uint4(0u, 0u, 0u, 0u);
            if (tile == (n + kTile - 1) / kTile - 1) {       // the head's last key tile: the first pass's resident operand
                rest = r_mine > 0.f ? -__fdiv_rn(p.sim_threshold, r_mine) : 0.f;
#pragma unroll
                for (int c = 0; c < 3; ++c) {
                    const __nv_bfloat16 h16 = __float2bfloat16_rn(rest);
                    part[c] = (uint32_t)__bfloat16_as_ushort(h16);
                    rest -= __bfloat162float(h16);
                }
                uint4 *thr = reinterpret_cast<uint4 *>(p.thr_split + ((size_t)head * kTile + lr) * 16);
                thr[0] = make_uint4(part[0] | (part[0] << 16), part[0] | (part[1] << 16), part[1] | (part[2] << 16), 0u);
                thr[1] = make_uint4(0u, 0u, 0u, 0u);
            }
        }
    }

    // fold the row groups of a warp, then the warps, in a fixed order (deterministic sums)
#pragma unroll
    for (int off = kLanesPerRow; off < 32; off <<= 1) {
#pragma unroll
        for (int e = 0; e < kHeld / 2; ++e) {
            acc2[e].x += __shfl_xor_sync(0xffffffffu, acc2[e].x, off);
            acc2[e].y += __shfl_xor_sync(0xffffffffu, acc2[e].y, off);
        }
    }
    __shared__ float part[kPrepWarps][D];
    if (sub == 0) {
#pragma unroll
        for (int u = 0; u < kVecPerLane; ++u) {
            const int col = (lane_in_row + u * kLanesPerRow) * kPerVec;
#pragma unroll
            for (int e = 0; e < kPerVec / 2; ++e) {
                part[warp][col + 2 * e] = acc2[u * kPerVec / 2 + e].x;
                part[warp][col + 2 * e + 1] = acc2[u * kPerVec / 2 + e].y;
            }
        }
    }
    __syncthreads();
    if (threadIdx.x < D) {
        float s = 0.f;
#pragma unroll
        for (int w = 0; w < kPrepWarps; ++w) s += part[w][threadIdx.x];
        p.tile_sum[((size_t)head * p.tiles + tile) * D + threadIdx.x] = s;
    }

    // The block that finishes a head's last tile adds the tile sums up, always in tile order, so the result does
    // not depend on which block that is.  (tile_done is zeroed by the memset that precedes this kernel.)
    __shared__ bool last_block;
    __syncthreads();                       // the block's tile sums are written ...
    if (threadIdx.x == 0) {
        __threadfence();                   // ... and made visible device-wide before the ticket is drawn
        last_block = (atomicAdd(&p.tile_done[head], 1u) == (unsigned)p.tiles - 1u);
    }
    __syncthreads();
    if (last_block && threadIdx.x < D) {
        __threadfence();
        const float *ts = p.tile_sum + (size_t)head * p.tiles * D + threadIdx.x;
        float s = 0.f;
        for (int t = 0; t < p.tiles; ++t) s += __ldcg(ts + (size_t)t * D);
        p.head_sum[(size_t)head * D + threadIdx.x] = s;
        // the same vector as three bf16 rows whose sum is s to fp32 accuracy (rows 3..15 of the 16-row block are
        // zero): appended to the query rows, it lets the tensor cores form Kbar_i . s along with the logits
        __nv_bfloat16 *hs = p.head_sum_bf16 + (size_t)head * 16 * D + threadIdx.x;
        float rest = s;
#pragma unroll
        for (int part_i = 0; part_i < 3; ++part_i) {
            const __nv_bfloat16 h16 = __float2bfloat16_rn(rest);
            hs[part_i * D] = h16;
            rest -= __bfloat162float(h16);
        }
        for (int z = 3; z < 16; ++z) hs[z * D] = __float2bfloat16_rn(0.f);
    }
}

// ---- the same stage for bf16 caches with d = 128 (the tensor-core route): sum_i r_i k_i on the tensor cores ------------
//
// The norms stay on the CUDA cores, one thread per row (the row read from shared memory once, packed fp32).  The
// weighted column sums sum_i r_i k_i[c] -- what made the kernel above instruction-bound -- are ONE small tensor-core
// product per tile: the key tile as TMA leaves it (rows of 128 d-elements, 128-byte swizzle) is used TRANSPOSED as the A
// operand (MN-major: M = d, K = the 128 rows), the B operand holds r_i in three bf16 parts (N = 16, rows 0..2), so
// D[c][0..2] sum to sum_i r_i k_i[c] to fp32 accuracy.  Eight K = 16 steps, accumulator = 16 TMEM columns.
constexpr int kPrepTcThreads = 128;                         // one thread per row of the tile
constexpr int kPrepTcTile = kTile * kHeadDim * 2;          // 32 KB
constexpr int kPrepTcB = 8 * 16 * 32;                      // 8 K-steps x [16 n][16 k] bf16, 32-byte rows (32-byte swizzle)
constexpr int kPrepTcBufs = 2;                             // tile buffers of a block: one in use, the others being filled
constexpr int kPrepTcBlocks = 3;                           // blocks per SM
constexpr int kPrepTcSmem = kPrepTcBufs * kPrepTcTile + kPrepTcB + 1024; // + slack for the 1024-byte alignment
constexpr uint32_t kPrepTcTmemCols = 32;

// One key tile of the work list: which head-problem, which tile, how many candidate rows it holds.
struct PrepTile {
    int head, tile, b, n, rows_here;
};

__device__ __forceinline__ PrepTile prep_tile_at(const Params &p, int idx, bool write_meta)
{
    PrepTile w;
    w.tile = idx % p.tiles;
    w.head = idx / p.tiles;               // head-problem index b * hkv + h
    w.b = w.head / p.hkv;
    int L = p.seq_lens[w.b];
    int budget_b = p.budgets ? p.budgets[w.b] : p.budget;             // Section 4.2's per-sequence (ratio) budgets
    if (L < 0 || L > p.cap || budget_b <= p.alpha || budget_b > p.budget) {
        if (write_meta) report(p.status, RKV_ERR_INVALID_ARG);
        L = kMetaInvalid;
        budget_b = p.budget;
    }
    if (write_meta && w.tile == 0 && w.head % p.hkv == 0) {
        p.meta[w.b] = L;
        p.meta[p.batch + w.b] = budget_b;
    }
    w.n = candidates_from_meta(L, budget_b, p.alpha);
    w.rows_here = min(max(w.n - w.tile * kTile, 0), kTile);
    return w;
}

// Persistent: kPrepTcBlocks blocks per SM, block x takes tiles x, x + gridDim.x, ... of the list (head-major) and
// keeps the copies of its next kPrepTcBufs - 1 tiles in flight while it works on the present one: what bounds this
// kernel is how many bytes an SM has under way, not what it does with them.  Barriers, the TMEM columns and the tensor
// map are set up once per block.
__global__ void __launch_bounds__(kPrepTcThreads, kPrepTcBlocks) prep_tc_kernel(Params p, const __grid_constant__ CUtensorMap map_k, int total)
{
    using namespace sm100;
    constexpr int D = kHeadDim;
    extern __shared__ uint8_t prep_tc_raw[];
    uint8_t *smem = reinterpret_cast<uint8_t *>((reinterpret_cast<uintptr_t>(prep_tc_raw) + 1023) & ~(uintptr_t)1023);
    uint8_t *bop = smem + kPrepTcBufs * kPrepTcTile;
    const uint32_t sbase = smem_u32(smem);
    __shared__ __align__(8) unsigned long long bars[kPrepTcBufs + 1];      // tile landed (per buffer); product done
    __shared__ uint32_t tmem_holder;
    __shared__ int abort_flag;
    const ErrSink sink = make_sink(p);
    const int t = threadIdx.x, warp = t >> 5;
    const uint32_t bar_tile0 = smem_u32(&bars[0]), bar_mma = smem_u32(&bars[kPrepTcBufs]);

    // thread 0: the tile of the block's k-th list entry into buffer k % kPrepTcBufs; an entry without candidates
    // completes the buffer's barrier phase without a copy, so phases and entries stay in step
    auto issue_copy = [&](int k) {
        const long long idx = (long long)blockIdx.x + (long long)k * gridDim.x;
        if (idx >= total) return;
        const PrepTile w = prep_tile_at(p, (int)idx, false);
        const int buf = k % kPrepTcBufs;
        const uint32_t bar = bar_tile0 + 8u * buf;
        if (w.rows_here <= 0) {
            mbar_arrive(bar);
            return;
        }
        const int y = (int)tile_row0(p, w.head, w.tile);
        mbar_expect_tx(bar, kPrepTcTile);
        tma_load_2d(sbase + buf * kPrepTcTile, &map_k, 0, y, bar);
        tma_load_2d(sbase + buf * kPrepTcTile + kPrepTcTile / 2, &map_k, 64, y, bar);
    };

    if (t == 0) {
        abort_flag = 0;
        for (int q = 0; q < kPrepTcBufs; ++q) mbar_init(bar_tile0 + 8u * q, 1);
        mbar_init(bar_mma, 1);
        asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory");
        for (int q = 0; q < kPrepTcBufs - 1; ++q) issue_copy(q);
    }
    if (warp == 0) {
        asm volatile("tcgen05.alloc.cta_group::1.sync.aligned.shared::cta.b32 [%0], %1;"
                     ::"r"(smem_u32(&tmem_holder)), "r"(kPrepTcTmemCols) : "memory");
        asm volatile("tcgen05.relinquish_alloc_permit.cta_group::1.sync.aligned;" ::: "memory");
    }
    // rows 3..15 of the B operand stay zero; rows 0..2 are rewritten in full for every tile
    for (int x = t; x < kPrepTcB / 16; x += kPrepTcThreads) reinterpret_cast<uint4 *>(bop)[x] = make_uint4(0u, 0u, 0u, 0u);
    tc_fence_before();
    __syncthreads();
    tc_fence_after();
    const uint32_t tmem = tmem_holder;
    uint32_t mma_parity = 0;

    int k = 0;
    for (int idx = (int)blockIdx.x; idx < total; idx += (int)gridDim.x, ++k) {
        const PrepTile w = prep_tile_at(p, idx, t == 0);
        const int head = w.head, tile = w.tile, n = w.n, rows_here = w.rows_here;
        const int buf = k % kPrepTcBufs;
        uint8_t *tile_smem = smem + buf * kPrepTcTile;
        // the buffer entry k - 1 used is free (its product was waited for, by every thread, before the last barrier)
        if (t == 0) issue_copy(k + kPrepTcBufs - 1);

        const bool landed = mbar_wait(bar_tile0 + 8u * buf, (uint32_t)(k / kPrepTcBufs) & 1u, &abort_flag, sink);
        const bool ok = __syncthreads_and(landed);           // the block goes on as a whole, or not at all

        // ---- one thread per row: norm, r, the slices; rows that are not candidates are cleared in shared memory
        // (they may hold anything, and 0 x NaN would spoil the product).  Two threads per row were measured slower:
        // the time of a tile is a chain of latencies (barrier, shared-memory loads, product, TMEM load), not of issue slots.
        const int rt = t;
        const int row = tile * kTile + rt;
        float r = 0.f, sq = 0.f;
        if (ok && rows_here > 0) {
            if (rt < rows_here) {
                float2 sq2[4];                       // four independent chains of packed multiply-adds
#pragma unroll
                for (int e = 0; e < 4; ++e) sq2[e] = make_float2(0.f, 0.f);
#pragma unroll
                for (int c = 0; c < 16; ++c) {
                    const uint4 vec = *reinterpret_cast<const uint4 *>(tile_smem + (c >> 3) * (kPrepTcTile / 2) + rt * 128 + (((c & 7) ^ (rt & 7)) << 4));
                    float f[8];
                    Elem<__nv_bfloat16>::unpack(vec, f);
#pragma unroll
                    for (int e = 0; e < 4; ++e) {
                        const float2 f2 = make_float2(f[2 * e], f[2 * e + 1]);
                        sq2[e] = __ffma2_rn(f2, f2, sq2[e]);
                    }
                }
                sq = ((sq2[0].x + sq2[0].y) + (sq2[1].x + sq2[1].y)) + ((sq2[2].x + sq2[2].y) + (sq2[3].x + sq2[3].y));
            } else {
#pragma unroll
                for (int c = 0; c < 16; ++c)
                    *reinterpret_cast<uint4 *>(tile_smem + (c >> 3) * (kPrepTcTile / 2) + rt * 128 + ((c & 7) << 4)) = make_uint4(0u, 0u, 0u, 0u);
            }
            if (rt < rows_here) {
                const float nrm = sq > 0.f ? sq * rsqrtf(sq) : 0.f;
                r = __fdividef(1.0f, nrm + p.eps);
            }
        }
        if (ok) {
            // r in three bf16 parts: row t of the B operand's K dimension, rows 0..2 of its N dimension
            float rest = r;
            uint32_t rp[3];
#pragma unroll
            for (int c = 0; c < 3; ++c) {
                const __nv_bfloat16 h16 = __float2bfloat16_rn(rest);
                rp[c] = (uint32_t)__bfloat16_as_ushort(h16);
                rest -= __bfloat162float(h16);
            }
            const int s = rt >> 4, kk = rt & 15;
#pragma unroll
            for (int nn = 0; nn < 3; ++nn)
                *reinterpret_cast<unsigned short *>(bop + s * 512 + nn * 32 + ((kk >> 3) << 4) + (kk & 7) * 2) = (unsigned short)rp[nn];
        }
        asm volatile("fence.proxy.async.shared::cta;" ::: "memory");       // generic writes -> tensor-core reads
        __syncthreads();

        // ---- sum_i r_i k_i[c]: D[c][nn] = sum_i K[i][c] R[nn][i], the tile as an MN-major operand
        if (ok && rows_here > 0 && t == 0) {
            // f32 accumulate, bf16 x bf16, A MN-major (bit 15), B K-major, M = 128, N = 16
            const uint32_t idesc = (1u << 4) | (1u << 7) | (1u << 10) | (1u << 15) | ((16u >> 3) << 17) | ((128u >> 4) << 24);
            tc_fence_after();
#pragma unroll
            for (int ks = 0; ks < 8; ++ks) {
                const uint32_t a_addr = sbase + buf * kPrepTcTile + ks * 2048;    // 16 rows of 128 bytes further
                const uint32_t b_addr = sbase + kPrepTcBufs * kPrepTcTile + ks * 512;
                // A: 64-element (128-byte) atoms along M 16 KB apart (the second TMA box), 8-row groups along K 1 KB apart
                uint64_t da = (uint64_t)((a_addr & 0x3FFFFu) >> 4) | ((uint64_t)(16384u >> 4) << 16) | ((uint64_t)(1024u >> 4) << 32) |
                              ((uint64_t)1 << 46) | ((uint64_t)2 << 61);
                // B: 32-byte rows, 8-row groups 256 B apart, 32-byte swizzle
                uint64_t db = (uint64_t)((b_addr & 0x3FFFFu) >> 4) | ((uint64_t)1 << 16) | ((uint64_t)(256u >> 4) << 32) |
                              ((uint64_t)1 << 46) | ((uint64_t)6 << 61);
                asm volatile("{\n\t.reg .pred pp;\n\tsetp.ne.b32 pp, %4, 0;\n\ttcgen05.mma.cta_group::1.kind::f16 [%0], %1, %2, %3, pp;\n\t}"
                             ::"r"(tmem), "l"(da), "l"(db), "r"(idesc), "r"(ks) : "memory");
            }
            umma_commit(bar_mma);
        }

        // ---- what a row leaves behind, written while the product runs
        if (ok) {
            p.inv_norm[(size_t)head * p.cap_pad + row] = r;
            p.self_dot[(size_t)head * p.cap_pad + row] = (r * r) * sq;     // Kbar_i . Kbar_i
            if (p.tri) {
                // the threshold slices of the scoring kernels (see prep_kernel above): 1 / r as (n1, n2, n3, n1, n2, n1, 0 ...),
                // and for the head's last key tile -T / r as (-t1, -t1, -t1, -t2, -t2, -t3, 0 ...)
                float rest = r > 0.f ? __fdiv_rn(1.0f, r) : 0.f;
                uint32_t part[3];
#pragma unroll
                for (int c = 0; c < 3; ++c) {
                    const __nv_bfloat16 h16 = __float2bfloat16_rn(rest);
                    part[c] = (uint32_t)__bfloat16_as_ushort(h16);
                    rest -= __bfloat162float(h16);
                }
                uint4 *dst = reinterpret_cast<uint4 *>(p.norm_split + ((size_t)head * p.cap_pad + row) * 16);
                dst[0] = make_uint4(part[0] | (part[1] << 16), part[2] | (part[0] << 16), part[1] | (part[0] << 16), 0u);
                dst[1] = make_uint4(0u, 0u, 0u, 0u);
                if (tile == (n + kTile - 1) / kTile - 1) {
                    rest = r > 0.f ? -__fdiv_rn(p.sim_threshold, r) : 0.f;
#pragma unroll
                    for (int c = 0; c < 3; ++c) {
                        const __nv_bfloat16 h16 = __float2bfloat16_rn(rest);
                        part[c] = (uint32_t)__bfloat16_as_ushort(h16);
                        rest -= __bfloat162float(h16);
                    }
                    uint4 *thr = reinterpret_cast<uint4 *>(p.thr_split + ((size_t)head * kTile + rt) * 16);
                    thr[0] = make_uint4(part[0] | (part[0] << 16), part[0] | (part[1] << 16), part[1] | (part[2] << 16), 0u);
                    thr[1] = make_uint4(0u, 0u, 0u, 0u);
                }
            }
        }

        float tsum = 0.f;
        bool done = ok;
        if (ok && rows_here > 0) {
            done = mbar_wait(bar_mma, mma_parity, &abort_flag, sink);
            mma_parity ^= 1u;
            if (done) {
                tc_fence_after();
                uint32_t acc[8];
                tmem_ld8(tmem + ((uint32_t)(warp * 32) << 16), acc);      // lane = column c of the keys
                tmem_wait8(acc);
                tsum = (__uint_as_float(acc[0]) + __uint_as_float(acc[1])) + __uint_as_float(acc[2]);
            }
        }
        tc_fence_before();
        done = __syncthreads_and(done);
        p.tile_sum[((size_t)head * p.tiles + tile) * D + t] = done ? tsum : 0.f;
        if (!done) break;
    }

    tc_fence_before();
    __syncthreads();
    if (warp == 0) {
        if (abort_flag) __nanosleep(200000);       // error path only: let the copies in flight land
        tc_fence_after();
        asm volatile("tcgen05.dealloc.cta_group::1.sync.aligned.b32 %0, %1;" ::"r"(tmem), "r"(kPrepTcTmemCols) : "memory");
    }
}

// ---- the same kernel for caches that are scored on a copy: 8-bit codes (d = 128) and bf16 keys of 64 dimensions --------
//
// Both store a key in 128 bytes.  The tile arrives as stored (16 KB, a ring of two stages); the thread that owns a row
// widens / pads it into the bf16 operand tile, taking the norm on the way; the tensor cores form the key sums from that
// tile as above, and the same tile is written out, by TMA, as the head's part of the scoring copy, which the later
// stages read.  The stored keys are read once and the copy is not read back here: a separate widening pass in front
// of prep_tc_kernel cost the prep stage a second sweep over keys twice the stored size.  Only for caches whose
// capacity is a whole number of tiles (a tile's store must not reach into the next head's rows).
constexpr int kFusedRaw = kTile * 128;                      // a stored tile: 16 KB
constexpr int kFusedOffRaw = kPrepTcBufs * kPrepTcTile;
constexpr int kFusedOffB = kFusedOffRaw + 2 * kFusedRaw;
constexpr int kFusedSmem = kFusedOffB + kPrepTcB + 1024;
constexpr int kFusedBlocks = 2;

template <bool kCodes>
__global__ void __launch_bounds__(kPrepTcThreads, kFusedBlocks)
prep_fused_kernel(Params p, const __grid_constant__ CUtensorMap map_src, const __grid_constant__ CUtensorMap map_wide,
                  const int32_t *src_table, int total)
{
    using namespace sm100;
    constexpr int D = kHeadDim;
    extern __shared__ uint8_t prep_tc_raw[];
    uint8_t *smem = reinterpret_cast<uint8_t *>((reinterpret_cast<uintptr_t>(prep_tc_raw) + 1023) & ~(uintptr_t)1023);
    uint8_t *bop = smem + kFusedOffB;
    const uint32_t sbase = smem_u32(smem);
    __shared__ __align__(8) unsigned long long bars[3];      // stored tile landed (per stage); product done
    __shared__ uint32_t tmem_holder;
    __shared__ int abort_flag;
    const ErrSink sink = make_sink(p);
    const int t = threadIdx.x, warp = t >> 5;
    const uint32_t bar_raw0 = smem_u32(&bars[0]), bar_mma = smem_u32(&bars[2]);

    // thread 0: the stored tile of the block's k-th list entry into stage k % 2 (an entry without candidates completes
    // the stage's barrier phase without a copy)
    auto issue_copy = [&](int k) {
        const long long idx = (long long)blockIdx.x + (long long)k * gridDim.x;
        if (idx >= total) return;
        const PrepTile w = prep_tile_at(p, (int)idx, false);
        const uint32_t bar = bar_raw0 + 8u * (k & 1);
        if (w.rows_here <= 0) {
            mbar_arrive(bar);
            return;
        }
        const int y = src_table ? src_table[(size_t)w.head * (p.cap / kTile) + w.tile] * kTile : w.head * p.cap + w.tile * kTile;
        mbar_expect_tx(bar, kFusedRaw);
        tma_load_2d(sbase + kFusedOffRaw + (k & 1) * kFusedRaw, &map_src, 0, y, bar);
    };

    if (t == 0) {
        abort_flag = 0;
        mbar_init(bar_raw0, 1);
        mbar_init(bar_raw0 + 8u, 1);
        mbar_init(bar_mma, 1);
        asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory");
        issue_copy(0);
    }
    if (warp == 0) {
        asm volatile("tcgen05.alloc.cta_group::1.sync.aligned.shared::cta.b32 [%0], %1;"
                     ::"r"(smem_u32(&tmem_holder)), "r"(kPrepTcTmemCols) : "memory");
        asm volatile("tcgen05.relinquish_alloc_permit.cta_group::1.sync.aligned;" ::: "memory");
    }
    for (int x = t; x < kPrepTcB / 16; x += kPrepTcThreads) reinterpret_cast<uint4 *>(bop)[x] = make_uint4(0u, 0u, 0u, 0u);
    tc_fence_before();
    __syncthreads();
    tc_fence_after();
    const uint32_t tmem = tmem_holder;
    uint32_t mma_parity = 0;

    int k = 0;
    for (int idx = (int)blockIdx.x; idx < total; idx += (int)gridDim.x, ++k) {
        const PrepTile w = prep_tile_at(p, idx, t == 0);
        const int head = w.head, tile = w.tile, n = w.n, rows_here = w.rows_here;
        const int buf = k & 1;
        uint8_t *tile_smem = smem + buf * kPrepTcTile;
        if (t == 0) {
            // the other stage was read, by every thread, before the last barrier; and the operand tile about to be
            // written was stored two entries ago: that store has to be through with shared memory
            issue_copy(k + 1);
            asm volatile("cp.async.bulk.wait_group.read 1;" ::: "memory");
        }
        const bool landed = mbar_wait(bar_raw0 + 8u * buf, (uint32_t)(k >> 1) & 1u, &abort_flag, sink);
        const bool ok = __syncthreads_and(landed);           // the block goes on as a whole, or not at all

        // ---- one thread per row: the stored row into the operand tile (bf16, 128 dimensions, the layout a TMA load
        // leaves), its norm on the way; rows that are not candidates become zeros
        const int rt = t;
        const int row = tile * kTile + rt;
        float r = 0.f, sq = 0.f;
        if (ok && rows_here > 0) {
            uint4 out[16];
#pragma unroll
            for (int c = 0; c < 16; ++c) out[c] = make_uint4(0u, 0u, 0u, 0u);
            if (rt < rows_here) {
                const uint8_t *raw = smem + kFusedOffRaw + buf * kFusedRaw + rt * 128;
                uint4 in[8];
#pragma unroll
                for (int c = 0; c < 8; ++c) in[c] = *reinterpret_cast<const uint4 *>(raw + ((c ^ (rt & 7)) << 4));
                float2 sq2[4];
#pragma unroll
                for (int e = 0; e < 4; ++e) sq2[e] = make_float2(0.f, 0.f);
#pragma unroll
                for (int c = 0; c < 8; ++c) {
                    if (kCodes) widen16(in[c], &out[2 * c], &out[2 * c + 1]);     // 16 codes -> bf16 chunks 2 c, 2 c + 1
                    else out[c] = in[c];                                           // 64 dimensions: chunks 0..7, the rest zeros
                }
#pragma unroll
                for (int c = 0; c < (kCodes ? 16 : 8); ++c) {
                    float f[8];
                    Elem<__nv_bfloat16>::unpack(out[c], f);
#pragma unroll
                    for (int e = 0; e < 4; ++e) {
                        const float2 f2 = make_float2(f[2 * e], f[2 * e + 1]);
                        sq2[e] = __ffma2_rn(f2, f2, sq2[e]);
                    }
                }
                sq = ((sq2[0].x + sq2[0].y) + (sq2[1].x + sq2[1].y)) + ((sq2[2].x + sq2[2].y) + (sq2[3].x + sq2[3].y));
                const float nrm = sq > 0.f ? sq * rsqrtf(sq) : 0.f;
                r = __fdividef(1.0f, nrm + p.eps);
            }
#pragma unroll
            for (int c = 0; c < 16; ++c)
                *reinterpret_cast<uint4 *>(tile_smem + (c >> 3) * (kPrepTcTile / 2) + rt * 128 + (((c & 7) ^ (rt & 7)) << 4)) = out[c];
        }
        if (ok) {
            float rest = r;
            uint32_t rp[3];
#pragma unroll
            for (int c = 0; c < 3; ++c) {
                const __nv_bfloat16 h16 = __float2bfloat16_rn(rest);
                rp[c] = (uint32_t)__bfloat16_as_ushort(h16);
                rest -= __bfloat162float(h16);
            }
            const int s = rt >> 4, kk = rt & 15;
#pragma unroll
            for (int nn = 0; nn < 3; ++nn)
                *reinterpret_cast<unsigned short *>(bop + s * 512 + nn * 32 + ((kk >> 3) << 4) + (kk & 7) * 2) = (unsigned short)rp[nn];
        }
        asm volatile("fence.proxy.async.shared::cta;" ::: "memory");       // generic writes -> tensor-core and TMA reads
        __syncthreads();

        if (ok && rows_here > 0 && t == 0) {
            const uint32_t idesc = (1u << 4) | (1u << 7) | (1u << 10) | (1u << 15) | ((16u >> 3) << 17) | ((128u >> 4) << 24);
            tc_fence_after();
#pragma unroll
            for (int ks = 0; ks < 8; ++ks) {
                const uint32_t a_addr = sbase + buf * kPrepTcTile + ks * 2048;
                const uint32_t b_addr = sbase + kFusedOffB + ks * 512;
                uint64_t da = (uint64_t)((a_addr & 0x3FFFFu) >> 4) | ((uint64_t)(16384u >> 4) << 16) | ((uint64_t)(1024u >> 4) << 32) |
                              ((uint64_t)1 << 46) | ((uint64_t)2 << 61);
                uint64_t db = (uint64_t)((b_addr & 0x3FFFFu) >> 4) | ((uint64_t)1 << 16) | ((uint64_t)(256u >> 4) << 32) |
                              ((uint64_t)1 << 46) | ((uint64_t)6 << 61);
                asm volatile("{\n\t.reg .pred pp;\n\tsetp.ne.b32 pp, %4, 0;\n\ttcgen05.mma.cta_group::1.kind::f16 [%0], %1, %2, %3, pp;\n\t}"
                             ::"r"(tmem), "l"(da), "l"(db), "r"(idesc), "r"(ks) : "memory");
            }
            umma_commit(bar_mma);
            // the tile, as the head's rows [128 tile, 128 tile + 128) of the scoring copy (contiguous, head after head)
            const int yw = head * p.cap + tile * kTile;
            asm volatile("cp.async.bulk.tensor.2d.global.shared::cta.bulk_group [%0, {%1, %2}], [%3];"
                         ::"l"(reinterpret_cast<uint64_t>(&map_wide)), "r"(0), "r"(yw), "r"(sbase + buf * kPrepTcTile) : "memory");
            asm volatile("cp.async.bulk.tensor.2d.global.shared::cta.bulk_group [%0, {%1, %2}], [%3];"
                         ::"l"(reinterpret_cast<uint64_t>(&map_wide)), "r"(64), "r"(yw), "r"(sbase + buf * kPrepTcTile + kPrepTcTile / 2) : "memory");
        }
        if (t == 0) asm volatile("cp.async.bulk.commit_group;" ::: "memory");      // one group per entry, empty or not

        if (ok) {
            p.inv_norm[(size_t)head * p.cap_pad + row] = r;
            p.self_dot[(size_t)head * p.cap_pad + row] = (r * r) * sq;     // Kbar_i . Kbar_i
            if (p.tri) {
                float rest = r > 0.f ? __fdiv_rn(1.0f, r) : 0.f;
                uint32_t part[3];
#pragma unroll
                for (int c = 0; c < 3; ++c) {
                    const __nv_bfloat16 h16 = __float2bfloat16_rn(rest);
                    part[c] = (uint32_t)__bfloat16_as_ushort(h16);
                    rest -= __bfloat162float(h16);
                }
                uint4 *dst = reinterpret_cast<uint4 *>(p.norm_split + ((size_t)head * p.cap_pad + row) * 16);
                dst[0] = make_uint4(part[0] | (part[1] << 16), part[2] | (part[0] << 16), part[1] | (part[0] << 16), 0u);
                dst[1] = make_uint4(0u, 0u, 0u, 0u);
                if (tile == (n + kTile - 1) / kTile - 1) {
                    rest = r > 0.f ? -__fdiv_rn(p.sim_threshold, r) : 0.f;
#pragma unroll
                    for (int c = 0; c < 3; ++c) {
                        const __nv_bfloat16 h16 = __float2bfloat16_rn(rest);
                        part[c] = (uint32_t)__bfloat16_as_ushort(h16);
                        rest -= __bfloat162float(h16);
                    }
                    uint4 *thr = reinterpret_cast<uint4 *>(p.thr_split + ((size_t)head * kTile + rt) * 16);
                    thr[0] = make_uint4(part[0] | (part[0] << 16), part[0] | (part[1] << 16), part[1] | (part[2] << 16), 0u);
                    thr[1] = make_uint4(0u, 0u, 0u, 0u);
                }
            }
        }

        float tsum = 0.f;
        bool done = ok;
        if (ok && rows_here > 0) {
            done = mbar_wait(bar_mma, mma_parity, &abort_flag, sink);
            mma_parity ^= 1u;
            if (done) {
                tc_fence_after();
                uint32_t acc[8];
                tmem_ld8(tmem + ((uint32_t)(warp * 32) << 16), acc);      // lane = column c of the keys
                tmem_wait8(acc);
                tsum = (__uint_as_float(acc[0]) + __uint_as_float(acc[1])) + __uint_as_float(acc[2]);
            }
        }
        tc_fence_before();
        done = __syncthreads_and(done);
        p.tile_sum[((size_t)head * p.tiles + tile) * D + t] = done ? tsum : 0.f;
        if (!done) break;
    }

    if (t == 0) asm volatile("cp.async.bulk.wait_group 0;" ::: "memory");      // the stores are through before the block leaves
    tc_fence_before();
    __syncthreads();
    if (warp == 0) {
        if (abort_flag) __nanosleep(200000);       // error path only: let the copies in flight land
        tc_fence_after();
        asm volatile("tcgen05.dealloc.cta_group::1.sync.aligned.b32 %0, %1;" ::"r"(tmem), "r"(kPrepTcTmemCols) : "memory");
    }
}

// The tile sums of a head added up in tile order (a launch of its own behind prep_tc_kernel: no tickets, no fences in
// the streaming kernel), also as three bf16 rows whose sum is s to fp32 accuracy (rows 3..15 of the 16-row block are
// zero): appended to the query rows, they let the tensor cores form Kbar_i . s along with the logits.
__global__ void __launch_bounds__(kHeadDim) head_sum_kernel(Params p)
{
    constexpr int D = kHeadDim;
    const int head = blockIdx.x, t = threadIdx.x;
    const float *ts = p.tile_sum + (size_t)head * p.tiles * D + t;
    float s = 0.f;
    for (int q = 0; q < p.tiles; ++q) s += ts[(size_t)q * D];
    p.head_sum[(size_t)head * D + t] = s;
    __nv_bfloat16 *hs = p.head_sum_bf16 + (size_t)head * 16 * D + t;
    float rest = s;
#pragma unroll
    for (int part_i = 0; part_i < 3; ++part_i) {
        const __nv_bfloat16 h16 = __float2bfloat16_rn(rest);
        hs[part_i * D] = h16;
        rest -= __bfloat162float(h16);
    }
    for (int z = 3; z < 16; ++z) hs[z * D] = __float2bfloat16_rn(0.f);
}

}  // namespace

template <typename T, int D>
static cudaError_t launch_prep_for(const Params &p, cudaStream_t s)
{
    const unsigned grid = (unsigned)p.tiles * (unsigned)(p.batch * p.hkv);
    const int smem = kTile * D * (int)sizeof(T) + 16;
    cudaError_t e = cudaFuncSetAttribute(prep_kernel<T, D>, cudaFuncAttributeMaxDynamicSharedMemorySize, smem);
    if (e != cudaSuccess) return e;
    prep_kernel<T, D><<<grid, kPrepThreads, smem, s>>>(p);
    return cudaGetLastError();
}

cudaError_t launch_prep(const Params &p, cudaStream_t s)
{
    const bool bf16 = p.dtype == RKV_BF16;
    if (p.fuse_mode != 0) {                 // the tensor-core form that also writes the scoring copy
        const uint64_t wide_rows = (uint64_t)p.batch * p.hkv * p.cap + kTile;
        const uint64_t src_rows = p.fuse_table ? (uint64_t)p.pool_pages * kTile : (uint64_t)p.batch * p.hkv * p.cap;
        CUtensorMap map_src, map_wide;
        if (!sm100::make_map_row128(&map_src, p.fuse_src, src_rows, p.fuse_mode == 1) ||
            !sm100::make_map(&map_wide, p.k_cache, wide_rows, kTile))
            return cudaErrorInvalidValue;
        int dev = 0, sms = 0;
        cudaError_t e;
        if ((e = cudaGetDevice(&dev)) != cudaSuccess) return e;
        if ((e = cudaDeviceGetAttribute(&sms, cudaDevAttrMultiProcessorCount, dev)) != cudaSuccess) return e;
        const int total = p.tiles * p.batch * p.hkv;
        const unsigned grid = (unsigned)std::min(total, kFusedBlocks * sms);
        if (p.fuse_mode == 1) {
            if ((e = cudaFuncSetAttribute(prep_fused_kernel<true>, cudaFuncAttributeMaxDynamicSharedMemorySize, kFusedSmem)) != cudaSuccess) return e;
            prep_fused_kernel<true><<<grid, kPrepTcThreads, kFusedSmem, s>>>(p, map_src, map_wide, p.fuse_table, total);
        } else {
            if ((e = cudaFuncSetAttribute(prep_fused_kernel<false>, cudaFuncAttributeMaxDynamicSharedMemorySize, kFusedSmem)) != cudaSuccess) return e;
            prep_fused_kernel<false><<<grid, kPrepTcThreads, kFusedSmem, s>>>(p, map_src, map_wide, p.fuse_table, total);
        }
        if ((e = cudaGetLastError()) != cudaSuccess) return e;
        head_sum_kernel<<<(unsigned)(p.batch * p.hkv), kHeadDim, 0, s>>>(p);
        return cudaGetLastError();
    }
    if (bf16 && p.d == kHeadDim) {          // the tensor-core form
        CUtensorMap map_k;
        if (!sm100::make_map(&map_k, p.k_cache, sm100::key_rows_total(p), kTile)) return cudaErrorInvalidValue;
        cudaError_t e = cudaFuncSetAttribute(prep_tc_kernel, cudaFuncAttributeMaxDynamicSharedMemorySize, kPrepTcSmem);
        if (e != cudaSuccess) return e;
        int dev = 0, sms = 0;
        if ((e = cudaGetDevice(&dev)) != cudaSuccess) return e;
        if ((e = cudaDeviceGetAttribute(&sms, cudaDevAttrMultiProcessorCount, dev)) != cudaSuccess) return e;
        const int total = p.tiles * p.batch * p.hkv;
        prep_tc_kernel<<<(unsigned)std::min(total, kPrepTcBlocks * sms), kPrepTcThreads, kPrepTcSmem, s>>>(p, map_k, total);
        if ((e = cudaGetLastError()) != cudaSuccess) return e;
        head_sum_kernel<<<(unsigned)(p.batch * p.hkv), kHeadDim, 0, s>>>(p);
        return cudaGetLastError();
    }
    switch (p.d) {
        case 64: return bf16 ? launch_prep_for<__nv_bfloat16, 64>(p, s) : launch_prep_for<float, 64>(p, s);
        case 128: return bf16 ? launch_prep_for<__nv_bfloat16, 128>(p, s) : launch_prep_for<float, 128>(p, s);
        case 256: return bf16 ? launch_prep_for<__nv_bfloat16, 256>(p, s) : launch_prep_for<float, 256>(p, s);
        default: return cudaErrorInvalidValue;
    }
}

}  // namespace rkv

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
    switch (p.d) {
        case 64: return bf16 ? launch_prep_for<__nv_bfloat16, 64>(p, s) : launch_prep_for<float, 64>(p, s);
        case 128: return bf16 ? launch_prep_for<__nv_bfloat16, 128>(p, s) : launch_prep_for<float, 128>(p, s);
        case 256: return bf16 ? launch_prep_for<__nv_bfloat16, 256>(p, s) : launch_prep_for<float, 256>(p, s);
        default: return cudaErrorInvalidValue;
    }
}

}  // namespace rkv

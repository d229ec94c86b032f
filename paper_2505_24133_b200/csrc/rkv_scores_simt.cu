// Stage "scores", CUDA-core version: plain fp32 arithmetic, one thread per row.
//
// Used for fp32 caches (small shapes) and, behind RKV_FLAG_SIMT_SCORES, as an independent on-GPU
// cross-check of the tensor-core kernel for bf16 caches.  It forms Eq. 5's matrix row by row in
// registers and accumulates Eq. 6's sums directly (no closed form), so the two kernels reach the
// same numbers along different routes.
//
// Block x of a head, x < tiles: rows [128 x, 128 x + 128) of the similarity matrix: for each row i the
// column sum over j of S[j][i] (S is symmetric before the retention rule, which for token i touches
// line i only), minus the entries of the up-to-beta largest j with S[j][i] > T.
// Block x == tiles: Eq. 2-3 pooled logits of the head's query group against every candidate key.
#include "rkv_common.cuh"

namespace rkv {

namespace {

constexpr int kSimtThreads = 128;

// kRows rows of D elements, starting at `src` (row first_row of its head), into shared memory as fp32, rows padded to
// D + 1 floats (thread-per-row reads then hit distinct banks); rows >= valid_rows are zero-filled.
template <typename T, int D, int kRows>
__device__ void load_tile_rows(const T *src, int first_row, int valid_rows, float *dst /*[kRows][D + 1]*/)
{
    constexpr int kPadRow = D + 1;
    constexpr int kHeadDim = D;
    constexpr int kPerVec = Elem<T>::kPerVec;
    constexpr int kVecPerRow = kHeadDim / kPerVec;
    for (int v = threadIdx.x; v < kRows * kVecPerRow; v += kSimtThreads) {
        const int r = v / kVecPerRow, c = (v % kVecPerRow) * kPerVec;
        float f[kPerVec];
        if (first_row + r < valid_rows) {
            uint4 raw = __ldg(reinterpret_cast<const uint4 *>(src + (size_t)r * kHeadDim + c));
            Elem<T>::unpack(raw, f);
        } else {
#pragma unroll
            for (int e = 0; e < kPerVec; ++e) f[e] = 0.f;
        }
#pragma unroll
        for (int e = 0; e < kPerVec; ++e) dst[r * kPadRow + c + e] = f[e];
    }
}

// D: head dimension (64, 128, 256).  The streamed keys come in sub-tiles of kRowsB rows (64 at D = 256, where two
// whole tiles would not fit shared memory).
template <typename T, int D>
__global__ void __launch_bounds__(kSimtThreads) scores_simt_kernel(Params p)
{
    constexpr int kHeadDim = D;
    constexpr int kPadRow = D + 1;
    constexpr int kRowsB = D <= 128 ? kTile : kTile / 2;
    extern __shared__ float smem[];
    float *tileA = smem;                       // [128][kPadRow]
    float *tileB = smem + kTile * kPadRow;     // [kRowsB][kPadRow]
    __shared__ float rB[kTile];

    const int blocks_per_head = p.tiles + 1;
    const int head = blockIdx.x / blocks_per_head;
    const int x = blockIdx.x % blocks_per_head;
    const int b = head / p.hkv, h = head % p.hkv;
    const int n = seq_candidates(p, b);
    if (n == 0) return;
    const int n_tiles = (n + kTile - 1) / kTile;
    // first of the (at most 128, page-aligned) rows of the head starting at `first_row`
    auto key_rows = [&](int first_row) {
        return static_cast<const T *>(p.k_cache) + (size_t)row_index(p, head, first_row) * kHeadDim;
    };
    const float *inv_norm = p.inv_norm + (size_t)head * p.cap_pad;
    const int t = threadIdx.x;

    if (x < p.tiles) {
        // ---------------- Eq. 5-6 + retention rule for rows [128 x, 128 x + 128)
        if (x >= n_tiles) return;
        const int i = x * kTile + t;
        load_tile_rows<T, D, kTile>(key_rows(x * kTile), x * kTile, n, tileA);
        const float ri = (i < n) ? inv_norm[i] : 0.f;
        float total = 0.f, removed = 0.f;
        int left = p.beta;
        for (int jt = (n_tiles * kTile) / kRowsB - 1; jt >= 0; --jt) {          // descending j: "largest positions first"
            __syncthreads();
            load_tile_rows<T, D, kRowsB>(key_rows(jt * kRowsB), jt * kRowsB, n, tileB);
            if (t < kRowsB) rB[t] = (jt * kRowsB + t < n) ? inv_norm[jt * kRowsB + t] : 0.f;
            __syncthreads();
            if (i < n) {
                for (int jj = kRowsB - 1; jj >= 0; --jj) {
                    const int j = jt * kRowsB + jj;
                    if (j >= n || j == i) continue;           // zero diagonal (Eq. 5)
                    float dot = 0.f;
#pragma unroll 16
                    for (int c = 0; c < kHeadDim; ++c) dot = fmaf(tileA[t * kPadRow + c], tileB[jj * kPadRow + c], dot);
                    const float s = (dot * rB[jj]) * ri;
                    total += s;
                    if (left > 0 && s > p.sim_threshold) {
                        removed += s;
                        --left;
                    }
                }
            }
        }
        if (i < n) p.sbar[(size_t)head * p.cap_pad + i] = (total - removed) / (float)n;
    } else {
        // ---------------- Eq. 2-3: max over the group of scaled logits, per (query row, key)
        const int rows = p.group * p.alpha;
        const T *Q = static_cast<const T *>(p.q_window) + ((size_t)b * p.hq + (size_t)h * p.group) * p.alpha * kHeadDim;
        load_tile_rows<T, D, kTile>(Q, 0, rows, tileA);       // query rows g * alpha + j
        const float scale = p.logit_scale;
        float *logits = p.logits + (size_t)head * p.alpha * p.cap_pad;
        for (int jt = 0; jt < (n_tiles * kTile) / kRowsB; ++jt) {
            __syncthreads();
            load_tile_rows<T, D, kRowsB>(key_rows(jt * kRowsB), jt * kRowsB, n, tileB);
            __syncthreads();
            const int i = jt * kRowsB + t;
            if (t < kRowsB && i < n) {
                for (int j = 0; j < p.alpha; ++j) {
                    float best = -INFINITY, total = 0.f;
                    for (int g = 0; g < p.group; ++g) {
                        const float *q = tileA + (g * p.alpha + j) * kPadRow;
                        float dot = 0.f;
#pragma unroll 16
                        for (int c = 0; c < kHeadDim; ++c) dot = fmaf(q[c], tileB[t * kPadRow + c], dot);
                        best = fmaxf(best, dot * scale);
                        total += dot * scale;
                    }
                    logits[(size_t)j * p.cap_pad + i] = p.gqa_mean_pool ? total / (float)p.group : best;
                }
            }
        }
    }
}

template <typename T, int D>
cudaError_t launch_simt_for(const Params &p, cudaStream_t s)
{
    const unsigned grid = (unsigned)(p.tiles + 1) * (unsigned)(p.batch * p.hkv);
    const size_t smem = (size_t)(kTile + (D <= 128 ? kTile : kTile / 2)) * (D + 1) * sizeof(float);
    cudaError_t e = cudaFuncSetAttribute(scores_simt_kernel<T, D>, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)smem);
    if (e != cudaSuccess) return e;
    scores_simt_kernel<T, D><<<grid, kSimtThreads, smem, s>>>(p);
    return cudaGetLastError();
}

}  // namespace

cudaError_t launch_scores_simt(const Params &p, cudaStream_t s)
{
    const bool bf16 = p.dtype == RKV_BF16;
    switch (p.d) {
        case 64: return bf16 ? launch_simt_for<__nv_bfloat16, 64>(p, s) : launch_simt_for<float, 64>(p, s);
        case 128: return bf16 ? launch_simt_for<__nv_bfloat16, 128>(p, s) : launch_simt_for<float, 128>(p, s);
        case 256: return bf16 ? launch_simt_for<__nv_bfloat16, 256>(p, s) : launch_simt_for<float, 256>(p, s);
        default: return cudaErrorInvalidValue;
    }
}

}  // namespace rkv

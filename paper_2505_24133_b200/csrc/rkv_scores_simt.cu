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
constexpr int kPadRow = kHeadDim + 1;   // padded smem row: thread-per-row reads hit distinct banks

template <typename T>
__device__ void load_tile_rows(const T *src, int first_row, int valid_rows, float *dst /*[128][kPadRow]*/)
{
    // rows >= valid_rows are zero-filled
    constexpr int kPerVec = Elem<T>::kPerVec;
    constexpr int kVecPerRow = kHeadDim / kPerVec;
    for (int v = threadIdx.x; v < kTile * kVecPerRow; v += kSimtThreads) {
        const int r = v / kVecPerRow, c = (v % kVecPerRow) * kPerVec;
        float f[kPerVec];
        if (first_row + r < valid_rows) {
            uint4 raw = __ldg(reinterpret_cast<const uint4 *>(src + (size_t)(first_row + r) * kHeadDim + c));
            Elem<T>::unpack(raw, f);
        } else {
#pragma unroll
            for (int e = 0; e < kPerVec; ++e) f[e] = 0.f;
        }
#pragma unroll
        for (int e = 0; e < kPerVec; ++e) dst[r * kPadRow + c + e] = f[e];
    }
}

template <typename T>
__global__ void __launch_bounds__(kSimtThreads) scores_simt_kernel(Params p)
{
    extern __shared__ float smem[];
    float *tileA = smem;                       // [128][kPadRow]
    float *tileB = smem + kTile * kPadRow;     // [128][kPadRow]
    __shared__ float rB[kTile];

    const int blocks_per_head = p.tiles + 1;
    const int head = blockIdx.x / blocks_per_head;
    const int x = blockIdx.x % blocks_per_head;
    const int b = head / p.hkv, h = head % p.hkv;
    const int n = seq_candidates(p, b);
    if (n == 0) return;
    const int n_tiles = (n + kTile - 1) / kTile;
    const T *K = static_cast<const T *>(p.k_cache) + (size_t)head * p.cap * kHeadDim;
    const float *inv_norm = p.inv_norm + (size_t)head * p.cap_pad;
    const int t = threadIdx.x;

    if (x < p.tiles) {
        // ---------------- Eq. 5-6 + retention rule for rows [128 x, 128 x + 128)
        if (x >= n_tiles) return;
        const int i = x * kTile + t;
        load_tile_rows<T>(K, x * kTile, n, tileA);
        const float ri = (i < n) ? inv_norm[i] : 0.f;
        float total = 0.f, removed = 0.f;
        int left = p.beta;
        for (int jt = n_tiles - 1; jt >= 0; --jt) {          // descending j: "largest positions first"
            __syncthreads();
            load_tile_rows<T>(K, jt * kTile, n, tileB);
            rB[t] = (jt * kTile + t < n) ? inv_norm[jt * kTile + t] : 0.f;
            __syncthreads();
            if (i < n) {
                for (int jj = kTile - 1; jj >= 0; --jj) {
                    const int j = jt * kTile + jj;
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
        load_tile_rows<T>(Q, 0, rows, tileA);                 // query rows g * alpha + j
        const float scale = rsqrtf((float)kHeadDim);
        float *logits = p.logits + (size_t)head * p.alpha * p.cap_pad;
        for (int jt = 0; jt < n_tiles; ++jt) {
            __syncthreads();
            load_tile_rows<T>(K, jt * kTile, n, tileB);
            __syncthreads();
            const int i = jt * kTile + t;
            if (i < n) {
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

constexpr size_t kSimtSmem = 2ull * kTile * kPadRow * sizeof(float);

}  // namespace

cudaError_t launch_scores_simt(const Params &p, cudaStream_t s)
{
    const unsigned grid = (unsigned)(p.tiles + 1) * (unsigned)(p.batch * p.hkv);
    cudaError_t e;
    if (p.dtype == RKV_BF16) {
        e = cudaFuncSetAttribute(scores_simt_kernel<__nv_bfloat16>, cudaFuncAttributeMaxDynamicSharedMemorySize,
                                 (int)kSimtSmem);
        if (e != cudaSuccess) return e;
        scores_simt_kernel<__nv_bfloat16><<<grid, kSimtThreads, kSimtSmem, s>>>(p);
    } else {
        e = cudaFuncSetAttribute(scores_simt_kernel<float>, cudaFuncAttributeMaxDynamicSharedMemorySize,
                                 (int)kSimtSmem);
        if (e != cudaSuccess) return e;
        scores_simt_kernel<float><<<grid, kSimtThreads, kSimtSmem, s>>>(p);
    }
    return cudaGetLastError();
}

}  // namespace rkv

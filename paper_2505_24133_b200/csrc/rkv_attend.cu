// Decode-step attention over the compressed cache (Section 3.1: between two firings of the compression the model
// decodes against the B_budget retained tokens plus the buffer; Eq. 1 with a single query row per head):
//
//   out[b][q] = sum_j softmax_j( q_new[b][q] . K[b][q / G][j] / sqrt(d) ) V[b][q / G][j],   j < seq_lens[b]
//
// HBM-bound: every cached K and V row is read once, 2 * 2 * G * d flop per 2 * d * sizeof(T) bytes (5 flop per byte
// for G = 5 at bf16), so the arithmetic stays on the CUDA cores in fp32 and the work goes into the data path: one
// block per (KV head, split of the rows), 64-row tiles of K and of V brought into shared memory by bulk copies
// (cp.async.bulk, three stages in flight, bounded waits), all G query heads of the group served from the same tile.
//   scores   8 lanes per row, 16 dims each (two or four 16-byte shared-memory loads), the G partial dot products of a
//            row folded over the 8 lanes by 3 shuffle steps; four rows per warp instruction
//   softmax  online, per tile: block-wide tile maximum per query head, running maximum and sum, base-2 exponentials
//   values   lanes over d: a lane owns 4 dims of the output of every query head, a warp walks its 8 rows of the tile
// With few head-problems the rows of a head are cut into splits (more blocks than SMs); a second small kernel merges
// the splits' partial results.
#include "rkv_sm100.cuh"

namespace rkv {

namespace {

using namespace sm100;

constexpr int kAttThreads = 256;
constexpr int kAttWarps = kAttThreads / 32;
constexpr int kAttRows = 64;            // rows per tile
constexpr int kAttStages = 3;
constexpr int kAttMaxG = 8;             // query heads per KV head served by one block

struct AttendParams {
    const void *k_cache, *v_cache, *q_new;
    const int32_t *seq_lens;
    float *out;                 // [batch][hq][d]
    float *partial;             // [P][splits][G][d + 2]: unnormalised output, running maximum (base-2 domain), sum
    int batch, hkv, hq, cap, splits;
    int32_t *status;
    long long wait_cycles;
};

template <typename T, int G>
__global__ void __launch_bounds__(kAttThreads, (G <= 4 && sizeof(T) == 2) ? 2 : 1) attend_kernel(AttendParams p)
{
    constexpr int kRowBytes = kHeadDim * (int)sizeof(T);
    constexpr int kTileBytesT = kAttRows * kRowBytes;
    constexpr int kPerVec = Elem<T>::kPerVec;               // elements per 16-byte vector
    constexpr int kVecPerRow = kHeadDim / kPerVec;          // 16 (bf16) or 32 (fp32)
    constexpr int kVecPerLane = kVecPerRow / 8;             // vectors of a row held by one of its 8 lanes
    extern __shared__ __align__(128) uint8_t att_smem[];    // kAttStages x (K tile, V tile), then the small arrays
    float *sc = reinterpret_cast<float *>(att_smem + kAttStages * 2 * kTileBytesT);      // [G][kAttRows] scores, then weights
    float *red = sc + G * kAttRows;                          // [kAttWarps][G] per-warp maxima / sums
    float *stat = red + kAttWarps * G;                       // [G][3]: running maximum, running sum, rescale factor
    unsigned long long *bars = reinterpret_cast<unsigned long long *>(stat + 3 * G + ((3 * G) & 1));
    __shared__ int abort_flag;

    const int head = blockIdx.x / p.splits, split = blockIdx.x % p.splits;
    const int b = head / p.hkv, h = head % p.hkv;
    const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
    const int L = p.seq_lens[b];
    const bool bad_len = L < 0 || L > p.cap;
    if (bad_len && threadIdx.x == 0 && split == 0 && h == 0) report(p.status, RKV_ERR_INVALID_ARG);
    const int Lc = bad_len ? 0 : L;
    // this block's rows: whole tiles, split evenly
    const int tiles_all = (Lc + kAttRows - 1) / kAttRows;
    const int t_begin = (int)((long long)split * tiles_all / p.splits), t_end = (int)((long long)(split + 1) * tiles_all / p.splits);
    const int n_tiles = t_end - t_begin;

    const T *K = static_cast<const T *>(p.k_cache) + (size_t)head * p.cap * kHeadDim;
    const T *V = static_cast<const T *>(p.v_cache) + (size_t)head * p.cap * kHeadDim;
    const ErrSink sink{p.status, nullptr, p.wait_cycles};

    if (threadIdx.x == 0) {
        abort_flag = 0;
        for (int s = 0; s < kAttStages; ++s) mbar_init(smem_u32(bars + s), 1);
        asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory");
    }
    if (threadIdx.x < G) {
        stat[threadIdx.x * 3] = -INFINITY;
        stat[threadIdx.x * 3 + 1] = 0.f;
    }
    __syncthreads();

    auto issue = [&](int t) {           // tile t of this block into stage t % kAttStages (one thread)
        const int s = t % kAttStages;
        const int row0 = (t_begin + t) * kAttRows;
        const uint32_t bytes = (uint32_t)min(kAttRows, Lc - row0) * kRowBytes;
        const uint32_t bar = smem_u32(bars + s);
        mbar_expect_tx(bar, 2 * bytes);
        asm volatile("cp.async.bulk.shared::cluster.global.mbarrier::complete_tx::bytes [%0], [%1], %2, [%3];"
                     ::"r"(smem_u32(att_smem + (size_t)s * 2 * kTileBytesT)), "l"(K + (size_t)row0 * kHeadDim), "r"(bytes), "r"(bar)
                     : "memory");
        asm volatile("cp.async.bulk.shared::cluster.global.mbarrier::complete_tx::bytes [%0], [%1], %2, [%3];"
                     ::"r"(smem_u32(att_smem + (size_t)s * 2 * kTileBytesT + kTileBytesT)), "l"(V + (size_t)row0 * kHeadDim), "r"(bytes),
                       "r"(bar)
                     : "memory");
    };
    if (threadIdx.x == 0)
        for (int t = 0; t < min(n_tiles, kAttStages); ++t) issue(t);

    // the group's queries, scaled by log2(e) / sqrt(d): lane j of a row's 8 lanes holds vectors j, j + 8, ...
    const int sub = lane >> 3, j8 = lane & 7;
    float qreg[G][kVecPerLane * kPerVec];
    {
        const float qscale = 1.4426950408889634f * rsqrtf((float)kHeadDim);
        const T *Q = static_cast<const T *>(p.q_new) + ((size_t)b * p.hq + (size_t)h * G) * kHeadDim;
#pragma unroll
        for (int g = 0; g < G; ++g)
#pragma unroll
            for (int u = 0; u < kVecPerLane; ++u) {
                const uint4 vec = *reinterpret_cast<const uint4 *>(Q + (size_t)g * kHeadDim + (j8 + 8 * u) * kPerVec);
                Elem<T>::unpack(vec, &qreg[g][u * kPerVec]);
#pragma unroll
                for (int e = 0; e < kPerVec; ++e) qreg[g][u * kPerVec + e] *= qscale;
            }
    }
    float acc[G][4];                     // lane owns dims 4 lane .. 4 lane + 3 of every head's output (this warp's rows)
#pragma unroll
    for (int g = 0; g < G; ++g)
#pragma unroll
        for (int e = 0; e < 4; ++e) acc[g][e] = 0.f;

    for (int t = 0; t < n_tiles; ++t) {
        const int s = t % kAttStages;
        const int row0 = (t_begin + t) * kAttRows;
        const int rows_here = min(kAttRows, Lc - row0);
        const bool landed = mbar_wait(smem_u32(bars + s), (t / kAttStages) & 1, &abort_flag, sink);
        if (!__syncthreads_and(landed)) {            // the block leaves as a whole, or not at all
            __nanosleep(200000);                     // error path only: let copies in flight land
            return;
        }
        const uint8_t *kt = att_smem + (size_t)s * 2 * kTileBytesT, *vt = kt + kTileBytesT;

        // ---- scores of the tile: warp w takes rows 8 w .. 8 w + 7, four at a time
        float wmax[G];
#pragma unroll
        for (int g = 0; g < G; ++g) wmax[g] = -INFINITY;
#pragma unroll
        for (int it = 0; it < 2; ++it) {
            const int r = warp * 8 + it * 4 + sub;
            float dot[G];
#pragma unroll
            for (int g = 0; g < G; ++g) dot[g] = 0.f;
            if (r < rows_here) {
#pragma unroll
                for (int u = 0; u < kVecPerLane; ++u) {
                    float kf[kPerVec];
                    Elem<T>::unpack(*reinterpret_cast<const uint4 *>(kt + (size_t)r * kRowBytes + (j8 + 8 * u) * 16), kf);
#pragma unroll
                    for (int g = 0; g < G; ++g)
#pragma unroll
                        for (int e = 0; e < kPerVec; ++e) dot[g] = fmaf(qreg[g][u * kPerVec + e], kf[e], dot[g]);
                }
            }
#pragma unroll
            for (int g = 0; g < G; ++g) {
#pragma unroll
                for (int off = 4; off > 0; off >>= 1) dot[g] += __shfl_xor_sync(0xffffffffu, dot[g], off);
                const float sv = r < rows_here ? dot[g] : -INFINITY;      // rows beyond the cached length take no part
                if (j8 == 0) sc[g * kAttRows + r] = sv;
                wmax[g] = fmaxf(wmax[g], sv);
            }
        }
#pragma unroll
        for (int g = 0; g < G; ++g) {
            float m = wmax[g];
#pragma unroll
            for (int off = 16; off > 0; off >>= 1) m = fmaxf(m, __shfl_xor_sync(0xffffffffu, m, off));
            if (lane == 0) red[warp * G + g] = m;
        }
        __syncthreads();
        // ---- online softmax: new running maximum, rescale factor, the tile's weights and their sum
        if (threadIdx.x < G) {
            const int g = threadIdx.x;
            float m = stat[g * 3];
#pragma unroll
            for (int w = 0; w < kAttWarps; ++w) m = fmaxf(m, red[w * G + g]);
            stat[g * 3 + 2] = exp2f(stat[g * 3] - m);          // 0 on the first tile (old maximum -inf)
            stat[g * 3] = m;
        }
        __syncthreads();
        for (int x = threadIdx.x; x < G * kAttRows; x += kAttThreads) {
            const int g = x / kAttRows;
            sc[x] = exp2f(sc[x] - stat[g * 3]);                 // -inf rows give 0
        }
        __syncthreads();
        if (warp < G) {          // one warp per query head adds up the tile's weights, in a fixed order
            const int g = warp;
            float sum = sc[g * kAttRows + lane] + sc[g * kAttRows + 32 + lane];
#pragma unroll
            for (int off = 16; off > 0; off >>= 1) sum += __shfl_xor_sync(0xffffffffu, sum, off);
            if (lane == 0) stat[g * 3 + 1] = stat[g * 3 + 1] * stat[g * 3 + 2] + sum;
        }
        static_assert(G <= kAttWarps, "every query head of the group needs a warp of its own for the sum");

        // ---- values: this warp's 8 rows, lanes over d
#pragma unroll
        for (int g = 0; g < G; ++g) {
            const float a = stat[g * 3 + 2];
#pragma unroll
            for (int e = 0; e < 4; ++e) acc[g][e] *= a;
        }
        const int r_lo = warp * 8, r_hi = min(r_lo + 8, rows_here);
        for (int r = r_lo; r < r_hi; ++r) {
            float vf[4];
            if (sizeof(T) == 2) {
                const uint2 raw = *reinterpret_cast<const uint2 *>(vt + (size_t)r * kRowBytes + lane * 8);
                const __nv_bfloat162 *h2 = reinterpret_cast<const __nv_bfloat162 *>(&raw);
                const float2 x0 = __bfloat1622float2(h2[0]), x1 = __bfloat1622float2(h2[1]);
                vf[0] = x0.x, vf[1] = x0.y, vf[2] = x1.x, vf[3] = x1.y;
            } else {
                const float4 raw = *reinterpret_cast<const float4 *>(vt + (size_t)r * kRowBytes + lane * 16);
                vf[0] = raw.x, vf[1] = raw.y, vf[2] = raw.z, vf[3] = raw.w;
            }
#pragma unroll
            for (int g = 0; g < G; ++g) {
                const float w = sc[g * kAttRows + r];
#pragma unroll
                for (int e = 0; e < 4; ++e) acc[g][e] = fmaf(w, vf[e], acc[g][e]);
            }
        }
        __syncthreads();                 // the stage and the score array are free again
        if (threadIdx.x == 0 && t + kAttStages < n_tiles) issue(t + kAttStages);
    }

    // ---- fold the warps' partial outputs (fixed order), then write the result of this block
    float *fold = reinterpret_cast<float *>(att_smem);        // [kAttWarps][G][128], the tile stages are free now
    __syncthreads();
#pragma unroll
    for (int g = 0; g < G; ++g)
        *reinterpret_cast<float4 *>(fold + ((size_t)warp * G + g) * kHeadDim + lane * 4) =
            make_float4(acc[g][0], acc[g][1], acc[g][2], acc[g][3]);
    __syncthreads();
    for (int x = threadIdx.x; x < G * kHeadDim; x += kAttThreads) {
        const int g = x / kHeadDim, c = x % kHeadDim;
        float sum = 0.f;
#pragma unroll
        for (int w = 0; w < kAttWarps; ++w) sum += fold[((size_t)w * G + g) * kHeadDim + c];
        if (p.splits == 1) {
            const float l = stat[g * 3 + 1];
            p.out[((size_t)b * p.hq + (size_t)h * G + g) * kHeadDim + c] = l > 0.f ? sum / l : 0.f;
        } else {
            float *part = p.partial + (((size_t)head * p.splits + split) * G + g) * (kHeadDim + 2);
            part[c] = sum;
            if (c == 0) {
                part[kHeadDim] = stat[g * 3];
                part[kHeadDim + 1] = stat[g * 3 + 1];
            }
        }
    }
}

// Merge the splits of one (KV head, query head): out = sum_s 2^(m_s - m) acc_s / sum_s 2^(m_s - m) l_s.
__global__ void __launch_bounds__(kHeadDim) attend_merge_kernel(AttendParams p, int G)
{
    const int head = blockIdx.x / G, g = blockIdx.x % G;
    const int b = head / p.hkv, h = head % p.hkv;
    const int c = threadIdx.x;
    const float *part = p.partial + ((size_t)head * p.splits * G + g) * (kHeadDim + 2);
    const size_t stride = (size_t)G * (kHeadDim + 2);
    float m = -INFINITY;
    for (int s = 0; s < p.splits; ++s) m = fmaxf(m, part[s * stride + kHeadDim]);
    float num = 0.f, den = 0.f;
    for (int s = 0; s < p.splits; ++s) {                   // fixed order
        const float ms = part[s * stride + kHeadDim];
        const float w = ms == -INFINITY ? 0.f : exp2f(ms - m);     // a split without rows
        num = fmaf(w, part[s * stride + c], num);
        den = fmaf(w, part[s * stride + kHeadDim + 1], den);
    }
    p.out[((size_t)b * p.hq + (size_t)h * G + g) * kHeadDim + c] = den > 0.f ? num / den : 0.f;
}

template <typename T, int G>
cudaError_t launch_one(const AttendParams &p, cudaStream_t s)
{
    const int tile_bytes = kAttRows * kHeadDim * (int)sizeof(T);
    const int smem = kAttStages * 2 * tile_bytes + (G * kAttRows + kAttWarps * G + 3 * G + 1) * 4 + kAttStages * 8 + 16;
    cudaError_t e = cudaFuncSetAttribute(attend_kernel<T, G>, cudaFuncAttributeMaxDynamicSharedMemorySize, smem);
    if (e != cudaSuccess) return e;
    attend_kernel<T, G><<<(unsigned)(p.batch * p.hkv * p.splits), kAttThreads, smem, s>>>(p);
    return cudaGetLastError();
}

template <typename T>
cudaError_t launch_dtype(const AttendParams &p, int G, cudaStream_t s)
{
    switch (G) {
        case 1: return launch_one<T, 1>(p, s);
        case 2: return launch_one<T, 2>(p, s);
        case 3: return launch_one<T, 3>(p, s);
        case 4: return launch_one<T, 4>(p, s);
        case 5: return launch_one<T, 5>(p, s);
        case 6: return launch_one<T, 6>(p, s);
        case 7: return launch_one<T, 7>(p, s);
        case 8: return launch_one<T, 8>(p, s);
        default: return cudaErrorInvalidValue;
    }
}

}  // namespace

int attend_max_group() { return kAttMaxG; }

// Splits of a head's rows: enough blocks for two waves of resident blocks (2 per SM), never finer than a tile.
int attend_splits(int heads, int cap, int sms)
{
    const int tiles = (cap + kAttRows - 1) / kAttRows;
    int splits = (4 * sms + heads - 1) / heads;
    splits = splits < 1 ? 1 : splits;
    return splits > tiles ? tiles : splits;
}

size_t attend_partial_bytes(int heads, int splits, int G)
{
    return splits > 1 ? (size_t)heads * splits * G * (kHeadDim + 2) * sizeof(float) : 0;
}

cudaError_t launch_attend(const void *k_cache, const void *v_cache, const void *q_new, const int32_t *seq_lens, float *out,
                          float *partial, int batch, int hkv, int hq, int cap, int splits, int dtype, int32_t *status,
                          long long wait_cycles, cudaStream_t s)
{
    AttendParams p;
    p.k_cache = k_cache;
    p.v_cache = v_cache;
    p.q_new = q_new;
    p.seq_lens = seq_lens;
    p.out = out;
    p.partial = partial;
    p.batch = batch;
    p.hkv = hkv;
    p.hq = hq;
    p.cap = cap;
    p.splits = splits;
    p.status = status;
    p.wait_cycles = wait_cycles;
    const int G = hq / hkv;
    cudaError_t e = dtype == RKV_BF16 ? launch_dtype<__nv_bfloat16>(p, G, s) : launch_dtype<float>(p, G, s);
    if (e != cudaSuccess || splits == 1) return e;
    attend_merge_kernel<<<(unsigned)(batch * hkv * G), kHeadDim, 0, s>>>(p, G);
    return cudaGetLastError();
}

}  // namespace rkv

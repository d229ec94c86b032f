// Decode-step attention over the compressed cache, CUDA-core form (fp32 caches; bf16 caches take the tensor-core kernel
// of rkv_attend_tc.cu) (Section 3.1: between two firings of the compression the model decodes against the B_budget
// retained tokens plus the buffer; Eq. 1 with a single query row per head):
//
//   out[b][q] = sum_j softmax_j( q_new[b][q] . K[b][q / G][j] / sqrt(d) ) V[b][q / G][j],   j < seq_lens[b]
//
// HBM-bound: every cached K and V row is read once, 2 * 2 * G * d flop per 2 * d * sizeof(T) bytes (5 flop per byte
// for G = 5 at bf16), so the arithmetic stays on the CUDA cores in fp32 and the work goes into the data path: one
// block per (KV head, split of the rows), 56-row tiles of K and of V brought into shared memory by bulk copies
// (cp.async.bulk, three stages in flight, bounded waits), all G query heads of the group served from the same tile.
//   scores   8 lanes per row, 16 dims each (two or four 16-byte shared-memory loads), the G partial dot products of a
//            row folded over the 8 lanes by 3 shuffle steps; four rows per warp instruction
//   softmax  online and per WARP: each of the 7 compute warps keeps its own running maximum and sum over its 8 rows
//            of every tile (base-2 exponentials), so the tile loop has no block-wide barrier; the warps' results are
//            merged once, at the end
//   values   lanes over d: a lane owns 4 dims of the output of every query head, a warp walks its 8 rows of the tile
// An eighth warp is the producer of the bulk copies; stages are handed back through mbarriers.
// With few head-problems the rows of a head are cut into splits (more blocks than SMs); a second small kernel merges
// the splits' partial results.
#include "rkv_sm100.cuh"

namespace rkv {

namespace {

using namespace sm100;

constexpr int kAttWarps = 7;             // compute warps
constexpr int kAttThreads = (kAttWarps + 1) * 32;     // + the producer warp
constexpr int kAttRows = 56;            // rows per tile: 8 per compute warp
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
    const int32_t *block_table;  // paged caches: [P][cap / 128] page ids (a page = 128 rows), else null
    int d_out;                   // head dimension of the output rows (the partial results always have rows of 128 + 2)
};

template <typename T, int G>
__global__ void __launch_bounds__(kAttThreads, (G <= 4 && sizeof(T) == 2) ? 2 : 1) attend_kernel(AttendParams p)
{
    constexpr int kRowBytes = kHeadDim * (int)sizeof(T);
    constexpr int kTileBytesT = kAttRows * kRowBytes;
    constexpr int kPerVec = Elem<T>::kPerVec;               // elements per 16-byte vector
    constexpr int kVecPerRow = kHeadDim / kPerVec;          // 16 (bf16) or 32 (fp32)
    constexpr int kVecPerLane = kVecPerRow / 8;             // vectors of a row held by one of its 8 lanes
    constexpr int GP = (G + 3) / 4 * 4;                     // query heads padded to whole float4s
    constexpr int kRowsPerWarp = kAttRows / kAttWarps;      // 8
    static_assert(kRowsPerWarp == 8, "a warp takes its rows four at a time, twice");
    extern __shared__ __align__(128) uint8_t att_smem[];    // kAttStages x (K tile, V tile), then the small arrays
    float *wts = reinterpret_cast<float *>(att_smem + kAttStages * 2 * kTileBytesT);     // [kAttWarps][kRowsPerWarp][GP] weights
    float *wstat = wts + kAttWarps * kRowsPerWarp * GP;     // [kAttWarps][G][2] per-warp running maximum and sum
    unsigned long long *bars = reinterpret_cast<unsigned long long *>(wstat + kAttWarps * G * 2);   // full[stages], empty[stages]
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

    const T *K = static_cast<const T *>(p.k_cache), *V = static_cast<const T *>(p.v_cache);
    // first of the rows [r, r + count) of the head in the caches' row view; with paged caches the rows must not cross a
    // page boundary
    auto row_at = [&](int r) -> size_t {
        return p.block_table ? (size_t)p.block_table[(size_t)head * (p.cap / kTile) + r / kTile] * kTile + r % kTile
                             : (size_t)head * p.cap + r;
    };
    const ErrSink sink{p.status, nullptr, p.wait_cycles};

    if (threadIdx.x == 0) {
        abort_flag = 0;
        for (int s = 0; s < kAttStages; ++s) {
            mbar_init(smem_u32(bars + s), 1);                          // full: the producer's arrival + the copies' bytes
            mbar_init(smem_u32(bars + kAttStages + s), kAttWarps);     // empty: every compute warp is done with the stage
        }
        asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory");
    }
    __syncthreads();

    float2 acc[G][2];                    // compute warps: lane owns dims 4 lane .. 4 lane + 3 of every head's output
#pragma unroll
    for (int g = 0; g < G; ++g) acc[g][0] = acc[g][1] = make_float2(0.f, 0.f);

    if (warp == kAttWarps) {
        // ------------------------------------------------------------------ producer warp: the tiles of K and V
        if (lane == 0) {
            for (int t = 0; t < n_tiles; ++t) {
                const int s = t % kAttStages;
                if (!mbar_wait(smem_u32(bars + kAttStages + s), ((t / kAttStages) & 1) ^ 1, &abort_flag, sink)) break;
                const int row0 = (t_begin + t) * kAttRows;
                const int rows = min(kAttRows, Lc - row0);
                const uint32_t bar = smem_u32(bars + s);
                mbar_expect_tx(bar, 2u * (uint32_t)rows * kRowBytes);
                // one copy per operand, or two where the tile crosses a page boundary of a paged cache
                const int first = p.block_table ? min(rows, kTile - row0 % kTile) : rows;
                for (int part = 0; part < 2; ++part) {
                    const int r0 = part == 0 ? 0 : first, cnt = part == 0 ? first : rows - first;
                    if (cnt <= 0) break;
                    const size_t src = row_at(row0 + r0) * kHeadDim;
                    const uint32_t bytes = (uint32_t)cnt * kRowBytes, off = (uint32_t)r0 * kRowBytes;
                    asm volatile("cp.async.bulk.shared::cluster.global.mbarrier::complete_tx::bytes [%0], [%1], %2, [%3];"
                                 ::"r"(smem_u32(att_smem + (size_t)s * 2 * kTileBytesT) + off), "l"(K + src), "r"(bytes), "r"(bar)
                                 : "memory");
                    asm volatile("cp.async.bulk.shared::cluster.global.mbarrier::complete_tx::bytes [%0], [%1], %2, [%3];"
                                 ::"r"(smem_u32(att_smem + (size_t)s * 2 * kTileBytesT + kTileBytesT) + off), "l"(V + src), "r"(bytes),
                                   "r"(bar)
                                 : "memory");
                }
            }
        }
        __syncwarp();
    } else {
        // ------------------------------------------------------------------ compute warps
        // Every warp runs its own online softmax over its 8 rows of each tile (no block-wide barrier in the loop); the
        // warps' results are merged once, at the end.
        // The group's queries, scaled by log2(e) / sqrt(d): lane j of a row's 8 lanes holds vectors j, j + 8, ...
        const int sub = lane >> 3, j8 = lane & 7;
        float qreg[G][kVecPerLane * kPerVec];     // (used in pairs: packed fp32 multiply-adds, two per instruction)
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
        float m_run[G], l_run[G];            // running maximum (base-2 domain) and sum of this warp, the same in every lane
#pragma unroll
        for (int g = 0; g < G; ++g) {
            m_run[g] = -INFINITY;
            l_run[g] = 0.f;
        }
        float *my_w = wts + warp * kRowsPerWarp * GP;
        bool ok = true;

        for (int t = 0; t < n_tiles && ok; ++t) {
            const int s = t % kAttStages;
            const int row0 = (t_begin + t) * kAttRows;
            const int rows_here = min(kAttRows, Lc - row0);
            ok = mbar_wait(smem_u32(bars + s), (t / kAttStages) & 1, &abort_flag, sink);
            if (!ok) break;
            const uint8_t *kt = att_smem + (size_t)s * 2 * kTileBytesT, *vt = kt + kTileBytesT;

            // ---- scores of this warp's rows 8 w .. 8 w + 7, four at a time; every lane of a row's 8 ends up with them
            float sv[2][G];
#pragma unroll
            for (int it = 0; it < 2; ++it) {
                const int r = warp * kRowsPerWarp + it * 4 + sub;
                float2 dot2[G];
#pragma unroll
                for (int g = 0; g < G; ++g) dot2[g] = make_float2(0.f, 0.f);
                if (r < rows_here) {
#pragma unroll
                    for (int u = 0; u < kVecPerLane; ++u) {
                        float kf[kPerVec];
                        Elem<T>::unpack(*reinterpret_cast<const uint4 *>(kt + (size_t)r * kRowBytes + (j8 + 8 * u) * 16), kf);
#pragma unroll
                        for (int g = 0; g < G; ++g)
#pragma unroll
                            for (int e = 0; e < kPerVec; e += 2)
                                dot2[g] = __ffma2_rn(make_float2(qreg[g][u * kPerVec + e], qreg[g][u * kPerVec + e + 1]),
                                                     make_float2(kf[e], kf[e + 1]), dot2[g]);
                    }
                }
#pragma unroll
                for (int g = 0; g < G; ++g) {
                    float dot = dot2[g].x + dot2[g].y;
#pragma unroll
                    for (int off = 4; off > 0; off >>= 1) dot += __shfl_xor_sync(0xffffffffu, dot, off);
                    sv[it][g] = r < rows_here ? dot : -INFINITY;          // rows beyond the cached length take no part
                }
            }
            // ---- online softmax of the warp: new maximum over its 8 rows, rescale, the rows' weights
            __syncwarp();                       // the previous tile's weights are no longer read
#pragma unroll
            for (int g = 0; g < G; ++g) {
                float m = fmaxf(sv[0][g], sv[1][g]);
                m = fmaxf(m, __shfl_xor_sync(0xffffffffu, m, 8));
                m = fmaxf(m, __shfl_xor_sync(0xffffffffu, m, 16));
                const float m_new = fmaxf(m_run[g], m);
                // (a warp whose rows all lie beyond the length keeps m = -inf: nothing to rescale, weights 0)
                const float a = m_new == -INFINITY ? 1.f : exp2f(m_run[g] - m_new);
                const float w0 = m_new == -INFINITY ? 0.f : exp2f(sv[0][g] - m_new);
                const float w1 = m_new == -INFINITY ? 0.f : exp2f(sv[1][g] - m_new);
                float wsum = j8 == 0 ? w0 + w1 : 0.f;                    // one lane per row counts
                wsum += __shfl_xor_sync(0xffffffffu, wsum, 8);
                wsum += __shfl_xor_sync(0xffffffffu, wsum, 16);
                l_run[g] = l_run[g] * a + wsum;
                m_run[g] = m_new;
                const float2 a2 = make_float2(a, a);
                acc[g][0] = __fmul2_rn(acc[g][0], a2);
                acc[g][1] = __fmul2_rn(acc[g][1], a2);
                if (j8 == 0) {
                    my_w[sub * GP + g] = w0;
                    my_w[(4 + sub) * GP + g] = w1;
                }
            }
            __syncwarp();
            // ---- values: this warp's rows, lanes over d
            const int r_lo = warp * kRowsPerWarp, r_hi = min(r_lo + kRowsPerWarp, rows_here);
            for (int r = r_lo; r < r_hi; ++r) {
                float2 v01, v23;
                if (sizeof(T) == 2) {
                    const uint2 raw = *reinterpret_cast<const uint2 *>(vt + (size_t)r * kRowBytes + lane * 8);
                    const __nv_bfloat162 *h2 = reinterpret_cast<const __nv_bfloat162 *>(&raw);
                    v01 = __bfloat1622float2(h2[0]);
                    v23 = __bfloat1622float2(h2[1]);
                } else {
                    const float4 raw = *reinterpret_cast<const float4 *>(vt + (size_t)r * kRowBytes + lane * 16);
                    v01 = make_float2(raw.x, raw.y);
                    v23 = make_float2(raw.z, raw.w);
                }
                float w[GP];                 // the row's weights of all query heads: one or two 16-byte broadcasts
#pragma unroll
                for (int g4 = 0; g4 < GP; g4 += 4) {
                    const float4 w4 = *reinterpret_cast<const float4 *>(my_w + (r - r_lo) * GP + g4);
                    w[g4] = w4.x, w[g4 + 1] = w4.y, w[g4 + 2] = w4.z, w[g4 + 3] = w4.w;
                }
#pragma unroll
                for (int g = 0; g < G; ++g) {
                    const float2 w2 = make_float2(w[g], w[g]);
                    acc[g][0] = __ffma2_rn(w2, v01, acc[g][0]);
                    acc[g][1] = __ffma2_rn(w2, v23, acc[g][1]);
                }
            }
            __syncwarp();
            if (lane == 0) mbar_arrive(smem_u32(bars + kAttStages + s));       // this warp is done with the stage
        }
        if (lane == 0) {
#pragma unroll
            for (int g = 0; g < G; ++g) {
                wstat[(warp * G + g) * 2] = m_run[g];
                wstat[(warp * G + g) * 2 + 1] = ok ? l_run[g] : 0.f;      // error path: zeros (the status word says why)
            }
        }
    }
    if (*reinterpret_cast<volatile int *>(&abort_flag)) __nanosleep(200000);   // error path only: let copies in flight land
    __syncthreads();                     // every warp is through with the tile stages
    if (warp < kAttWarps) {
        float *fold_w = reinterpret_cast<float *>(att_smem);      // [kAttWarps][G][128], in the room of the stages
#pragma unroll
        for (int g = 0; g < G; ++g)
            *reinterpret_cast<float4 *>(fold_w + ((size_t)warp * G + g) * kHeadDim + lane * 4) =
                make_float4(acc[g][0].x, acc[g][0].y, acc[g][1].x, acc[g][1].y);
    }
    __syncthreads();

    // ---- merge the warps' results (fixed order): out = sum_w 2^(m_w - m) acc_w / sum_w 2^(m_w - m) l_w
    const float *fold = reinterpret_cast<const float *>(att_smem);
    for (int x = threadIdx.x; x < G * kHeadDim; x += blockDim.x) {
        const int g = x / kHeadDim, c = x % kHeadDim;
        float m = -INFINITY;
#pragma unroll
        for (int w = 0; w < kAttWarps; ++w) m = fmaxf(m, wstat[(w * G + g) * 2]);
        float num = 0.f, den = 0.f;
#pragma unroll
        for (int w = 0; w < kAttWarps; ++w) {
            const float mw = wstat[(w * G + g) * 2];
            const float f = mw == -INFINITY ? 0.f : exp2f(mw - m);
            num = fmaf(f, fold[((size_t)w * G + g) * kHeadDim + c], num);
            den = fmaf(f, wstat[(w * G + g) * 2 + 1], den);
        }
        if (p.splits == 1) {
            p.out[((size_t)b * p.hq + (size_t)h * G + g) * kHeadDim + c] = den > 0.f ? num / den : 0.f;
        } else {
            float *part = p.partial + (((size_t)head * p.splits + split) * G + g) * (kHeadDim + 2);
            part[c] = num;
            if (c == 0) {
                part[kHeadDim] = m;
                part[kHeadDim + 1] = den;
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
    if (c < p.d_out) p.out[((size_t)b * p.hq + (size_t)h * G + g) * p.d_out + c] = den > 0.f ? num / den : 0.f;
}

template <typename T, int G>
cudaError_t launch_one(const AttendParams &p, cudaStream_t s)
{
    const int tile_bytes = kAttRows * kHeadDim * (int)sizeof(T);
    const int smem = kAttStages * 2 * tile_bytes + (kAttWarps * (kAttRows / kAttWarps) * ((G + 3) / 4 * 4) + kAttWarps * G * 2) * 4 +
                     2 * kAttStages * 8 + 16;
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

// Head dimension 128 for every cache type; 64 for bf16 caches (the tensor-core kernel pads the tiles to 128).
bool attend_supported(int G, int dtype, int head_dim)
{
    if (G > kAttMaxG) return false;
    return head_dim == kHeadDim || (head_dim == 64 && dtype == RKV_BF16);
}

// bf16 and 8-bit caches go to the tensor-core kernel whatever the group size (it runs at the rate HBM can be read at; this kernel
// reached 0.74 of the copy bandwidth at G = 4 and ran out of issue slots from G = 5 on); fp32 caches stay here.
bool attend_uses_tc(int G, int dtype) { return (dtype == RKV_BF16 || dtype == RKV_FP8_E4M3) && G >= 1; }

// Splits of a head's rows: enough blocks for two waves of resident blocks (2 per SM), never finer than a tile.
int attend_splits(int heads, int cap, int sms, int G, int dtype)
{
    if (attend_uses_tc(G, dtype)) return attend_tc_splits(heads, cap, sms);
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
                          long long wait_cycles, const int32_t *block_table, long long pool_pages, int head_dim, cudaStream_t s)
{
    const int G = hq / hkv;
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
    p.block_table = block_table;
    p.d_out = head_dim;
    cudaError_t e;
    if (attend_uses_tc(G, dtype))
        e = launch_attend_tc(k_cache, v_cache, q_new, seq_lens, out, partial, batch, hkv, hq, cap, splits, status, wait_cycles,
                             block_table, pool_pages, dtype == RKV_FP8_E4M3 ? 1 : (head_dim == 64 ? 2 : 0), s);
    else
        e = launch_dtype<float>(p, G, s);
    if (e != cudaSuccess || splits == 1) return e;
    attend_merge_kernel<<<(unsigned)(batch * hkv * G), kHeadDim, 0, s>>>(p, G);
    return cudaGetLastError();
}

}  // namespace rkv

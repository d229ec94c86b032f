// Stage "select": one thread block per head-problem finishes the scores and picks the kept tokens.
//
//   Eq. 3  softmax over the candidate keys of each of the alpha pooled-logit rows
//   Eq. 4  sliding max over {i-W .. i+W-1} per row (taken on the logits: exp is monotone, so the
//          max of the weights is the weight of the max), mean over the alpha rows  -> I
//   Eq. 6  R = softmax over tokens of the column means left by the scoring stage
//   Eq. 7  Z = lambda I - (1 - lambda) R
//   top-k  exact k-th largest Z by a 4 x 8-bit radix select over order-preserving integer keys in shared
//          memory; among equal scores the later position is kept; the kept candidate positions are written
//          in ascending order, then the alpha observation positions.
//
// Latency-bound (about 40 bytes per token, all of it L2-resident scratch).
#include "rkv_common.cuh"

namespace rkv {

namespace {

constexpr int kSelThreads = 1024;
constexpr int kSelWarps = kSelThreads / 32;
constexpr int kMaxItems = RKV_MAX_CAP / kSelThreads;   // tokens per thread, upper bound

__device__ __forceinline__ uint32_t order_key(float z)
{
    // monotone map float -> uint32: larger float <=> larger key (-0 and +0 differ; harmless)
    uint32_t u = __float_as_uint(z);
    return (u & 0x80000000u) ? ~u : (u | 0x80000000u);
}

__device__ __forceinline__ float block_max(float v, float *scratch)
{
#pragma unroll
    for (int off = 16; off > 0; off >>= 1) v = fmaxf(v, __shfl_xor_sync(0xffffffffu, v, off));
    __syncthreads();
    if ((threadIdx.x & 31) == 0) scratch[threadIdx.x >> 5] = v;
    __syncthreads();
    float r = scratch[threadIdx.x & 31];    // kSelWarps == 32
#pragma unroll
    for (int off = 16; off > 0; off >>= 1) r = fmaxf(r, __shfl_xor_sync(0xffffffffu, r, off));
    return r;
}

__device__ __forceinline__ float block_sum(float v, float *scratch)
{
    // fixed reduction tree: the result does not depend on scheduling
#pragma unroll
    for (int off = 16; off > 0; off >>= 1) v += __shfl_xor_sync(0xffffffffu, v, off);
    __syncthreads();
    if ((threadIdx.x & 31) == 0) scratch[threadIdx.x >> 5] = v;
    __syncthreads();
    float r = scratch[threadIdx.x & 31];
#pragma unroll
    for (int off = 16; off > 0; off >>= 1) r += __shfl_xor_sync(0xffffffffu, r, off);
    return r;
}

__global__ void __launch_bounds__(kSelThreads) select_kernel(Params p)
{
    extern __shared__ float row[];                 // [cap_pad] one logits row / the Sbar row, then the keys
    __shared__ float scratch[kSelWarps];
    __shared__ uint32_t hist[256];
    __shared__ uint32_t sel_prefix, sel_want;
    __shared__ uint32_t warp_tot[kSelWarps];

    const int head = blockIdx.x;
    const int b = head / p.hkv;
    const int tid = threadIdx.x;
    const int L = p.meta[b];
    int32_t *out = p.out_idx + (size_t)head * p.budget;

    if (L <= p.budget) {      // Algorithm 1's guard (or an invalid length): nothing is compressed
        for (int j = tid; j < p.budget; j += kSelThreads) out[j] = (j < L) ? j : -1;
        return;
    }
    const int n = L - p.alpha;
    const int k = p.budget - p.alpha;
    const int W = p.pool_w;

    // ---- Eq. 3-4: importance
    float I_acc[kMaxItems];
#pragma unroll
    for (int t = 0; t < kMaxItems; ++t) I_acc[t] = 0.f;
    const float *logits = p.logits + (size_t)head * p.alpha * p.cap_pad;
    for (int j = 0; j < p.alpha; ++j) {
        __syncthreads();
        float m = -INFINITY;
        for (int i = tid; i < n; i += kSelThreads) {
            const float l = logits[(size_t)j * p.cap_pad + i];
            row[i] = l;
            m = fmaxf(m, l);
        }
        m = block_max(m, scratch);
        float s = 0.f;
        for (int i = tid; i < n; i += kSelThreads) s += expf(row[i] - m);
        s = block_sum(s, scratch);
        const float inv = 1.0f / s;
#pragma unroll
        for (int t = 0; t < kMaxItems; ++t) {
            const int i = tid + t * kSelThreads;
            if (i < n) {
                float best = row[i];
                const int lo = max(i - W, 0), hi = min(i + W - 1, n - 1);
                for (int u = lo; u <= hi; ++u) best = fmaxf(best, row[u]);
                I_acc[t] += expf(best - m) * inv;
            }
        }
    }

    // ---- Eq. 6: R = softmax(Sbar)
    __syncthreads();
    const float *sbar = p.sbar + (size_t)head * p.cap_pad;
    float m = -INFINITY;
    for (int i = tid; i < n; i += kSelThreads) {
        float v = sbar[i];
        if (p.tri) v = v / (float)n;        // the triangle kernels leave the column sum minus the removed entries
        row[i] = v;
        m = fmaxf(m, v);
    }
    m = block_max(m, scratch);
    float s = 0.f;
    for (int i = tid; i < n; i += kSelThreads) s += expf(row[i] - m);
    s = block_sum(s, scratch);
    const float inv = 1.0f / s;
    const float inv_alpha = 1.0f / (float)p.alpha;

    // ---- Eq. 7 and the integer keys (kept in the same shared row, one owner per slot)
    uint32_t *keys = reinterpret_cast<uint32_t *>(row);
    const size_t dbg = (size_t)head * p.cap;
#pragma unroll
    for (int t = 0; t < kMaxItems; ++t) {
        const int i = tid + t * kSelThreads;
        if (i < n) {
            const float I = I_acc[t] * inv_alpha;
            const float sb = row[i];
            const float R = expf(sb - m) * inv;
            const float Z = p.lambda * I - (1.0f - p.lambda) * R;
            if (p.dbg_I) p.dbg_I[dbg + i] = I;
            if (p.dbg_Sbar) p.dbg_Sbar[dbg + i] = sb;
            if (p.dbg_R) p.dbg_R[dbg + i] = R;
            if (p.dbg_Z) p.dbg_Z[dbg + i] = Z;
            keys[i] = order_key(Z);
        }
    }
    if (tid == 0) {
        sel_prefix = 0u;
        sel_want = (uint32_t)k;
    }

    // ---- radix select: the k-th largest key, 8 bits at a time from the top
    for (int shift = 24; shift >= 0; shift -= 8) {
        if (tid < 256) hist[tid] = 0u;
        __syncthreads();
        const uint32_t prefix = sel_prefix;
        const uint32_t high_mask = (shift == 24) ? 0u : (0xffffffffu << (shift + 8));
        for (int i = tid; i < n; i += kSelThreads) {
            const uint32_t key = keys[i];
            if ((key & high_mask) == prefix) atomicAdd(&hist[(key >> shift) & 255u], 1u);
        }
        __syncthreads();
        if (tid < 32) {
            // lane l owns digits 255-8l .. 248-8l (descending); find the digit holding the want-th key
            const uint32_t want = sel_want;        // read before any lane may overwrite it below
            uint32_t local[8], sum = 0u;
#pragma unroll
            for (int e = 0; e < 8; ++e) {
                local[e] = hist[255 - (tid * 8 + e)];
                sum += local[e];
            }
            uint32_t incl = sum;
#pragma unroll
            for (int off = 1; off < 32; off <<= 1) {
                const uint32_t o = __shfl_up_sync(0xffffffffu, incl, off);
                if (tid >= off) incl += o;
            }
            uint32_t run = incl - sum;             // keys in larger digits, owned by earlier lanes
            __syncwarp();
#pragma unroll
            for (int e = 0; e < 8; ++e) {          // exactly one (lane, e) holds the want-th key
                if (run < want && want <= run + local[e]) {
                    sel_prefix = prefix | ((uint32_t)(255 - (tid * 8 + e)) << shift);
                    sel_want = want - run;
                }
                run += local[e];
            }
        }
        __syncthreads();
    }
    const uint32_t theta = sel_prefix;   // key of the k-th largest score
    const uint32_t need_eq = sel_want;   // how many tokens equal to theta are kept (the latest ones)

    // ---- emit the kept positions in ascending order
    const int per = (n + kSelThreads - 1) / kSelThreads;      // contiguous tokens per thread
    const int first = tid * per, last = min(first + per, n);
    uint32_t gt = 0u, eq = 0u;
    for (int i = first; i < last; ++i) {
        const uint32_t key = keys[i];
        gt += (key > theta);
        eq += (key == theta);
    }
    uint32_t packed = (gt << 16) | eq;     // n <= 8192: both counts fit 16 bits, sums never carry across
    uint32_t incl = packed;
    const int lane = tid & 31, warp = tid >> 5;
#pragma unroll
    for (int off = 1; off < 32; off <<= 1) {
        const uint32_t o = __shfl_up_sync(0xffffffffu, incl, off);
        if (lane >= off) incl += o;
    }
    if (lane == 31) warp_tot[warp] = incl;
    __syncthreads();
    uint32_t wsum = warp_tot[lane], wincl = wsum;
#pragma unroll
    for (int off = 1; off < 32; off <<= 1) {
        const uint32_t o = __shfl_up_sync(0xffffffffu, wincl, off);
        if (lane >= off) wincl += o;
    }
    const uint32_t total = __shfl_sync(0xffffffffu, wincl, 31);
    const uint32_t warp_excl = __shfl_sync(0xffffffffu, wincl - wsum, warp);
    const uint32_t excl = warp_excl + incl - packed;
    const uint32_t total_eq = total & 0xffffu;
    const uint32_t skip_eq = total_eq - need_eq;    // the earliest ties are the ones dropped
    uint32_t g = excl >> 16, q = excl & 0xffffu;
    for (int i = first; i < last; ++i) {
        const uint32_t key = keys[i];
        const uint32_t kept_before = g + (q > skip_eq ? q - skip_eq : 0u);
        if (key > theta) {
            out[kept_before] = i;
            ++g;
        } else if (key == theta) {
            if (q >= skip_eq) out[kept_before] = i;
            ++q;
        }
    }
    for (int j = tid; j < p.alpha; j += kSelThreads) out[k + j] = n + j;   // observation tokens
}

}  // namespace

cudaError_t launch_select(const Params &p, cudaStream_t s)
{
    const size_t smem = (size_t)p.cap_pad * sizeof(float);
    cudaError_t e = cudaFuncSetAttribute(select_kernel, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)smem);
    if (e != cudaSuccess) return e;
    select_kernel<<<(unsigned)(p.batch * p.hkv), kSelThreads, smem, s>>>(p);
    return cudaGetLastError();
}

}  // namespace rkv

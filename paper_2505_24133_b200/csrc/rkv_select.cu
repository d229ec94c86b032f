// Stage "select": three kernels finish the scores and pick the kept tokens.
//
//   row_stats   one block per (head, query row): the maximum and the sum of exponentials of the row's n pooled
//               logits, i.e. the softmax of Eq. 3 in two numbers
//   importance  one block per (head, 1024 tokens): Eq. 4's sliding max over {i-W .. i+W-1} per row (taken on the
//               logits: exp is monotone, so the max of the weights is the weight of the max), the softmax weight of
//               that maximum, mean over the alpha rows  -> I
//   select      one block per head:
//     Eq. 6  R = softmax over tokens of the column means left by the scoring stage
//     Eq. 7  Z = lambda I - (1 - lambda) R
//     top-k  exact k-th largest Z by a 4 x 8-bit radix select over order-preserving integer keys in shared
//            memory; among equal scores the later position is kept; the kept candidate positions are written
//            in ascending order, then the alpha observation positions.
//
// All three read scratch that the scoring stage has just written (L2-resident for small batches).
#include "rkv_common.cuh"

namespace rkv {

namespace {

constexpr int kSelThreadsFused = 512;     // single-kernel form (small caches, often few heads): more threads per head
constexpr int kSelThreadsSplit = 256;     // three-kernel form: more blocks per SM hide the many block-wide barriers

__device__ __forceinline__ uint32_t order_key(float z)
{
    // monotone map float -> uint32: larger float <=> larger key (-0 and +0 differ; harmless)
    uint32_t u = __float_as_uint(z);
    return (u & 0x80000000u) ? ~u : (u | 0x80000000u);
}

template <int kSelThreads>
__device__ __forceinline__ float block_max(float v, float *scratch)
{
#pragma unroll
    for (int off = 16; off > 0; off >>= 1) v = fmaxf(v, __shfl_xor_sync(0xffffffffu, v, off));
    __syncthreads();
    if ((threadIdx.x & 31) == 0) scratch[threadIdx.x >> 5] = v;
    __syncthreads();
    constexpr int kSelWarps = kSelThreads / 32;
    float r = (threadIdx.x & 31) < kSelWarps ? scratch[threadIdx.x & 31] : -INFINITY;
#pragma unroll
    for (int off = 16; off > 0; off >>= 1) r = fmaxf(r, __shfl_xor_sync(0xffffffffu, r, off));
    return r;
}

template <int kSelThreads>
__device__ __forceinline__ float block_sum(float v, float *scratch)
{
    // fixed reduction tree: the result does not depend on scheduling
#pragma unroll
    for (int off = 16; off > 0; off >>= 1) v += __shfl_xor_sync(0xffffffffu, v, off);
    __syncthreads();
    if ((threadIdx.x & 31) == 0) scratch[threadIdx.x >> 5] = v;
    __syncthreads();
    constexpr int kSelWarps = kSelThreads / 32;
    float r = (threadIdx.x & 31) < kSelWarps ? scratch[threadIdx.x & 31] : 0.f;
#pragma unroll
    for (int off = 16; off > 0; off >>= 1) r += __shfl_xor_sync(0xffffffffu, r, off);
    return r;
}

constexpr size_t kFusedSmemLimit = 64 * 1024;   // largest shared-memory footprint for the single-kernel form
constexpr int kStatThreads = 256;
constexpr int kImpThreads = 256;
constexpr int kImpTokens = 1024;     // tokens per importance block

// Eq. 3 in two numbers per (head, query row): row_stat[..][0] = max_i logit, [1] = 1 / sum_i exp(logit - max).
__global__ void __launch_bounds__(kStatThreads) row_stats_kernel(Params p)
{
    __shared__ float scratch[kStatThreads / 32];
    const int head = blockIdx.x / p.alpha, j = blockIdx.x % p.alpha;
    const int n = seq_candidates(p, head / p.hkv);
    if (n == 0) return;
    const float *row = p.logits + ((size_t)head * p.alpha + j) * p.cap_pad;
    const int tid = threadIdx.x, lane = tid & 31, warp = tid >> 5;
    float m = -INFINITY;
    for (int i = tid; i < n; i += kStatThreads) m = fmaxf(m, row[i]);
#pragma unroll
    for (int off = 16; off > 0; off >>= 1) m = fmaxf(m, __shfl_xor_sync(0xffffffffu, m, off));
    if (lane == 0) scratch[warp] = m;
    __syncthreads();
    m = scratch[0];
#pragma unroll
    for (int w = 1; w < kStatThreads / 32; ++w) m = fmaxf(m, scratch[w]);
    __syncthreads();
    float s = 0.f;
    for (int i = tid; i < n; i += kStatThreads) s += expf(row[i] - m);      // second read: the row is in L1/L2
#pragma unroll
    for (int off = 16; off > 0; off >>= 1) s += __shfl_xor_sync(0xffffffffu, s, off);
    if (lane == 0) scratch[warp] = s;
    __syncthreads();
    if (tid == 0) {
        float t = 0.f;
        for (int w = 0; w < kStatThreads / 32; ++w) t += scratch[w];            // fixed order
        p.row_stat[((size_t)head * p.alpha + j) * 2] = m;
        p.row_stat[((size_t)head * p.alpha + j) * 2 + 1] = 1.0f / t;
    }
}

// Eq. 4 for kImpTokens tokens of one head.
__global__ void __launch_bounds__(kImpThreads) importance_kernel(Params p)
{
    const int chunks = (p.cap + kImpTokens - 1) / kImpTokens;
    const int head = blockIdx.x / chunks, i0 = (blockIdx.x % chunks) * kImpTokens;
    const int n = seq_candidates(p, head / p.hkv);
    if (i0 >= n) return;
    const int W = p.pool_w;
    const float *logits = p.logits + (size_t)head * p.alpha * p.cap_pad;
    const float *stat = p.row_stat + (size_t)head * p.alpha * 2;
    const float inv_alpha = 1.0f / (float)p.alpha;
    for (int i = i0 + threadIdx.x; i < min(i0 + kImpTokens, n); i += kImpThreads) {
        const int lo = max(i - W, 0), hi = min(i + W - 1, n - 1);
        if (p.mean_then_pool) {
            // Algorithm 1's order: the mean of the alpha softmax weights at each position of the window, then the max
            float best = 0.f;
            for (int u = min(lo, i); u <= max(hi, i); ++u) {
                float mean = 0.f;
                for (int j = 0; j < p.alpha; ++j)
                    mean += expf(logits[(size_t)j * p.cap_pad + u] - stat[2 * j]) * stat[2 * j + 1];
                best = fmaxf(best, mean * inv_alpha);
            }
            p.imp[(size_t)head * p.cap_pad + i] = best;
            continue;
        }
        float acc = 0.f;
        for (int j = 0; j < p.alpha; ++j) {
            const float *row = logits + (size_t)j * p.cap_pad;
            float best = row[i];
            for (int u = lo; u <= hi; ++u) best = fmaxf(best, row[u]);
            acc += expf(best - stat[2 * j]) * stat[2 * j + 1];
        }
        p.imp[(size_t)head * p.cap_pad + i] = acc * inv_alpha;
    }
}

// Exact top-k over n order-preserving keys in shared memory (written by the caller, one owner per slot; no barrier
// needed before the call), later position first among equal keys.  Writes the k kept positions in ascending order and
// then the alpha observation positions n .. n+alpha-1 into `copies` index lists of `budget` entries, `budget` apart.
template <int kSelThreads>
__device__ __forceinline__ void radix_select_emit(const uint32_t *keys, int n, int k, int alpha, int budget,
                                                  int32_t *out, int copies)
{
    constexpr int kSelWarps = kSelThreads / 32;
    __shared__ uint32_t hist[256];
    __shared__ uint32_t sel_prefix, sel_want;
    __shared__ uint32_t warp_tot[kSelWarps];
    const int tid = threadIdx.x;
    if (tid == 0) {
        sel_prefix = 0u;
        sel_want = (uint32_t)k;
    }

    // ---- radix select: the k-th largest key, 8 bits at a time from the top
    for (int shift = 24; shift >= 0; shift -= 8) {
        for (int t = tid; t < 256; t += kSelThreads) hist[t] = 0u;
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
    uint32_t wsum = lane < kSelWarps ? warp_tot[lane] : 0u, wincl = wsum;
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
            for (int c = 0; c < copies; ++c) out[(size_t)c * budget + kept_before] = i;
            ++g;
        } else if (key == theta) {
            if (q >= skip_eq)
                for (int c = 0; c < copies; ++c) out[(size_t)c * budget + kept_before] = i;
            ++q;
        }
    }
    for (int j = tid; j < alpha; j += kSelThreads)
        for (int c = 0; c < copies; ++c) out[(size_t)c * budget + k + j] = n + j;   // observation tokens
    for (int j = k + alpha + tid; j < budget; j += kSelThreads)                     // a sequence with a smaller budget of its own
        for (int c = 0; c < copies; ++c) out[(size_t)c * budget + j] = -1;
}

// Eq. 4 with the default window W = 4 (positions i-4 .. i+3), eight consecutive tokens per thread: per query row
// four 16-byte loads bring the 16 logits those windows cover, and the eight maxima come from a doubling scheme in
// registers (the general kernel above reads each logit nine times).
constexpr int kImp8Threads = 256;
constexpr int kImp8Tokens = kImp8Threads * 8;

__global__ void __launch_bounds__(kImp8Threads) importance_w4_kernel(Params p)
{
    const int chunks = (p.cap + kImp8Tokens - 1) / kImp8Tokens;
    const int head = blockIdx.x / chunks;
    const int i0 = (blockIdx.x % chunks) * kImp8Tokens + threadIdx.x * 8;     // first token of this thread
    const int n = seq_candidates(p, head / p.hkv);
    if (i0 >= n) return;
    const float *logits = p.logits + (size_t)head * p.alpha * p.cap_pad;
    const float *stat = p.row_stat + (size_t)head * p.alpha * 2;
    const float kNegInf = -INFINITY;
    const bool interior = i0 >= 4 && i0 + 11 < n;      // all 16 positions i0-4 .. i0+11 are candidates
    float acc[8];
#pragma unroll
    for (int t = 0; t < 8; ++t) acc[t] = 0.f;
    for (int j = 0; j < p.alpha; ++j) {
        const float *row = logits + (size_t)j * p.cap_pad;
        float x[16];                                    // x[u] = logit at position i0 - 4 + u
        {
            const float4 *r4 = reinterpret_cast<const float4 *>(row + i0);       // i0 is a multiple of 8
            const float4 a = i0 >= 4 ? r4[-1] : make_float4(kNegInf, kNegInf, kNegInf, kNegInf);
            const float4 b = r4[0], c = r4[1];          // i0 + 7 < cap_pad (a multiple of 128)
            const float4 d = i0 + 8 < p.cap_pad ? r4[2] : make_float4(kNegInf, kNegInf, kNegInf, kNegInf);
            x[0] = a.x, x[1] = a.y, x[2] = a.z, x[3] = a.w, x[4] = b.x, x[5] = b.y, x[6] = b.z, x[7] = b.w;
            x[8] = c.x, x[9] = c.y, x[10] = c.z, x[11] = c.w, x[12] = d.x, x[13] = d.y, x[14] = d.z, x[15] = d.w;
        }
        if (!interior) {                                // the window is clipped to the candidates [0, n)
#pragma unroll
            for (int u = 0; u < 16; ++u) {
                const int pos = i0 - 4 + u;
                if (pos < 0 || pos >= n) x[u] = kNegInf;
            }
        }
        float m2[15], m4[13];
#pragma unroll
        for (int u = 0; u < 15; ++u) m2[u] = fmaxf(x[u], x[u + 1]);
#pragma unroll
        for (int u = 0; u < 13; ++u) m4[u] = fmaxf(m2[u], m2[u + 2]);
        const float mj = stat[2 * j], inv = stat[2 * j + 1];
#pragma unroll
        for (int t = 0; t < 8; ++t)                     // token i0 + t: positions i0 + t - 4 .. i0 + t + 3 = x[t .. t+7]
            acc[t] += expf(fmaxf(m4[t], m4[t + 4]) - mj) * inv;
    }
    const float inv_alpha = 1.0f / (float)p.alpha;
    float *out = p.imp + (size_t)head * p.cap_pad + i0;
#pragma unroll
    for (int t = 0; t < 8; ++t)
        if (i0 + t < n) out[t] = acc[t] * inv_alpha;
}

// kFused: the block first does the work of row_stats_kernel and importance_kernel for its head, with the pooled
// logits in shared memory (small caches only: one launch instead of three, all of them latency-bound there).
template <bool kFused>
__global__ void __launch_bounds__(kFused ? kSelThreadsFused : kSelThreadsSplit, kFused ? 2 : 4) select_kernel(Params p)
{
    constexpr int kSelThreads = kFused ? kSelThreadsFused : kSelThreadsSplit;
    constexpr int kSelWarps = kSelThreads / 32;
    extern __shared__ float row[];                 // [cap_pad] one logits row / the Sbar row, then the keys;
                                                   // kFused: then [cap_pad] importance and [alpha][cap_pad] logits
    __shared__ float stat_s[2 * RKV_MAX_GROUP_ROWS];
    __shared__ float scratch[kSelWarps];

    const int head = blockIdx.x;
    const int b = head / p.hkv;
    const int tid = threadIdx.x;
    const int L = p.meta[b];
    int32_t *out = p.out_idx + (size_t)head * p.budget;

    if (call_aborted(p)) {    // a bounded wait of an earlier stage ran out: the scores are incomplete, nothing is selected
        for (int j = tid; j < p.budget; j += kSelThreads) out[j] = -1;
        return;
    }
    const int budget_b = seq_budget(p, b);
    if (L <= budget_b) {      // Algorithm 1's guard (or an invalid length): nothing is compressed
        for (int j = tid; j < p.budget; j += kSelThreads) out[j] = (j < L) ? j : -1;
        return;
    }
    const int n = L - p.alpha;
    const int k = budget_b - p.alpha;

    const float *imp = p.imp + (size_t)head * p.cap_pad;
    if (kFused) {
        float *imp_s = row + p.cap_pad, *lg = row + 2 * p.cap_pad;
        const float *logits = p.logits + (size_t)head * p.alpha * p.cap_pad;
        const int lane = tid & 31, warp = tid >> 5;
        for (int j = 0; j < p.alpha; ++j)
            for (int i = tid; i < n; i += kSelThreads) lg[j * p.cap_pad + i] = logits[(size_t)j * p.cap_pad + i];
        __syncthreads();
        for (int j = warp; j < p.alpha; j += kSelWarps) {      // Eq. 3: one warp per query row
            const float *r = lg + j * p.cap_pad;
            float mj = -INFINITY;
            for (int i = lane; i < n; i += 32) mj = fmaxf(mj, r[i]);
#pragma unroll
            for (int off = 16; off > 0; off >>= 1) mj = fmaxf(mj, __shfl_xor_sync(0xffffffffu, mj, off));
            float sj = 0.f;
            for (int i = lane; i < n; i += 32) sj += expf(r[i] - mj);
#pragma unroll
            for (int off = 16; off > 0; off >>= 1) sj += __shfl_xor_sync(0xffffffffu, sj, off);
            if (lane == 0) {
                stat_s[2 * j] = mj;
                stat_s[2 * j + 1] = 1.0f / sj;
            }
        }
        __syncthreads();
        const int W = p.pool_w;
        const float inv_alpha = 1.0f / (float)p.alpha;
        if (p.mean_then_pool) {
            // Algorithm 1's order: the mean of the alpha softmax weights per position (kept in `row`, free until
            // Eq. 6), then the max over the window
            for (int i = tid; i < n; i += kSelThreads) {
                float mean = 0.f;
                for (int j = 0; j < p.alpha; ++j) mean += expf(lg[j * p.cap_pad + i] - stat_s[2 * j]) * stat_s[2 * j + 1];
                row[i] = mean * inv_alpha;
            }
            __syncthreads();
            for (int i = tid; i < n; i += kSelThreads) {
                float best = row[i];
                for (int u = max(i - W, 0); u <= min(i + W - 1, n - 1); ++u) best = fmaxf(best, row[u]);
                imp_s[i] = best;
            }
            __syncthreads();                                    // `row` is about to be reused
        } else
        for (int i = tid; i < n; i += kSelThreads) {            // Eq. 4
            const int lo = max(i - W, 0), hi = min(i + W - 1, n - 1);
            float acc = 0.f;
            for (int j = 0; j < p.alpha; ++j) {
                const float *r = lg + j * p.cap_pad;
                float best = r[i];
                for (int u = lo; u <= hi; ++u) best = fmaxf(best, r[u]);
                acc += expf(best - stat_s[2 * j]) * stat_s[2 * j + 1];
            }
            imp_s[i] = acc * inv_alpha;
        }
        imp = imp_s;
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
    m = block_max<kSelThreads>(m, scratch);
    float s = 0.f;
    for (int i = tid; i < n; i += kSelThreads) s += expf(row[i] - m);
    s = block_sum<kSelThreads>(s, scratch);
    const float inv = 1.0f / s;

    // ---- Eq. 7 and the integer keys (kept in the same shared row, one owner per slot)
    uint32_t *keys = reinterpret_cast<uint32_t *>(row);
    const size_t dbg = (size_t)head * p.cap;
    for (int i = tid; i < n; i += kSelThreads) {
        {
            const float I = imp[i];
            const float sb = row[i];
            const float R = expf(sb - m) * inv;
            const float Z = p.lambda * I - (1.0f - p.lambda) * R;
            if (p.dbg_I) p.dbg_I[dbg + i] = I;
            if (p.dbg_Sbar) p.dbg_Sbar[dbg + i] = sb;
            if (p.dbg_R) p.dbg_R[dbg + i] = R;
            if (p.dbg_Z) p.dbg_Z[dbg + i] = Z;
            if (p.head_mean) p.imp[(size_t)head * p.cap_pad + i] = Z;     // slot i is read (above) and written by this thread only
            keys[i] = order_key(Z);
        }
    }
    if (p.head_mean) return;      // Z of this head is in p.imp; select_mean_kernel picks the sequence's positions
    radix_select_emit<kSelThreads>(keys, n, k, p.alpha, p.budget, out, 1);
}

// Algorithm 1's aggregated selection, one block per sequence: AggScore_i = mean over the KV heads of Z_i^h (left in
// p.imp by select_kernel), exact top-k on it, the same index list written for every head of the sequence.
__global__ void __launch_bounds__(kSelThreadsSplit, 4) select_mean_kernel(Params p)
{
    constexpr int kSelThreads = kSelThreadsSplit;
    extern __shared__ float row[];
    const int b = blockIdx.x, tid = threadIdx.x;
    const int L = p.meta[b];
    if (call_aborted(p)) return;    // select_kernel has written -1 everywhere
    if (L <= seq_budget(p, b)) return;      // select_kernel has written the identity lists
    const int n = L - p.alpha;
    uint32_t *keys = reinterpret_cast<uint32_t *>(row);
    const float *z = p.imp + (size_t)b * p.hkv * p.cap_pad;
    const float hkv = (float)p.hkv;
    for (int i = tid; i < n; i += kSelThreads) {
        float acc = 0.f;
        for (int h = 0; h < p.hkv; ++h) acc += z[(size_t)h * p.cap_pad + i];      // fixed head order
        keys[i] = order_key(acc / hkv);
    }
    radix_select_emit<kSelThreads>(keys, n, seq_budget(p, b) - p.alpha, p.alpha, p.budget, p.out_idx + (size_t)b * p.hkv * p.budget, p.hkv);
}

}  // namespace

bool select_is_fused(int cap_pad, int alpha) { return (size_t)(alpha + 2) * cap_pad * sizeof(float) <= kFusedSmemLimit; }

static cudaError_t launch_select_mean(const Params &p, cudaStream_t s)
{
    const size_t smem = (size_t)p.cap_pad * sizeof(float);
    cudaError_t e = cudaFuncSetAttribute(select_mean_kernel, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)smem);
    if (e != cudaSuccess) return e;
    select_mean_kernel<<<(unsigned)p.batch, kSelThreadsSplit, smem, s>>>(p);
    return cudaGetLastError();
}

cudaError_t launch_select(const Params &p, cudaStream_t s)
{
    const unsigned heads = (unsigned)(p.batch * p.hkv);
    cudaError_t e;
    if (select_is_fused(p.cap_pad, p.alpha)) {
        // small caches: one kernel does row statistics, importance and selection
        if ((e = mark_kernel(p, 2, s)) != cudaSuccess || (e = mark_kernel(p, 3, s)) != cudaSuccess) return e;
        const size_t smem = (size_t)(p.alpha + 2) * p.cap_pad * sizeof(float);
        if ((e = cudaFuncSetAttribute(select_kernel<true>, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)smem)) !=
            cudaSuccess)
            return e;
        select_kernel<true><<<heads, kSelThreadsFused, smem, s>>>(p);
        if ((e = cudaGetLastError()) != cudaSuccess) return e;
        return p.head_mean ? launch_select_mean(p, s) : cudaSuccess;
    }
    row_stats_kernel<<<heads * (unsigned)p.alpha, kStatThreads, 0, s>>>(p);
    if ((e = cudaGetLastError()) != cudaSuccess) return e;
    if ((e = mark_kernel(p, 2, s)) != cudaSuccess) return e;
    if (p.pool_w == 4 && !p.mean_then_pool)
        importance_w4_kernel<<<heads * (unsigned)((p.cap + kImp8Tokens - 1) / kImp8Tokens), kImp8Threads, 0, s>>>(p);
    else
        importance_kernel<<<heads * (unsigned)((p.cap + kImpTokens - 1) / kImpTokens), kImpThreads, 0, s>>>(p);
    if ((e = cudaGetLastError()) != cudaSuccess) return e;
    if ((e = mark_kernel(p, 3, s)) != cudaSuccess) return e;
    const size_t smem = (size_t)p.cap_pad * sizeof(float);
    if ((e = cudaFuncSetAttribute(select_kernel<false>, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)smem)) !=
        cudaSuccess)
        return e;
    select_kernel<false><<<heads, kSelThreadsSplit, smem, s>>>(p);
    if ((e = cudaGetLastError()) != cudaSuccess) return e;
    return p.head_mean ? launch_select_mean(p, s) : cudaSuccess;
}

}  // namespace rkv

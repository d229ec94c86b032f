// Internal declarations shared by the kernels of the R-KV compression library (sm_100a).
// Nothing here is part of the public ABI (see include/rkv.h).
#pragma once

#include <cuda_bf16.h>
#include <cuda_fp8.h>
#include <cuda_runtime.h>
#include <stdint.h>

#include "rkv.h"

namespace rkv {

constexpr int kHeadDim = 128;   // d of the tensor-core kernels (other head dimensions go through the CUDA-core kernels)
constexpr int kTile = 128;      // keys per tile (rows of one tensor-core operand tile)

// meta[b] values
constexpr int kMetaInvalid = -1;

// Everything a kernel needs; passed by value.
struct Params {
    // caller tensors
    void *k_cache;
    void *v_cache;
    const void *q_window;
    int32_t *seq_lens;
    int32_t *out_idx;
    // shapes
    int batch, hkv, hq, group;      // group = G
    int d;                          // head dimension: 64, 128 or 256
    int cap, cap_pad, tiles;        // cap_pad = tiles * kTile
    int budget, buffer, alpha;
    int dtype;                      // of the keys the scoring stages read (bf16 for 8-bit caches: their widened copy)
    int store_row_bytes;            // bytes of a row of the caches as stored (what the gather moves)
    float logit_scale;              // Eq. 2's 1 / sqrt(d) with the caches' own head dimension (d above may be a padded one)
    // prep writes the scoring copy itself (k_cache above) from the stored keys: 0 = no, 1 = rows of 128 E4M3 codes,
    // 2 = rows of 64 bf16
    int fuse_mode;
    const void *fuse_src;           // the stored keys
    const int32_t *fuse_table;      // their block table (paged caches), else null
    // hyper-parameters
    int pool_w, beta;
    int head_mean;                  // Algorithm 1's aggregated selection: one kept set per sequence from the
                                    // head-averaged Z (select_kernel then leaves Z in `imp` and a second kernel selects)
    int gqa_mean_pool;              // Eq. 3 with the mean over the group's query heads instead of the max
    int mean_then_pool;             // importance in Algorithm 1's order (mean over query rows, then pooling)
    float sim_threshold, eps, lambda;
    // workspace carve-up
    float *inv_norm;     // [P][cap_pad]         r_i = 1 / (||k_i|| + eps); 0 for i >= n
    __nv_bfloat16 *norm_split;    // [P][cap_pad][16]  (n1, n2, n3, n1, n2, n1, 0 ...): 1 / r_i as three bf16 parts, laid
                                  // out as the extra K = 16 slice the scoring passes append to a key row
    __nv_bfloat16 *thr_split;     // [P][128][16]      (-t1, -t1, -t1, -t2, -t2, -t3, 0 ...): -T / r_j of the keys of the
                                  // head's LAST key tile as three bf16 parts, the slice the first scoring pass appends
                                  // to that tile's rows; the dot product of the two kinds of slice is -T / (r_i r_j)
                                  // to fp32 accuracy.  Both are written by the prep stage (two-pass route only).
    float *tile_sum;     // [P][tiles][128]      sum over the tile's candidate rows of r_i * k_i
    float *head_sum;     // [P][128]             sum over all candidate rows of r_i * k_i (the tile sums added up)
    float *logits;       // [P][alpha][cap_pad]  Eq. 2-3: group-max of scaled logits
    float *row_stat;     // [P][alpha][2]        Eq. 3 per row: max logit, 1 / sum of exp(logit - max)
    float *imp;          // [P][cap_pad]         Eq. 4: importance I (head_mean: overwritten with Z by select_kernel)
    float *sbar;         // [P][cap_pad]         Eq. 6 column means after the retention rule.  With `tri` set the scoring
                         //                      kernels leave column SUMS minus the removed entries (the select stage
                         //                      divides by n)
    int32_t *left;       // [P][cap_pad]         tri: partners a token still lacks after the scan of its own line
    int32_t *strag;      // [P][cap_pad]         tri: positions of the head's tokens with left > 0, ascending
    int32_t *strag_count;// [P]                  tri: how many
    int4 *strag_items;   // [P * cap_pad / 256]  tri: work list of the second scoring pass: {head, first listed
                         //                      token, tokens (1..256), first streamed tile}
    uint32_t *best;      // [P][cap_pad]         symmetric route: largest partner position + 1 found so far (0 = none)
    int32_t *dense;      // [P]                  1: the head is scored by the symmetric route of the second pass
    int4 *dense_items;   // [P * ceil(tiles/2)]  its work list: {head, pair of row tiles, n, -}
    int dense_ok;        // the symmetric route may be chosen (beta = 1, not switched off)
    float *self_dot;     // [P][cap_pad]         Kbar_i . Kbar_i (1 up to rounding and eps; 0 for a zero key)
    __nv_bfloat16 *head_sum_bf16;   // [P][16][128] head_sum split into three bf16 rows (hi, mid, lo), 13 zero rows
    int32_t *meta;       // [2][batch]           snapshot of seq_lens (kMetaInvalid if out of range), then each
                         //                      sequence's budget (p.budget unless the caller gave per-sequence ones)
    const int32_t *budgets;   // optional [batch]: per-sequence budgets (alpha < budgets[b] <= budget), else null
    const int32_t *block_table;   // optional [P][cap / 128]: paged caches, page (= key tile) ids into the pools, else null
    int pages_per_head;           // cap / 128 (paged caches)
    long long pool_pages;         // pages in the pools (paged caches)
    // zeroed by the prep stage's memset, in this order, contiguous:
    unsigned long long *counters;   // [8]       [0] = similarity tiles computed by the tcgen05 kernels, [1] = item
                                    //           ticket of the first scoring pass, [2] = entries in strag_items,
                                    //           [3] = item ticket of the second pass, [4] = the call's abort word
                                    //           (non-zero once a bounded wait ran out: later kernels of the call
                                    //           then leave the caches, lengths and index lists alone),
                                    //           [5] = listed-token x key-tile pairs the second pass has to form,
                                    //           [8 + 2 r], [9 + 2 r] = work items and item ticket of its round r,
                                    //           [16], [17] = the same for the symmetric route
    uint32_t *tile_done;            // [P]       tiles of the head finished by the prep stage
    size_t zero_bytes;              // bytes from `counters` to the end of `tile_done`
    int tri;                        // 1: the triangle kernels score (bf16 default); 0: another kernel does
    // optional outputs
    void *const *kernel_events;     // see rkv_desc_t
    unsigned long long *dbg_counters;
    int32_t *status;
    long long wait_cycles;          // limit of every bounded wait, in clock64() ticks
    float *dbg_I, *dbg_Sbar, *dbg_R, *dbg_Z;
};

__host__ __device__ inline size_t align_up(size_t x, size_t a) { return (x + a - 1) / a * a; }

// Record optional event i of p.kernel_events on the stream.
inline cudaError_t mark_kernel(const Params &p, int i, cudaStream_t s)
{
    return (p.kernel_events && p.kernel_events[i]) ? cudaEventRecord(static_cast<cudaEvent_t>(p.kernel_events[i]), s)
                                                   : cudaSuccess;
}

__device__ __forceinline__ void report(int32_t *status, int code)
{
    if (status) atomicCAS(status, 0, code);
}

constexpr int kAbortWord = 4;       // index of the call's abort word in Params::counters
constexpr int kPairsWord = 5;       // index of the second pass's useful-work count
constexpr int kDenseWords = 16;     // counters[16], [17]: work items and item ticket of the symmetric route

// Where a bounded wait records that it ran out: the caller's optional status word, and the call's own abort word
// in the workspace, which the later kernels of the same call read.
struct ErrSink {
    int32_t *status;
    unsigned long long *abort_word;
    long long wait_cycles;
};
__device__ __forceinline__ ErrSink make_sink(const Params &p)
{
    return ErrSink{p.status, p.counters + kAbortWord, p.wait_cycles};
}
__device__ __forceinline__ void report_timeout(const ErrSink &sink)
{
    report(sink.status, RKV_ERR_TIMEOUT);
    if (sink.abort_word) atomicExch(sink.abort_word, 1ull);
}
// True once some kernel of this call has given up on a wait.
__device__ __forceinline__ bool call_aborted(const Params &p)
{
    return *reinterpret_cast<volatile unsigned long long *>(p.counters + kAbortWord) != 0ull;
}

// Number of candidates of a sequence of length L with the given budget: 0 = nothing to compress.
__device__ __forceinline__ int candidates_from_meta(int L, int budget, int alpha)
{
    return (L > budget) ? (L - alpha) : 0;
}
// Where key tile `tile` (128 rows) of head-problem `head` starts, in rows of the 2-D [rows][d] view of k_cache / v_cache:
// head after head for contiguous caches, through the block table for paged ones (a page holds one key tile).
__device__ __forceinline__ long long tile_row0(const Params &p, int head, int tile)
{
    return p.block_table ? (long long)p.block_table[(size_t)head * p.pages_per_head + tile] * kTile
                         : (long long)head * p.cap + (long long)tile * kTile;
}
// ... and row r of the head.
__device__ __forceinline__ long long row_index(const Params &p, int head, int r)
{
    return tile_row0(p, head, r / kTile) + (r % kTile);
}
// The same for sequence b as every stage after prep sees it (length and budget snapshots left by the prep stage).
__device__ __forceinline__ int seq_budget(const Params &p, int b) { return p.meta[p.batch + b]; }
__device__ __forceinline__ int seq_candidates(const Params &p, int b)
{
    return candidates_from_meta(p.meta[b], p.meta[p.batch + b], p.alpha);
}

template <typename T> struct Elem;
template <> struct Elem<__nv_bfloat16> {
    static constexpr int kPerVec = 8;   // elements per 16-byte vector
    __device__ static void unpack(const uint4 &v, float *f)
    {
        const __nv_bfloat162 *h = reinterpret_cast<const __nv_bfloat162 *>(&v);
#pragma unroll
        for (int i = 0; i < 4; ++i) {
            float2 t = __bfloat1622float2(h[i]);
            f[2 * i] = t.x;
            f[2 * i + 1] = t.y;
        }
    }
};
template <> struct Elem<float> {
    static constexpr int kPerVec = 4;
    __device__ static void unpack(const uint4 &v, float *f)
    {
        f[0] = __uint_as_float(v.x);
        f[1] = __uint_as_float(v.y);
        f[2] = __uint_as_float(v.z);
        f[3] = __uint_as_float(v.w);
    }
};

// 16 E4M3 codes -> 16 bf16 values (the conversion instruction goes through f16, which holds every E4M3 value too).
// (Measured against integer / packed-bf16 decodes of the codes -- shift the low seven bits into a bf16 pattern and
// multiply by 2^120 --: those were exact too, but slower in the kernel that widens tiles on their way to the tensor
// cores.)
__device__ __forceinline__ void widen16(const uint4 &codes, uint4 *lo, uint4 *hi)
{
    const uint32_t w[4] = {codes.x, codes.y, codes.z, codes.w};
    uint32_t out[8];
#pragma unroll
    for (int q = 0; q < 4; ++q) {
#pragma unroll
        for (int h = 0; h < 2; ++h) {
            const __half2_raw pair = __nv_cvt_fp8x2_to_halfraw2((__nv_fp8x2_storage_t)((w[q] >> (16 * h)) & 0xFFFFu), __NV_E4M3);
            const float2 f = __half22float2(*reinterpret_cast<const __half2 *>(&pair));
            const __nv_bfloat162 b2 = __floats2bfloat162_rn(f.x, f.y);
            out[2 * q + h] = *reinterpret_cast<const uint32_t *>(&b2);
        }
    }
    *lo = make_uint4(out[0], out[1], out[2], out[3]);
    *hi = make_uint4(out[4], out[5], out[6], out[7]);
}

// launchers (one per stage); each returns cudaGetLastError() of its launch
cudaError_t launch_prep(const Params &p, cudaStream_t s);
cudaError_t launch_widen_keys(const Params &stored, __nv_bfloat16 *wide, int wide_d, const void *q_src, void *q_dst,
                              bool keys, cudaStream_t s);
cudaError_t launch_scores_simt(const Params &p, cudaStream_t s);
cudaError_t launch_scores_sm100(const Params &p, cudaStream_t s);
cudaError_t launch_scores_tri_sm100(const Params &p, cudaStream_t s);
cudaError_t launch_select(const Params &p, cudaStream_t s);
cudaError_t launch_gather(const Params &p, cudaStream_t s);
cudaError_t launch_append(void *k_cache, void *v_cache, const void *k_new, const void *v_new, int32_t *seq_lens, int batch,
                          int hkv, int cap, int row_bytes, int32_t *status, const int32_t *block_table, cudaStream_t s);
cudaError_t launch_push_query(void *q_window, const void *q_new, int batch, int hq, int alpha, int slot, int row_bytes,
                              cudaStream_t s);
cudaError_t launch_attend(const void *k_cache, const void *v_cache, const void *q_new, const int32_t *seq_lens, float *out,
                          float *partial, int batch, int hkv, int hq, int cap, int splits, int dtype, int32_t *status,
                          long long wait_cycles, const int32_t *block_table, long long pool_pages, int head_dim, cudaStream_t s);
cudaError_t launch_attend_tc(const void *k_cache, const void *v_cache, const void *q_new, const int32_t *seq_lens, float *out,
                             float *partial, int batch, int hkv, int hq, int cap, int splits, int32_t *status,
                             long long wait_cycles, const int32_t *block_table, long long pool_pages, int src, cudaStream_t s);
int attend_tc_splits(int heads, int cap, int sms);
int attend_max_group();
int attend_splits(int heads, int cap, int sms, int G, int dtype);
bool attend_supported(int G, int dtype, int head_dim);
size_t attend_partial_bytes(int heads, int splits, int G);
bool scores_sm100_available();
long long sm100_default_wait_cycles();          // default limit of the kernels' bounded waits (about two seconds)
bool scores_dense_possible(int tiles, int beta);   // the symmetric route of the second pass may be taken (two more launches)
int scores_pass2_rounds(int tiles);            // list + scan rounds of the second scoring pass for caches of `tiles` key tiles
bool select_is_fused(int cap_pad, int alpha);   // the select stage is one kernel (small caches) instead of three

}  // namespace rkv

// C ABI of the R-KV compression library: argument checks, workspace carve-up, stage launches.
// See include/rkv.h for the contract of every entry point.
#include <cstdio>
#include <cstring>

#include "rkv_common.cuh"

namespace rkv {

namespace {

thread_local rkv_desc_t g_desc;
thread_local bool g_desc_set = false;
thread_local char g_cuda_error[256] = "";

int cuda_fail(cudaError_t e, const char *where)
{
    snprintf(g_cuda_error, sizeof(g_cuda_error), "%s: %s", where, cudaGetErrorString(e));
    return RKV_ERR_CUDA;
}

struct Layout {
    size_t k_wide, q_wide, best, dense, dense_items, inv_norm, norm_split, thr_split, tile_sum, head_sum, logits, row_stat, imp, sbar, left, strag, strag_count, strag_items, self_dot, head_sum_bf16, meta, counters,
        tile_done, zero_bytes, total;
    int cap, cap_pad, tiles, tri;
};

// The tensor-core scoring kernels are built for bf16 keys of 128 dimensions.  bf16 and 8-bit caches of 128 dimensions
// use them directly (8-bit: on a widened copy), those of 64 dimensions on a copy padded with zeros to 128 (dot products
// and norms do not see the padding); fp32 caches, 256 dimensions, or a request for it go to the CUDA-core kernel.
// Bytes of a cache element and of a query element.  8-bit caches (E4M3 codes) are scored on a bf16 copy of their keys
// in the workspace (every E4M3 value is a bf16 value), with bf16 queries.
size_t cache_esz(const rkv_desc_t *d) { return d->dtype == RKV_BF16 ? 2 : d->dtype == RKV_F32 ? 4 : 1; }
size_t query_esz(const rkv_desc_t *d) { return d->dtype == RKV_F32 ? 4 : 2; }

bool use_simt(const rkv_desc_t *d)
{
    return d->dtype == RKV_F32 || d->head_dim == 256 || (d->flags & RKV_FLAG_SIMT_SCORES);
}
// The head dimension is padded from 64 to 128 in the scoring copy (keys and observation queries).
bool pads_dim(const rkv_desc_t *d) { return d->head_dim == 64 && !use_simt(d); }
// The scoring stages read a copy of the keys in the workspace instead of the cache itself.
bool needs_copy(const rkv_desc_t *d) { return d->dtype == RKV_FP8_E4M3 || pads_dim(d); }
// Head dimension the scoring stages see.
int scoring_dim(const rkv_desc_t *d) { return pads_dim(d) ? kHeadDim : d->head_dim; }
// The prep kernel writes the copy of the keys itself (instead of a widening pass in front of it): stored rows of 128
// bytes that become 128 bf16, in caches whose capacity is a whole number of 128-row tiles.  1: E4M3 codes, 2: bf16 of
// 64 dimensions.
int fuse_mode(const rkv_desc_t *d, long long cap)
{
    if (!needs_copy(d) || scoring_dim(d) != kHeadDim || cap % kTile != 0) return 0;
    if (d->dtype == RKV_FP8_E4M3 && d->head_dim == kHeadDim) return 1;
    if (d->dtype == RKV_BF16 && d->head_dim == 64) return 2;
    return 0;
}

// 1 when the triangle tensor-core kernels score (bf16 caches, unless a cross-check kernel is asked for).
int use_tri(const rkv_desc_t *d) { return !(use_simt(d) || (d->flags & RKV_FLAG_ROWBLOCK_SCORES)); }

// Returns RKV_OK and fills *lay when the shape arguments are usable.
int check_shapes(const rkv_desc_t *d, int budget, int buffer, int alpha, Layout *lay)
{
    if (!d) return RKV_ERR_INVALID_ARG;
    if (d->batch < 1 || d->n_kv_heads < 1 || d->n_q_heads < 1) return RKV_ERR_INVALID_ARG;
    if (d->n_q_heads % d->n_kv_heads != 0) return RKV_ERR_INVALID_ARG;
    if (alpha < 1 || budget <= alpha || buffer < 1) return RKV_ERR_INVALID_ARG;
    if (d->pool_w < 0 || d->pool_w > 64 || d->beta < 0) return RKV_ERR_INVALID_ARG;
    if (!(d->sim_threshold >= 0.f && d->sim_threshold <= 1.f) || !(d->eps >= 0.f)) return RKV_ERR_INVALID_ARG;
    if (d->head_dim != 64 && d->head_dim != 128 && d->head_dim != 256) return RKV_ERR_UNSUPPORTED;
    if (d->dtype != RKV_BF16 && d->dtype != RKV_F32 && d->dtype != RKV_FP8_E4M3) return RKV_ERR_UNSUPPORTED;
    const long long cap = (long long)budget + buffer;
    if (cap > RKV_MAX_CAP) return RKV_ERR_UNSUPPORTED;
    if ((long long)(d->n_q_heads / d->n_kv_heads) * alpha > RKV_MAX_GROUP_ROWS) return RKV_ERR_UNSUPPORTED;
    if ((long long)d->batch * d->n_kv_heads > (1ll << 24)) return RKV_ERR_UNSUPPORTED;
    if (d->block_table) {      // paged caches: a page is one key tile
        if (cap % kTile != 0 || d->pool_pages < 1 || d->pool_pages > (1ll << 23)) return RKV_ERR_INVALID_ARG;
        if (reinterpret_cast<uintptr_t>(d->block_table) & 3u) return RKV_ERR_INVALID_ARG;
    }
    if (lay) {
        const size_t P = (size_t)d->batch * d->n_kv_heads;
        lay->cap = (int)cap;
        lay->tiles = (int)((cap + kTile - 1) / kTile);
        lay->cap_pad = lay->tiles * kTile;
        size_t off = 0;
        // the scoring copy (8-bit caches, padded head dimension): the keys as bf16, head after head, plus one tile of zero
        // rows behind the last head; with a padded head dimension the observation queries as well
        lay->k_wide = off;
        if (needs_copy(d)) off = align_up(off + (P * lay->cap + kTile) * (size_t)scoring_dim(d) * sizeof(__nv_bfloat16), 256);
        lay->q_wide = off;
        if (pads_dim(d)) off = align_up(off + (size_t)d->batch * d->n_q_heads * alpha * kHeadDim * sizeof(__nv_bfloat16), 256);
        lay->inv_norm = off;  off = align_up(off + P * lay->cap_pad * sizeof(float), 256);
        lay->norm_split = off;  off = align_up(off + P * lay->cap_pad * 16 * sizeof(__nv_bfloat16), 256);
        lay->thr_split = off;   off = align_up(off + P * kTile * 16 * sizeof(__nv_bfloat16), 256);
        const size_t hd = (size_t)scoring_dim(d);
        lay->tile_sum = off;  off = align_up(off + P * lay->tiles * hd * sizeof(float), 256);
        lay->head_sum = off;  off = align_up(off + P * hd * sizeof(float), 256);
        lay->logits = off;    off = align_up(off + P * alpha * lay->cap_pad * sizeof(float), 256);
        lay->row_stat = off;  off = align_up(off + P * alpha * 2 * sizeof(float), 256);
        lay->imp = off;       off = align_up(off + P * lay->cap_pad * sizeof(float), 256);
        lay->sbar = off;      off = align_up(off + P * lay->cap_pad * sizeof(float), 256);
        lay->tri = use_tri(d);
        const size_t tri = (size_t)lay->tri;
        lay->left = off;        off = align_up(off + tri * P * lay->cap_pad * sizeof(int32_t), 256);
        lay->strag = off;       off = align_up(off + tri * P * lay->cap_pad * sizeof(int32_t), 256);
        lay->strag_count = off; off = align_up(off + tri * P * sizeof(int32_t), 256);
        lay->strag_items = off; off = align_up(off + tri * P * (lay->cap_pad / 256 + 1) * sizeof(int4), 256);
        lay->best = off;        off = align_up(off + tri * P * lay->cap_pad * sizeof(uint32_t), 256);
        lay->dense = off;       off = align_up(off + tri * P * sizeof(int32_t), 256);
        lay->dense_items = off; off = align_up(off + tri * P * ((lay->tiles + 1) / 2) * sizeof(int4), 256);
        lay->self_dot = off;    off = align_up(off + P * lay->cap_pad * sizeof(float), 256);
        lay->head_sum_bf16 = off; off = align_up(off + P * 16 * hd * sizeof(__nv_bfloat16), 256);
        lay->meta = off;        off = align_up(off + 2 * (size_t)d->batch * sizeof(int32_t), 256);
        // the region the prep stage zeroes: counters and per-head tile tickets
        lay->counters = off;    off = align_up(off + 32 * sizeof(unsigned long long), 256);
        lay->tile_done = off;   off = align_up(off + P * sizeof(uint32_t), 256);
        lay->zero_bytes = off - lay->counters;
        lay->total = off;
    }
    return RKV_OK;
}

bool aligned16(const void *p) { return (reinterpret_cast<uintptr_t>(p) & 15u) == 0; }

int run(const rkv_desc_t *d, void *k_cache, void *v_cache, const void *q_window, int32_t *seq_lens, int budget,
        int buffer, int alpha, float lambda, int32_t *out_idx, void *stream, uint32_t stages)
{
    Layout lay;
    int rc = check_shapes(d, budget, buffer, alpha, &lay);
    if (rc != RKV_OK) return rc;
    if (!k_cache || !v_cache || !q_window || !seq_lens || !out_idx) return RKV_ERR_INVALID_ARG;
    if (!aligned16(k_cache) || !aligned16(v_cache) || !aligned16(q_window)) return RKV_ERR_INVALID_ARG;
    if ((reinterpret_cast<uintptr_t>(seq_lens) & 3u) || (reinterpret_cast<uintptr_t>(out_idx) & 3u) ||
        (reinterpret_cast<uintptr_t>(d->budgets) & 3u))
        return RKV_ERR_INVALID_ARG;
    if (!(lambda >= 0.f && lambda <= 1.f)) return RKV_ERR_INVALID_ARG;
    if ((stages & ~RKV_STAGE_ALL) != 0u || stages == 0u) return RKV_ERR_INVALID_ARG;
    if (!d->workspace || d->workspace_bytes < lay.total) return RKV_ERR_WORKSPACE;
    if (reinterpret_cast<uintptr_t>(d->workspace) & 255u) return RKV_ERR_WORKSPACE;
    if (!use_simt(d) && !scores_sm100_available()) return RKV_ERR_UNSUPPORTED;

    Params p;
    memset(&p, 0, sizeof(p));
    p.k_cache = k_cache;
    p.v_cache = v_cache;
    p.q_window = q_window;
    p.seq_lens = seq_lens;
    p.out_idx = out_idx;
    p.batch = d->batch;
    p.hkv = d->n_kv_heads;
    p.hq = d->n_q_heads;
    p.group = d->n_q_heads / d->n_kv_heads;
    p.d = d->head_dim;
    p.logit_scale = 1.0f / sqrtf((float)d->head_dim);
    p.cap = lay.cap;
    p.cap_pad = lay.cap_pad;
    p.tiles = lay.tiles;
    p.budget = budget;
    p.buffer = buffer;
    p.alpha = alpha;
    p.dtype = d->dtype;
    p.store_row_bytes = (int)(d->head_dim * cache_esz(d));
    p.pool_w = d->pool_w;
    p.beta = d->beta;
    p.mean_then_pool = (d->flags & RKV_FLAG_MEAN_THEN_POOL) ? 1 : 0;
    p.head_mean = (d->flags & RKV_FLAG_HEAD_MEAN) ? 1 : 0;
    p.gqa_mean_pool = (d->flags & RKV_FLAG_GQA_MEAN_POOL) ? 1 : 0;
    p.sim_threshold = d->sim_threshold;
    p.eps = d->eps;
    p.lambda = lambda;
    char *ws = static_cast<char *>(d->workspace);
    p.inv_norm = reinterpret_cast<float *>(ws + lay.inv_norm);
    p.norm_split = reinterpret_cast<__nv_bfloat16 *>(ws + lay.norm_split);
    p.thr_split = reinterpret_cast<__nv_bfloat16 *>(ws + lay.thr_split);
    p.tile_sum = reinterpret_cast<float *>(ws + lay.tile_sum);
    p.head_sum = reinterpret_cast<float *>(ws + lay.head_sum);
    p.logits = reinterpret_cast<float *>(ws + lay.logits);
    p.row_stat = reinterpret_cast<float *>(ws + lay.row_stat);
    p.imp = reinterpret_cast<float *>(ws + lay.imp);
    p.sbar = reinterpret_cast<float *>(ws + lay.sbar);
    p.left = reinterpret_cast<int32_t *>(ws + lay.left);
    p.strag = reinterpret_cast<int32_t *>(ws + lay.strag);
    p.strag_count = reinterpret_cast<int32_t *>(ws + lay.strag_count);
    p.strag_items = reinterpret_cast<int4 *>(ws + lay.strag_items);
    p.self_dot = reinterpret_cast<float *>(ws + lay.self_dot);
    p.best = reinterpret_cast<uint32_t *>(ws + lay.best);
    p.dense = reinterpret_cast<int32_t *>(ws + lay.dense);
    p.dense_items = reinterpret_cast<int4 *>(ws + lay.dense_items);
    p.dense_ok = (d->beta == 1 && !(d->flags & RKV_FLAG_NO_SYMMETRIC)) ? 1 : 0;
    p.head_sum_bf16 = reinterpret_cast<__nv_bfloat16 *>(ws + lay.head_sum_bf16);
    p.meta = reinterpret_cast<int32_t *>(ws + lay.meta);
    p.counters = reinterpret_cast<unsigned long long *>(ws + lay.counters);
    p.tile_done = reinterpret_cast<uint32_t *>(ws + lay.tile_done);
    p.zero_bytes = lay.zero_bytes;
    p.tri = lay.tri;
    p.status = d->device_status;
    p.budgets = d->budgets;
    p.block_table = d->block_table;
    p.pages_per_head = lay.cap / kTile;
    p.pool_pages = d->pool_pages;
    p.wait_cycles = d->wait_limit_cycles > 0 ? (long long)d->wait_limit_cycles : sm100_default_wait_cycles();
    p.kernel_events = d->kernel_events;
    p.dbg_counters = d->dbg_counters;
    p.dbg_I = d->dbg_I;
    p.dbg_Sbar = d->dbg_Sbar;
    p.dbg_R = d->dbg_R;
    p.dbg_Z = d->dbg_Z;

    cudaStream_t s = static_cast<cudaStream_t>(stream);
    void *const *ev = d->stage_events;
    cudaError_t e;
    auto mark = [&](int i) -> cudaError_t {
        return ev && ev[i] ? cudaEventRecord(static_cast<cudaEvent_t>(ev[i]), s) : cudaSuccess;
    };
    if ((e = mark(0)) != cudaSuccess) return cuda_fail(e, "cudaEventRecord");
    // What the gather moves is the caller's caches as they are stored; for 8-bit caches every stage before it reads the
    // bf16 copy of the keys (contiguous: the block table, if any, is followed once, by the widening kernel).
    Params stored = p;
    if (needs_copy(d)) {
        p.k_cache = ws + lay.k_wide;
        p.block_table = nullptr;
        p.dtype = RKV_BF16;
        p.d = scoring_dim(d);
        if (pads_dim(d)) p.q_window = ws + lay.q_wide;
        p.fuse_mode = fuse_mode(d, lay.cap);
        p.fuse_src = stored.k_cache;
        p.fuse_table = stored.block_table;
    }
    if (stages & RKV_STAGE_PREP) {
        if ((e = cudaMemsetAsync(p.counters, 0, p.zero_bytes, s)) != cudaSuccess) return cuda_fail(e, "cudaMemsetAsync");
        if (needs_copy(d) &&
            (e = launch_widen_keys(stored, static_cast<__nv_bfloat16 *>(p.k_cache), p.d, pads_dim(d) ? stored.q_window : nullptr,
                                   pads_dim(d) ? ws + lay.q_wide : nullptr, p.fuse_mode == 0, s)) != cudaSuccess)
            return cuda_fail(e, "widen launch");
        if ((e = launch_prep(p, s)) != cudaSuccess) return cuda_fail(e, "prep launch");
    }
    if ((e = mark(1)) != cudaSuccess) return cuda_fail(e, "cudaEventRecord");
    if (stages & RKV_STAGE_SCORES) {
        e = use_simt(d) ? launch_scores_simt(p, s)
                        : (p.tri ? launch_scores_tri_sm100(p, s) : launch_scores_sm100(p, s));
        if (e != cudaSuccess) return cuda_fail(e, "scores launch");
        if (!p.tri && ((e = mark_kernel(p, 0, s)) != cudaSuccess || (e = mark_kernel(p, 1, s)) != cudaSuccess))
            return cuda_fail(e, "cudaEventRecord");
        if (p.dbg_counters &&
            (e = cudaMemcpyAsync(p.dbg_counters, p.counters, 8 * sizeof(unsigned long long), cudaMemcpyDeviceToDevice, s)) !=
                cudaSuccess)
            return cuda_fail(e, "cudaMemcpyAsync");
    }
    if ((e = mark(2)) != cudaSuccess) return cuda_fail(e, "cudaEventRecord");
    if (stages & RKV_STAGE_SELECT)
        if ((e = launch_select(p, s)) != cudaSuccess) return cuda_fail(e, "select launch");
    if ((e = mark(3)) != cudaSuccess) return cuda_fail(e, "cudaEventRecord");
    if (stages & RKV_STAGE_GATHER)
        if ((e = launch_gather(stored, s)) != cudaSuccess) return cuda_fail(e, "gather launch");
    if ((e = mark(4)) != cudaSuccess) return cuda_fail(e, "cudaEventRecord");
    return RKV_OK;
}

struct HostLayout {
    size_t k, v, q, seq, idx, inner, total;
    size_t kv_bytes, q_bytes, seq_bytes, idx_bytes, row_bytes;
};

int host_layout(const rkv_desc_t *d, int budget, int buffer, int alpha, HostLayout *h)
{
    Layout lay;
    int rc = check_shapes(d, budget, buffer, alpha, &lay);
    if (rc != RKV_OK) return rc;
    const size_t P = (size_t)d->batch * d->n_kv_heads;
    h->row_bytes = (size_t)d->head_dim * cache_esz(d);
    h->kv_bytes = P * lay.cap * h->row_bytes;
    h->q_bytes = (size_t)d->batch * d->n_q_heads * alpha * d->head_dim * query_esz(d);
    h->seq_bytes = (size_t)d->batch * sizeof(int32_t);
    h->idx_bytes = P * budget * sizeof(int32_t);
    size_t off = 0;
    h->k = off;      off = align_up(off + h->kv_bytes, 256);
    h->v = off;      off = align_up(off + h->kv_bytes, 256);
    h->q = off;      off = align_up(off + h->q_bytes, 256);
    h->seq = off;    off = align_up(off + h->seq_bytes, 256);
    h->idx = off;    off = align_up(off + h->idx_bytes, 256);
    h->inner = off;  off = off + lay.total;
    h->total = off;
    return RKV_OK;
}

}  // namespace
}  // namespace rkv

using namespace rkv;

extern "C" {

void rkv_desc_default(rkv_desc_t *desc)
{
    if (!desc) return;
    memset(desc, 0, sizeof(*desc));
    desc->head_dim = kHeadDim;
    desc->dtype = RKV_BF16;
    desc->pool_w = 4;
    desc->beta = 1;
    desc->sim_threshold = 0.5f;
    desc->eps = 1e-8f;
}

size_t rkv_workspace_bytes(const rkv_desc_t *desc, int32_t budget, int32_t buffer, int32_t alpha)
{
    Layout lay;
    return check_shapes(desc, budget, buffer, alpha, &lay) == RKV_OK ? lay.total : 0;
}

int rkv_set_desc(const rkv_desc_t *desc)
{
    if (!desc) return RKV_ERR_INVALID_ARG;
    g_desc = *desc;
    g_desc_set = true;
    return RKV_OK;
}

int rkv_compress(void *k_cache, void *v_cache, const void *q_window, int32_t *seq_lens, int32_t budget,
                 int32_t buffer, int32_t alpha, float lambda, int32_t *out_idx, void *stream)
{
    if (!g_desc_set) return RKV_ERR_INVALID_ARG;
    return run(&g_desc, k_cache, v_cache, q_window, seq_lens, budget, buffer, alpha, lambda, out_idx, stream,
               RKV_STAGE_ALL);
}

int rkv_compress_ex(const rkv_desc_t *desc, void *k_cache, void *v_cache, const void *q_window,
                    int32_t *seq_lens, int32_t budget, int32_t buffer, int32_t alpha, float lambda,
                    int32_t *out_idx, void *stream)
{
    return run(desc, k_cache, v_cache, q_window, seq_lens, budget, buffer, alpha, lambda, out_idx, stream,
               RKV_STAGE_ALL);
}

int rkv_compress_stages(const rkv_desc_t *desc, void *k_cache, void *v_cache, const void *q_window,
                        int32_t *seq_lens, int32_t budget, int32_t buffer, int32_t alpha, float lambda,
                        int32_t *out_idx, void *stream, uint32_t stage_mask)
{
    return run(desc, k_cache, v_cache, q_window, seq_lens, budget, buffer, alpha, lambda, out_idx, stream,
               stage_mask);
}

size_t rkv_host_workspace_bytes(const rkv_desc_t *desc, int32_t budget, int32_t buffer, int32_t alpha)
{
    HostLayout h;
    return host_layout(desc, budget, buffer, alpha, &h) == RKV_OK ? h.total : 0;
}

int rkv_compress_host(const rkv_desc_t *desc, void *host_k_cache, void *host_v_cache, const void *host_q_window,
                      int32_t *host_seq_lens, int32_t budget, int32_t buffer, int32_t alpha, float lambda,
                      int32_t *host_out_idx, void *stream)
{
    HostLayout h;
    int rc = host_layout(desc, budget, buffer, alpha, &h);
    if (rc != RKV_OK) return rc;
    if (!host_k_cache || !host_v_cache || !host_q_window || !host_seq_lens || !host_out_idx || desc->block_table)
        return RKV_ERR_INVALID_ARG;      // (the host-buffer form takes contiguous caches only)
    if (!desc->workspace || desc->workspace_bytes < h.total) return RKV_ERR_WORKSPACE;
    if (reinterpret_cast<uintptr_t>(desc->workspace) & 255u) return RKV_ERR_WORKSPACE;
    cudaStream_t s = static_cast<cudaStream_t>(stream);
    char *ws = static_cast<char *>(desc->workspace);
    cudaError_t e;
    if ((e = cudaMemcpyAsync(ws + h.k, host_k_cache, h.kv_bytes, cudaMemcpyHostToDevice, s)) != cudaSuccess ||
        (e = cudaMemcpyAsync(ws + h.v, host_v_cache, h.kv_bytes, cudaMemcpyHostToDevice, s)) != cudaSuccess ||
        (e = cudaMemcpyAsync(ws + h.q, host_q_window, h.q_bytes, cudaMemcpyHostToDevice, s)) != cudaSuccess ||
        (e = cudaMemcpyAsync(ws + h.seq, host_seq_lens, h.seq_bytes, cudaMemcpyHostToDevice, s)) != cudaSuccess)
        return cuda_fail(e, "host to device copy");
    rkv_desc_t inner = *desc;
    inner.workspace = ws + h.inner;
    inner.workspace_bytes = desc->workspace_bytes - h.inner;
    rc = run(&inner, ws + h.k, ws + h.v, ws + h.q, reinterpret_cast<int32_t *>(ws + h.seq), budget, buffer, alpha,
             lambda, reinterpret_cast<int32_t *>(ws + h.idx), stream, RKV_STAGE_ALL);
    if (rc != RKV_OK) return rc;
    // rows [0, budget) of every head come back; rows beyond are unspecified after a compression and are left
    // as the host has them
    const size_t P = (size_t)desc->batch * desc->n_kv_heads;
    const size_t cap = (size_t)budget + buffer;
    if ((e = cudaMemcpy2DAsync(host_k_cache, cap * h.row_bytes, ws + h.k, cap * h.row_bytes, budget * h.row_bytes, P,
                               cudaMemcpyDeviceToHost, s)) != cudaSuccess ||
        (e = cudaMemcpy2DAsync(host_v_cache, cap * h.row_bytes, ws + h.v, cap * h.row_bytes, budget * h.row_bytes, P,
                               cudaMemcpyDeviceToHost, s)) != cudaSuccess ||
        (e = cudaMemcpyAsync(host_seq_lens, ws + h.seq, h.seq_bytes, cudaMemcpyDeviceToHost, s)) != cudaSuccess ||
        (e = cudaMemcpyAsync(host_out_idx, ws + h.idx, h.idx_bytes, cudaMemcpyDeviceToHost, s)) != cudaSuccess)
        return cuda_fail(e, "device to host copy");
    return RKV_OK;
}

int rkv_append(const rkv_desc_t *d, void *k_cache, void *v_cache, const void *k_new, const void *v_new, int32_t *seq_lens,
               int32_t budget, int32_t buffer, void *stream)
{
    // shape checks as for the compression (alpha plays no part here: any valid value)
    int rc = check_shapes(d, budget, buffer, 1, nullptr);
    if (rc != RKV_OK) return rc;
    if (!k_cache || !v_cache || !k_new || !v_new || !seq_lens) return RKV_ERR_INVALID_ARG;
    if (!aligned16(k_cache) || !aligned16(v_cache) || !aligned16(k_new) || !aligned16(v_new)) return RKV_ERR_INVALID_ARG;
    if (reinterpret_cast<uintptr_t>(seq_lens) & 3u) return RKV_ERR_INVALID_ARG;
    const int row_bytes = (int)(d->head_dim * cache_esz(d));
    const cudaError_t e = launch_append(k_cache, v_cache, k_new, v_new, seq_lens, d->batch, d->n_kv_heads, budget + buffer,
                                        row_bytes, d->device_status, d->block_table, static_cast<cudaStream_t>(stream));
    return e == cudaSuccess ? RKV_OK : cuda_fail(e, "append launch");
}

int rkv_push_query(const rkv_desc_t *d, void *q_window, const void *q_new, int32_t alpha, int32_t slot, void *stream)
{
    if (!d || alpha < 1 || slot < 0 || slot >= alpha) return RKV_ERR_INVALID_ARG;
    int rc = check_shapes(d, alpha + 1, 1, alpha, nullptr);        // descriptor fields and alpha against the group limit
    if (rc != RKV_OK) return rc;
    if (!q_window || !q_new || !aligned16(q_window) || !aligned16(q_new)) return RKV_ERR_INVALID_ARG;
    const int row_bytes = (int)(d->head_dim * query_esz(d));
    const cudaError_t e = launch_push_query(q_window, q_new, d->batch, d->n_q_heads, alpha, slot, row_bytes,
                                            static_cast<cudaStream_t>(stream));
    return e == cudaSuccess ? RKV_OK : cuda_fail(e, "push_query launch");
}

static int attend_plan(const rkv_desc_t *d, int32_t budget, int32_t buffer, int *splits, size_t *bytes)
{
    int rc = check_shapes(d, budget, buffer, 1, nullptr);
    if (rc != RKV_OK) return rc;
    const int G = d->n_q_heads / d->n_kv_heads;
    if (!attend_supported(G, d->dtype, d->head_dim)) return RKV_ERR_UNSUPPORTED;
    int dev = 0, sms = 0;
    if (cudaGetDevice(&dev) != cudaSuccess || cudaDeviceGetAttribute(&sms, cudaDevAttrMultiProcessorCount, dev) != cudaSuccess)
        sms = 148;       // sizing only (no device here): the B200's count
    *splits = attend_splits(d->batch * d->n_kv_heads, budget + buffer, sms, G, d->dtype);
    *bytes = attend_partial_bytes(d->batch * d->n_kv_heads, *splits, G);
    return RKV_OK;
}

size_t rkv_decode_workspace_bytes(const rkv_desc_t *desc, int32_t budget, int32_t buffer)
{
    int splits = 1;
    size_t bytes = 0;
    return attend_plan(desc, budget, buffer, &splits, &bytes) == RKV_OK ? bytes : 0;
}

int rkv_decode_attention(const rkv_desc_t *d, const void *k_cache, const void *v_cache, const void *q_new,
                         const int32_t *seq_lens, float *out, int32_t budget, int32_t buffer, void *stream)
{
    int splits = 1;
    size_t bytes = 0;
    int rc = attend_plan(d, budget, buffer, &splits, &bytes);
    if (rc != RKV_OK) return rc;
    if (!k_cache || !v_cache || !q_new || !seq_lens || !out) return RKV_ERR_INVALID_ARG;
    if (!aligned16(k_cache) || !aligned16(v_cache) || !aligned16(q_new) || !aligned16(out)) return RKV_ERR_INVALID_ARG;
    if (reinterpret_cast<uintptr_t>(seq_lens) & 3u) return RKV_ERR_INVALID_ARG;
    if (bytes > 0) {
        if (!d->workspace || d->workspace_bytes < bytes) return RKV_ERR_WORKSPACE;
        if (reinterpret_cast<uintptr_t>(d->workspace) & 255u) return RKV_ERR_WORKSPACE;
    }
    const long long wait = d->wait_limit_cycles > 0 ? (long long)d->wait_limit_cycles : sm100_default_wait_cycles();
    const cudaError_t e = launch_attend(k_cache, v_cache, q_new, seq_lens, out, static_cast<float *>(d->workspace), d->batch,
                                        d->n_kv_heads, d->n_q_heads, budget + buffer, splits, d->dtype, d->device_status,
                                        wait, d->block_table, d->pool_pages, d->head_dim, static_cast<cudaStream_t>(stream));
    return e == cudaSuccess ? RKV_OK : cuda_fail(e, "decode attention launch");
}

int rkv_launch_count(const rkv_desc_t *desc, uint32_t stage_mask)
{
    int c = 0;
    for (uint32_t bit = 1; bit <= RKV_STAGE_GATHER; bit <<= 1) c += (stage_mask & bit) ? 1 : 0;
    if (stage_mask & RKV_STAGE_SELECT) c += 2;      // row statistics and importance run ahead of the selection kernel
    // bf16 keys of 128 dimensions: the tile sums are added up per head by a kernel of its own behind the prep kernel
    if (desc && (stage_mask & RKV_STAGE_PREP) && desc->dtype != RKV_F32 && (desc->head_dim == 0 || scoring_dim(desc) == kHeadDim)) c += 1;
    if (desc && (stage_mask & RKV_STAGE_PREP) && needs_copy(desc)) c += 1;       // the kernel that writes the scoring copy
    if (desc && (stage_mask & RKV_STAGE_SELECT) && (desc->flags & RKV_FLAG_HEAD_MEAN)) c += 1;   // per-sequence selection
    // the two-pass scoring path is the first pass plus up to two rounds of (listing, second pass) while the
    // retention rule is on
    if (desc && (stage_mask & RKV_STAGE_SCORES) && use_tri(desc) && desc->beta > 0 && desc->sim_threshold < 1.0f) {
        c += 4;
        if (desc->beta == 1 && !(desc->flags & RKV_FLAG_NO_SYMMETRIC)) c += 2;      // symmetric route: scan and finish
    }
    return c;
}

int rkv_launch_count_for(const rkv_desc_t *desc, int32_t budget, int32_t buffer, int32_t alpha, uint32_t stage_mask)
{
    Layout lay;
    if (check_shapes(desc, budget, buffer, alpha, &lay) != RKV_OK) return 0;
    int c = rkv_launch_count(desc, stage_mask);
    // the prep kernel writes the copy of the keys itself and nothing else needs a pass of its own
    if ((stage_mask & RKV_STAGE_PREP) && fuse_mode(desc, lay.cap) != 0 && !pads_dim(desc)) c -= 1;
    if ((stage_mask & RKV_STAGE_SELECT) && select_is_fused(lay.cap_pad, alpha)) c -= 2;
    if ((stage_mask & RKV_STAGE_SCORES) && use_tri(desc) && desc->beta > 0 && desc->sim_threshold < 1.0f)
    {
        c -= lay.tiles < 2 ? 4                                      // one key tile: the first scoring pass has seen everything
                           : 2 * (2 - scores_pass2_rounds(lay.tiles));   // small caches take one round
        if (desc->beta == 1 && !(desc->flags & RKV_FLAG_NO_SYMMETRIC) && !scores_dense_possible(lay.tiles, desc->beta)) c -= 2;
    }
    return c;
}

const char *rkv_status_string(int status)
{
    switch (status) {
        case RKV_OK: return "RKV_OK";
        case RKV_ERR_INVALID_ARG: return "RKV_ERR_INVALID_ARG";
        case RKV_ERR_UNSUPPORTED: return "RKV_ERR_UNSUPPORTED";
        case RKV_ERR_WORKSPACE: return "RKV_ERR_WORKSPACE";
        case RKV_ERR_CUDA: return "RKV_ERR_CUDA";
        case RKV_ERR_TIMEOUT: return "RKV_ERR_TIMEOUT";
        default: return "RKV_ERR_UNKNOWN";
    }
}

const char *rkv_last_cuda_error(void) { return g_cuda_error; }

}  // extern "C"

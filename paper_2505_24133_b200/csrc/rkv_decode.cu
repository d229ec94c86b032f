// The two cache updates of a decode step that surround the compression (Section 3.1: newly generated tokens enter the
// buffer part of the cache; Algorithm 1's observation buffer M_alpha holds the last alpha queries).  Plain byte
// movement, one 16-byte vector per thread.
#include "rkv_common.cuh"

namespace rkv {

namespace {

constexpr int kDecThreads = 256;

// k_new / v_new [batch][hkv][row_vecs] -> row seq_lens[b] of every head of sequence b
__global__ void __launch_bounds__(kDecThreads) append_kernel(uint4 *k_cache, uint4 *v_cache, const uint4 *k_new,
                                                             const uint4 *v_new, const int32_t *seq_lens, long long total,
                                                             int hkv, int cap, int row_vecs, int32_t *status,
                                                             const int32_t *block_table)
{
    const long long t = (long long)blockIdx.x * kDecThreads + threadIdx.x;
    if (t >= total) return;
    const int vec = (int)(t % row_vecs);
    const int head = (int)(t / row_vecs);          // b * hkv + h
    const int L = seq_lens[head / hkv];
    if (L >= 0 && L < cap) {
        // row L of the head: head after head, or through the block table (pages of kTile rows) for paged caches
        const size_t row = block_table ? (size_t)block_table[(size_t)head * (cap / kTile) + L / kTile] * kTile + L % kTile
                                       : (size_t)head * cap + L;
        const size_t dst = row * row_vecs + vec;
        k_cache[dst] = k_new[t];
        v_cache[dst] = v_new[t];
    } else if (vec == 0 && head % hkv == 0) {
        report(status, RKV_ERR_INVALID_ARG);        // the cache of this sequence is full (or its length invalid)
    }
}

// seq_lens[b] += 1 for the sequences that took the new token (a launch of its own: every copy above has read the
// old length by then)
__global__ void __launch_bounds__(kDecThreads) bump_kernel(int32_t *seq_lens, int batch, int cap)
{
    const int b = blockIdx.x * kDecThreads + threadIdx.x;
    if (b >= batch) return;
    const int L = seq_lens[b];
    if (L >= 0 && L < cap) seq_lens[b] = L + 1;
}

// q_new [batch][hq][row_vecs] -> row `slot` of every query head's window [batch][hq][alpha][row_vecs]
__global__ void __launch_bounds__(kDecThreads) push_query_kernel(uint4 *q_window, const uint4 *q_new, long long total,
                                                                 int alpha, int slot, int row_vecs)
{
    const long long t = (long long)blockIdx.x * kDecThreads + threadIdx.x;
    if (t >= total) return;
    const int vec = (int)(t % row_vecs);
    const long long qh = t / row_vecs;                  // b * hq + query head
    q_window[((size_t)qh * alpha + slot) * row_vecs + vec] = q_new[t];
}

}  // namespace

cudaError_t launch_append(void *k_cache, void *v_cache, const void *k_new, const void *v_new, int32_t *seq_lens, int batch,
                          int hkv, int cap, int row_bytes, int32_t *status, const int32_t *block_table, cudaStream_t s)
{
    const int row_vecs = row_bytes / 16;
    const long long total = (long long)batch * hkv * row_vecs;
    const unsigned grid = (unsigned)((total + kDecThreads - 1) / kDecThreads);
    append_kernel<<<grid, kDecThreads, 0, s>>>(static_cast<uint4 *>(k_cache), static_cast<uint4 *>(v_cache),
                                               static_cast<const uint4 *>(k_new), static_cast<const uint4 *>(v_new),
                                               seq_lens, total, hkv, cap, row_vecs, status, block_table);
    cudaError_t e = cudaGetLastError();
    if (e != cudaSuccess) return e;
    bump_kernel<<<(unsigned)((batch + kDecThreads - 1) / kDecThreads), kDecThreads, 0, s>>>(seq_lens, batch, cap);
    return cudaGetLastError();
}

cudaError_t launch_push_query(void *q_window, const void *q_new, int batch, int hq, int alpha, int slot, int row_bytes,
                              cudaStream_t s)
{
    const int row_vecs = row_bytes / 16;
    const long long total = (long long)batch * hq * row_vecs;
    const unsigned grid = (unsigned)((total + kDecThreads - 1) / kDecThreads);
    push_query_kernel<<<grid, kDecThreads, 0, s>>>(static_cast<uint4 *>(q_window), static_cast<const uint4 *>(q_new), total,
                                                   alpha, slot, row_vecs);
    return cudaGetLastError();
}

}  // namespace rkv

// Stage "gather": Algorithm 1's gather + concatenate, done in place.
//
// For every head, row j of K and of V becomes row idx[j] (j < budget).  idx is strictly ascending, so
// idx[j] >= j: rows only move towards lower positions and the untouched prefix (idx[j] == j) is free.
// One thread block owns one (head, K|V) stream (or a column slice of it) and walks it in chunks of 64 rows or more: load the chunk's source
// rows into registers, barrier, store.  A later chunk reads only rows at or beyond its own first row, which
// no earlier chunk writes, so one barrier per chunk is all the ordering in-place compaction needs.
// No scratch copy, no reallocation.  HBM-bound: 16-byte loads and stores, a row is 4 (8-bit, d = 64) to 64 (fp32, d = 256) lanes wide.
// The block of (KV head 0, K) also stores the new length, seq_lens[b] = budget.
#include "rkv_common.cuh"

namespace rkv {

namespace {

constexpr int kGatherThreads = 256;
constexpr int kChunkRows = 64;

// kVecPerRow: 16-byte vectors per row; kSplit: column slices a row is cut into, each moved by a block of its own
// (slices are disjoint bytes, so they need no ordering among themselves; small batches need the extra blocks to
// keep enough bytes in flight).
template <int kVecPerRow, int kSplit>
__global__ void __launch_bounds__(kGatherThreads) gather_kernel(Params p)
{
    constexpr int kVecPerSlice = kVecPerRow / kSplit;                           // vectors of a row this block moves
    constexpr int kRows = kChunkRows * kSplit;                                  // rows per chunk: 16 KB in flight per block
    constexpr int kVecPerThread = kRows * kVecPerSlice / kGatherThreads;       // 4 or 8
    constexpr int kRowsPerStep = kGatherThreads / kVecPerSlice;
    const int slice = blockIdx.x % kSplit;
    const int stream = blockIdx.x / kSplit;
    const int head = stream >> 1;
    const int which = stream & 1;
    const int b = head / p.hkv;
    const int L = p.meta[b];
    const int budget_b = seq_budget(p, b);
    if (L <= budget_b) return;                      // nothing was selected for this sequence
    if (call_aborted(p)) return;                    // a bounded wait ran out earlier in this call: caches and lengths stay as they are
    if (which == 0 && slice == 0 && head % p.hkv == 0 && threadIdx.x == 0) p.seq_lens[b] = budget_b;

    // rows are addressed through row_index(): head after head, or page by page for paged caches
    uint4 *base = reinterpret_cast<uint4 *>(which ? p.v_cache : p.k_cache) + slice * kVecPerSlice;
    const int32_t *idx = p.out_idx + (size_t)head * p.budget;
    const int lane_vec = threadIdx.x % kVecPerSlice;
    const int lane_row = threadIdx.x / kVecPerSlice;

    for (int j0 = 0; j0 < budget_b; j0 += kRows) {
        const int j_end = min(j0 + kRows, budget_b);
        if (idx[j_end - 1] == j_end - 1) continue;   // ascending and idx[j] >= j: the whole chunk is in place
        uint4 held[kVecPerThread];
        int src[kVecPerThread];
#pragma unroll
        for (int q = 0; q < kVecPerThread; ++q) {
            const int j = j0 + q * kRowsPerStep + lane_row;
            src[q] = (j < j_end) ? idx[j] : -1;
            if (src[q] >= 0 && src[q] != j) held[q] = base[(size_t)row_index(p, head, src[q]) * kVecPerRow + lane_vec];
        }
        __syncthreads();                             // every source row of the chunk is in registers
#pragma unroll
        for (int q = 0; q < kVecPerThread; ++q) {
            const int j = j0 + q * kRowsPerStep + lane_row;
            if (src[q] >= 0 && src[q] != j) base[(size_t)row_index(p, head, j) * kVecPerRow + lane_vec] = held[q];
        }
    }
}

}  // namespace

cudaError_t launch_gather(const Params &p, cudaStream_t s)
{
    const unsigned streams = 2u * (unsigned)(p.batch * p.hkv);
    int dev = 0, sms = 0;
    cudaError_t e;
    if ((e = cudaGetDevice(&dev)) != cudaSuccess) return e;
    if ((e = cudaDeviceGetAttribute(&sms, cudaDevAttrMultiProcessorCount, dev)) != cudaSuccess) return e;
    // Few streams: cut the rows into column slices, as many (4, 2) as still fit the SMs in one wave of resident blocks
    // (8 per SM): a second, partly filled wave would leave SMs idle for much of the kernel.
    const unsigned wave = 8u * (unsigned)sms;
    const int split = streams * 4u <= wave ? 4 : (streams * 2u <= wave ? 2 : (streams < wave ? 4 : 1));
    const int vec_per_row = p.store_row_bytes / 16;      // 16-byte vectors per row: 4 .. 64
#define RKV_GATHER_CASE(V)                                                                      \
    case V:                                                                                     \
        if (split == 4) gather_kernel<V, 4><<<streams * 4u, kGatherThreads, 0, s>>>(p);         \
        else if (split == 2) gather_kernel<V, 2><<<streams * 2u, kGatherThreads, 0, s>>>(p);    \
        else gather_kernel<V, 1><<<streams, kGatherThreads, 0, s>>>(p);                         \
        break;
    switch (vec_per_row) {
        RKV_GATHER_CASE(4)
        RKV_GATHER_CASE(8)
        RKV_GATHER_CASE(16)
        RKV_GATHER_CASE(32)
        RKV_GATHER_CASE(64)
        default: return cudaErrorInvalidValue;
    }
#undef RKV_GATHER_CASE
    return cudaGetLastError();
}

}  // namespace rkv

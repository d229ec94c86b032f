// The scoring copy of the keys, ahead of the prep stage: 8-bit caches widened to bf16, and / or a head dimension of 64
// padded with zeros to the 128 the tensor-core kernels are built for (dot products and norms do not see the zeros; the
// observation queries are padded alongside).
//
// An 8-bit cache holds E4M3 codes (1 sign, 4 exponent bits with bias 7, 3 mantissa bits; no infinities).  Eq. 1-7 are
// defined on the values the codes stand for, and every such value is a bf16 value, so the scoring stages run unchanged
// (bf16 tensor-core products, fp32 accumulation) on a widened copy of the keys; the values never change, the gather
// moves the stored bytes.  The copy is contiguous, head after head with `cap` rows each, whatever the layout of the
// cache (a block table is followed here, once).  Rows at or beyond a sequence's length are written as zeros, so the
// stages that read whole 128-row tiles meet no stale bit patterns.
//
// HBM-bound: 1 byte read and 2 written per element, 16 elements per thread and step.
#include "rkv_common.cuh"

namespace rkv {

namespace {

constexpr int kWidenThreads = 256;

// Block x < tiles * head-problems: 128-row tile x % tiles of head-problem x / tiles.  src_vecs: 16-byte vectors of a
// stored row; dst_vecs: of a row of the copy (bf16; wider than the widened row when the head dimension is padded: the
// rest of the row is zeros).  The blocks after those pad the observation queries the same way (bf16 rows only).
__global__ void __launch_bounds__(kWidenThreads)
widen_keys_kernel(Params p, int key_blocks, __nv_bfloat16 *wide, int src_vecs, int dst_vecs, int codes, const uint4 *q_src, uint4 *q_dst,
                  int q_rows)
{
    if ((int)blockIdx.x >= key_blocks) {
        // queries: rows of src_q_vecs = dst_vecs / 2 vectors (bf16, 64 dimensions) -> rows of dst_vecs, zero-padded
        const int q_vecs = dst_vecs / 2;
        const int row0 = ((int)blockIdx.x - key_blocks) * kTile;
        for (int x = threadIdx.x; x < kTile * dst_vecs; x += kWidenThreads) {
            const int r = row0 + x / dst_vecs, c = x % dst_vecs;
            if (r < q_rows) q_dst[(size_t)r * dst_vecs + c] = c < q_vecs ? __ldg(q_src + (size_t)r * q_vecs + c) : make_uint4(0u, 0u, 0u, 0u);
        }
        return;
    }
    const int tile = blockIdx.x % p.tiles;
    const int head = blockIdx.x / p.tiles;
    const int b = head / p.hkv;
    const int L = p.seq_lens[b];
    const int valid = (L < 0 || L > p.cap) ? 0 : L;            // an invalid length is reported by the prep stage
    const bool last_head = head == p.batch * p.hkv - 1;
    // rows of this head end at cap; the last head also owns the zero rows up to the end of its last tile
    const int row_end = min((tile + 1) * kTile, last_head ? p.cap_pad : p.cap);
    const uint4 *src = static_cast<const uint4 *>(p.k_cache);
    uint4 *dst = reinterpret_cast<uint4 *>(wide);
    const int out_per_src = codes ? 2 : 1;                     // vectors a stored vector becomes
    const int slots = dst_vecs / out_per_src;                  // work units per row (those past src_vecs write zeros)
    const int units = (row_end - tile * kTile) * slots;
    for (int x = threadIdx.x; x < units; x += kWidenThreads) {
        const int r = tile * kTile + x / slots, c = x % slots;
        uint4 lo = make_uint4(0u, 0u, 0u, 0u), hi = lo;
        if (r < valid && c < src_vecs) {
            const uint4 v = __ldg(src + (size_t)row_index(p, head, r) * src_vecs + c);
            if (codes) widen16(v, &lo, &hi);
            else lo = v;
        }
        uint4 *out = dst + ((size_t)head * p.cap + r) * dst_vecs + out_per_src * c;
        out[0] = lo;
        if (codes) out[1] = hi;
    }
}

}  // namespace

// stored: the caches as the caller holds them (d = stored head dimension).  wide_d: head dimension of the copy.
// q_src / q_dst: the observation queries and their padded copy (null when the head dimension is not padded).
// keys = false: the queries only (the prep stage writes the copy of the keys itself).
cudaError_t launch_widen_keys(const Params &stored, __nv_bfloat16 *wide, int wide_d, const void *q_src, void *q_dst,
                              bool keys, cudaStream_t s)
{
    const int codes = stored.dtype == RKV_FP8_E4M3 ? 1 : 0;
    const int q_rows = q_dst ? stored.batch * stored.hq * stored.alpha : 0;
    const unsigned key_blocks = keys ? (unsigned)stored.tiles * (unsigned)(stored.batch * stored.hkv) : 0u;
    const unsigned grid = key_blocks + (unsigned)((q_rows + kTile - 1) / kTile);
    if (grid == 0u) return cudaSuccess;
    widen_keys_kernel<<<grid, kWidenThreads, 0, s>>>(stored, (int)key_blocks, wide, stored.store_row_bytes / 16, wide_d * 2 / 16, codes,
                                                     static_cast<const uint4 *>(q_src), static_cast<uint4 *>(q_dst), q_rows);
    return cudaGetLastError();
}

}  // namespace rkv

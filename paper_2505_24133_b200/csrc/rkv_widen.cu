// 8-bit caches: the keys of every head-problem widened to bf16 in the workspace, ahead of the prep stage.
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

// Block x: 128-row tile x % tiles of head-problem x / tiles.  vec_per_row = d / 16 (16-byte vectors of a stored row).
__global__ void __launch_bounds__(kWidenThreads) widen_keys_kernel(Params p, __nv_bfloat16 *wide, int vec_per_row)
{
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
    const int vecs = (row_end - tile * kTile) * vec_per_row;
    for (int x = threadIdx.x; x < vecs; x += kWidenThreads) {
        const int r = tile * kTile + x / vec_per_row, c = x % vec_per_row;
        uint4 lo = make_uint4(0u, 0u, 0u, 0u), hi = lo;
        if (r < valid) widen16(__ldg(src + (size_t)row_index(p, head, r) * vec_per_row + c), &lo, &hi);
        uint4 *out = dst + ((size_t)head * p.cap + r) * (2 * vec_per_row) + 2 * c;
        out[0] = lo;
        out[1] = hi;
    }
}

}  // namespace

cudaError_t launch_widen_keys(const Params &stored, __nv_bfloat16 *wide, cudaStream_t s)
{
    const unsigned grid = (unsigned)stored.tiles * (unsigned)(stored.batch * stored.hkv);
    widen_keys_kernel<<<grid, kWidenThreads, 0, s>>>(stored, wide, stored.d / 16);
    return cudaGetLastError();
}

}  // namespace rkv

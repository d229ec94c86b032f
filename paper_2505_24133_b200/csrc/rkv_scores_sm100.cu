// Stage "scores", tensor-core version for bf16 caches: tcgen05.mma with TMEM accumulators, fed by TMA.
//
// Work items per head-problem (blockIdx.x = head * (row_blocks + 1) + x):
//
//   x < row_blocks   rows [256 x, 256 x + 256) of Eq. 5's similarity matrix.  The block keeps its 256 key rows
//                    resident in shared memory as two 128-row operand tiles and streams every 128-key tile J of
//                    the head through a TMA ring, from the last tile to the first.  Each J tile costs two
//                    M128 x N128 x K128 products into two TMEM accumulators (raw bf16 keys; exact products,
//                    fp32 accumulation).  Eight epilogue warps, one thread per matrix row, read the accumulators
//                    back, scale by r_j (and compare against T / r_i) in fp32 and apply Section 3.3's retention
//                    rule: scanning j downwards, the first beta entries with S[j][i] > T are summed up as
//                    "removed".  The plain column sum of Eq. 6 needs no per-element work: it is
//                    Kbar_i . (sum_j Kbar_j) - Kbar_i . Kbar_i, taken from the prep stage's tile sums.
//                    Result: sbar[i] = (sum_j S[j][i] - removed_i) / n.  The n x n matrix never leaves TMEM.
//
//   x == row_blocks  Eq. 2-3 for the head's query group: the same ring streams the key tiles as the M operand
//                    against the resident G*alpha query rows (N operand), so every thread ends up with all
//                    G*alpha logits of one key and takes the max over the group locally.
//
// Warp roles (320 threads): warp 0 = TMA producer, warp 1 = MMA issuer and TMEM owner, warps 2..9 = epilogue
// (warp w may touch TMEM lanes 32 (w % 4) .. +31; warps 2-5 serve accumulator half 0, warps 6-9 half 1).
// Every wait on an mbarrier is bounded; on expiry the block records RKV_ERR_TIMEOUT, stops issuing work,
// and leaves through the common exit that frees TMEM.
// No TMA multicast and no cluster launch: each block fetches its own tiles; a head's keys stay L2-resident
// while its blocks run side by side.
#include "rkv_sm100.cuh"

namespace rkv {

namespace {

using namespace sm100;

constexpr int kThreads = 320;
constexpr int kStages = 3;                       // ring depth of streamed key tiles
constexpr int kHalfBytes = kTile * 64 * 2;       // one TMA box: 128 rows x 64 bf16 (128-byte swizzled rows)
constexpr int kTileBytes = 2 * kHalfBytes;       // 32 KB: a 128 x 128 bf16 operand tile
constexpr int kRowsPerBlock = 2 * kTile;         // 256 matrix rows per row block
constexpr uint32_t kTmemCols = 512;

// shared memory carve-up (offsets from a 1024-byte aligned base)
constexpr int kOffB = 0;                                   // kStages streamed key tiles
constexpr int kOffA = kOffB + kStages * kTileBytes;        // 2 resident tiles (row blocks) / the query tile
constexpr int kOffR = kOffA + 2 * kTileBytes;              // inverse norms of the head, up to RKV_MAX_CAP floats
constexpr int kOffS = kOffR + RKV_MAX_CAP * 4;             // sum_j Kbar_j, 128 floats
constexpr int kOffBar = kOffS + kHeadDim * 4;              // mbarriers
constexpr int kNumBars = 2 * kStages + 4 + 1;
constexpr int kOffMisc = kOffBar + kNumBars * 8;           // tmem base, abort flag
constexpr int kSmemBytes = kOffMisc + 16 + 1024;           // + slack for the manual 1024-byte alignment
// The query block stages up to 128 x 128 fp32 logits in the second resident tile and the norm vector behind it
// (neither is used there): 64 KB, contiguous.
constexpr int kOffStage = kOffA + kTileBytes;
static_assert(kOffStage + RKV_MAX_GROUP_ROWS * kTile * 4 <= kOffS, "logit staging must fit");
static_assert(kSmemBytes <= 227 * 1024, "shared memory budget");

__device__ __forceinline__ void epi_barrier() { asm volatile("bar.sync 1, 256;" ::: "memory"); }

// mbarrier addresses (8 bytes each, from bar0): full[kStages], empty[kStages], acc_full[2], acc_empty[2], resident
struct Barriers {
    uint32_t bar0;
    __device__ __forceinline__ uint32_t full(int s) const { return bar0 + 8 * s; }
    __device__ __forceinline__ uint32_t empty(int s) const { return bar0 + 8 * (kStages + s); }
    __device__ __forceinline__ uint32_t acc_full(int a) const { return bar0 + 8 * (2 * kStages + a); }
    __device__ __forceinline__ uint32_t acc_empty(int a) const { return bar0 + 8 * (2 * kStages + 2 + a); }
    __device__ __forceinline__ uint32_t resident() const { return bar0 + 8 * (2 * kStages + 4); }
};

__global__ void __launch_bounds__(kThreads, 1)
scores_sm100_kernel(Params p, const __grid_constant__ CUtensorMap map_k, const __grid_constant__ CUtensorMap map_q,
                    int row_blocks, int q_rows_pad)
{
    extern __shared__ uint8_t smem_raw[];
    uint8_t *smem = reinterpret_cast<uint8_t *>((reinterpret_cast<uintptr_t>(smem_raw) + 1023) & ~(uintptr_t)1023);
    const uint32_t sbase = smem_u32(smem);
    float *r_s = reinterpret_cast<float *>(smem + kOffR);
    float *sum_s = reinterpret_cast<float *>(smem + kOffS);
    uint32_t *tmem_holder = reinterpret_cast<uint32_t *>(smem + kOffMisc);
    volatile int *abort_flag = reinterpret_cast<volatile int *>(smem + kOffMisc + 4);

    const Barriers bar{sbase + kOffBar};

    // Once any block has recorded an error (a wait that ran out), the blocks still to run return at once
    // instead of each waiting out its own limit.
    __shared__ int bail;
    const ErrSink sink = make_sink(p);
    if (threadIdx.x == 0) bail = call_aborted(p) ? 1 : 0;      // a wait of this call has run out: nothing more is started
    __syncthreads();
    if (bail) return;

    const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
    const int items = row_blocks + 1;
    const int head = blockIdx.x / items;
    const int x = blockIdx.x % items;
    const int b = head / p.hkv, h = head % p.hkv;
    const int n = seq_candidates(p, b);
    const bool is_q = (x == row_blocks);
    const int row0 = x * kRowsPerBlock;
    if (n == 0 || (!is_q && row0 >= n)) return;            // uniform for the block; nothing allocated yet

    const int n_tiles = (n + kTile - 1) / kTile;
    const bool rule_on = p.beta > 0 && p.sim_threshold < 1.0f;
    const int n_iter = is_q ? n_tiles : (rule_on ? n_tiles : 0);   // streamed tiles
    const int num_m = is_q ? 1 : ((n - row0 > kTile) ? 2 : 1);     // accumulator halves in use

    if (threadIdx.x == 0) {
        for (int s = 0; s < kStages; ++s) {
            mbar_init(bar.full(s), 1);
            mbar_init(bar.empty(s), 1);
        }
        for (int a = 0; a < 2; ++a) {
            mbar_init(bar.acc_full(a), 1);
            mbar_init(bar.acc_empty(a), 4 * num_m);
        }
        mbar_init(bar.resident(), 1);
        *abort_flag = 0;
        asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory");
    }
    if (warp == 1) {
        asm volatile("tcgen05.alloc.cta_group::1.sync.aligned.shared::cta.b32 [%0], %1;"
                     ::"r"(smem_u32(tmem_holder)), "r"(kTmemCols) : "memory");
        asm volatile("tcgen05.relinquish_alloc_permit.cta_group::1.sync.aligned;" ::: "memory");
    }
    tc_fence_before();
    __syncthreads();
    tc_fence_after();
    const uint32_t tmem_base = *tmem_holder;

    if (warp == 0) {
        // ------------------------------------------------------------------ TMA producer
        if (lane == 0) {
            if (is_q) {
                const int q_row = (b * p.hq + h * p.group) * p.alpha;
                mbar_expect_tx(bar.resident(), (uint32_t)(2 * q_rows_pad * 128));
                tma_load_2d(sbase + kOffA, &map_q, 0, q_row, bar.resident());
                tma_load_2d(sbase + kOffA + kHalfBytes, &map_q, 64, q_row, bar.resident());
            } else {
                mbar_expect_tx(bar.resident(), (uint32_t)(num_m * kTileBytes));
                for (int m = 0; m < num_m; ++m) {
                    const int y = (int)tile_row0(p, head, row0 / kTile + m);
                    tma_load_2d(sbase + kOffA + m * kTileBytes, &map_k, 0, y, bar.resident());
                    tma_load_2d(sbase + kOffA + m * kTileBytes + kHalfBytes, &map_k, 64, y, bar.resident());
                }
            }
            for (int t = 0; t < n_iter; ++t) {
                const int s = t % kStages;
                const int jt = n_tiles - 1 - t;                       // last tile first
                if (!mbar_wait(bar.empty(s), ((t / kStages) & 1) ^ 1, abort_flag, sink)) break;
                mbar_expect_tx(bar.full(s), kTileBytes);
                const uint32_t dst = sbase + kOffB + s * kTileBytes;
                const int y = (int)tile_row0(p, head, jt);
                tma_load_2d(dst, &map_k, 0, y, bar.full(s));
                tma_load_2d(dst + kHalfBytes, &map_k, 64, y, bar.full(s));
            }
        }
    } else if (warp == 1) {
        // ------------------------------------------------------------------ MMA issuer
        if (lane == 0) {
            const uint32_t idesc = is_q ? instr_desc(kTile, q_rows_pad) : instr_desc(kTile, kTile);
            bool ok = mbar_wait(bar.resident(), 0, abort_flag, sink);
            for (int t = 0; ok && t < n_iter; ++t) {
                const int s = t % kStages, a = t & 1;
                if (!mbar_wait(bar.full(s), (t / kStages) & 1, abort_flag, sink)) break;
                if (!mbar_wait(bar.acc_empty(a), ((t >> 1) & 1) ^ 1, abort_flag, sink)) break;
                tc_fence_after();
                const uint32_t stage = sbase + kOffB + s * kTileBytes;
                for (int m = 0; m < num_m; ++m) {
                    const uint32_t resident = sbase + kOffA + m * kTileBytes;
                    const uint32_t d_tmem = tmem_base + a * 256 + m * 128;
#pragma unroll
                    for (int k = 0; k < 8; ++k) {
                        // K = 16 per instruction: 32 bytes along the swizzled row; k >= 4 is the second box
                        const uint32_t koff = (k >> 2) * kHalfBytes + (k & 3) * 32;
                        const uint64_t da = smem_desc((is_q ? stage : resident) + koff);
                        const uint64_t db = smem_desc((is_q ? resident : stage) + koff);
                        umma(d_tmem, da, db, idesc, k > 0);
                    }
                }
                umma_commit(bar.empty(s));       // the stage may be refilled once these MMAs have read it
                umma_commit(bar.acc_full(a));    // the accumulators are complete
            }
        }
        __syncwarp();
    } else {
        // ------------------------------------------------------------------ epilogue warps
        const int ew = warp - 2;                 // 0..7
        const int half = ew >> 2;                // accumulator half (row tile) this warp serves
        const int quad = warp & 3;               // TMEM lane quadrant this warp may access
        const int et = threadIdx.x - 64;         // 0..255
        const bool warp_active = half < num_m;
        const int lrow = quad * 32 + lane;       // row within the 128-row tile
        const uint32_t lane_base = tmem_base + ((uint32_t)(quad * 32) << 16);

        if (!is_q) {
            // inverse norms of the whole head and sum_j Kbar_j into shared memory
            const float *inv_norm = p.inv_norm + (size_t)head * p.cap_pad;
            for (int v = et; v < n_tiles * (kTile / 4); v += 256)
                reinterpret_cast<float4 *>(r_s)[v] = __ldg(reinterpret_cast<const float4 *>(inv_norm) + v);
            if (et < kHeadDim) sum_s[et] = p.head_sum[(size_t)head * kHeadDim + et];
            epi_barrier();

            const int i = row0 + half * kTile + lrow;
            const bool row_ok = warp_active && i < n;
            const float ri = row_ok ? r_s[i] : 0.f;
            float total = 0.f;
            bool ok = mbar_wait(bar.resident(), 0, abort_flag, sink);
            if (ok && warp_active) {
                // Kbar_i . s - Kbar_i . Kbar_i from the resident (swizzled) tile: 16-byte chunk c of row r sits at
                // chunk position c ^ (r & 7) of the row's 128 bytes
                const uint8_t *tile = smem + kOffA + half * kTileBytes;
                float dot = 0.f, sq = 0.f;
#pragma unroll
                for (int hb = 0; hb < 2; ++hb) {
#pragma unroll
                    for (int c = 0; c < 8; ++c) {
                        const uint4 raw = *reinterpret_cast<const uint4 *>(tile + hb * kHalfBytes + lrow * 128 +
                                                                           ((c ^ (lrow & 7)) << 4));
                        float f[8];
                        Elem<__nv_bfloat16>::unpack(raw, f);
#pragma unroll
                        for (int e = 0; e < 8; ++e) {
                            dot = fmaf(f[e], sum_s[hb * 64 + c * 8 + e], dot);
                            sq = fmaf(f[e], f[e], sq);
                        }
                    }
                }
                total = ri * dot - (ri * ri) * sq;
            }
            const float kInf = __int_as_float(0x7f800000);
            float thr = (row_ok && ri > 0.f) ? __fdiv_rn(p.sim_threshold, ri) : kInf;   // compare g * r_j with T / r_i
            int left = row_ok ? p.beta : 0;
            if (left == 0) thr = kInf;
            float removed = 0.f;

            for (int t = 0; ok && t < n_iter; ++t) {
                const int a = t & 1;
                const int jt = n_tiles - 1 - t;
                if (!mbar_wait(bar.acc_full(a), (t >> 1) & 1, abort_flag, sink)) break;
                if (warp_active) {
                    tc_fence_after();
                    const bool any_live = __any_sync(0xffffffffu, thr < kInf);
                    if (any_live) {
#pragma unroll 1
                        for (int c0 = kTile - 32; c0 >= 0; c0 -= 32) {          // columns downwards
                            uint32_t g[32];
                            tmem_ld32(lane_base + a * 256 + half * 128 + c0, g);
                            const float4 *rj4 = reinterpret_cast<const float4 *>(r_s + jt * kTile + c0);
                            float rj[32];
#pragma unroll
                            for (int q4 = 0; q4 < 8; ++q4) {
                                const float4 t4 = rj4[q4];
                                rj[4 * q4] = t4.x; rj[4 * q4 + 1] = t4.y; rj[4 * q4 + 2] = t4.z; rj[4 * q4 + 3] = t4.w;
                            }
                            tmem_ld_wait();
                            float v[32], mx = 0.f;
#pragma unroll
                            for (int c = 0; c < 32; ++c) {
                                v[c] = __uint_as_float(g[c]) * rj[c];
                                mx = fmaxf(mx, v[c]);                            // NaN-ignoring max
                            }
                            if (mx > thr) {
                                const int jbase = jt * kTile + c0;
#pragma unroll
                                for (int c = 31; c >= 0; --c) {
                                    if (v[c] > thr && jbase + c != i) {          // zero diagonal (Eq. 5)
                                        removed += v[c];
                                        if (--left == 0) thr = kInf;
                                    }
                                }
                            }
                        }
                    }
                    tc_fence_before();
                    __syncwarp();
                    if (lane == 0) mbar_arrive(bar.acc_empty(a));
                }
            }
            if (row_ok) p.sbar[(size_t)head * p.cap_pad + i] = (total - removed * ri) / (float)n;
        } else {
            // Eq. 2-3: thread = key, all G * alpha logits of that key in its accumulator row
            float *stage_f = reinterpret_cast<float *>(smem + kOffStage);           // [q_rows_pad][128] floats
            float *logits = p.logits + (size_t)head * p.alpha * p.cap_pad;
            const float scale = p.logit_scale;                                    // 1 / sqrt(d)
            for (int t = 0; t < n_iter; ++t) {
                const int a = t & 1;
                const int jt = n_tiles - 1 - t;
                if (!mbar_wait(bar.acc_full(a), (t >> 1) & 1, abort_flag, sink)) break;
                if (warp_active) {
                    tc_fence_after();
                    const int i = jt * kTile + lrow;
                    for (int c0 = 0; c0 < q_rows_pad; c0 += 16) {
                        uint32_t g[16];
                        tmem_ld16(lane_base + a * 256 + c0, g);
                        tmem_ld_wait();
#pragma unroll
                        for (int c = 0; c < 16; ++c) stage_f[(c0 + c) * kTile + lrow] = __uint_as_float(g[c]);
                    }
                    tc_fence_before();
                    __syncwarp();
                    if (lane == 0) mbar_arrive(bar.acc_empty(a));
                    if (i < n) {
                        for (int j = 0; j < p.alpha; ++j) {
                            float best = -INFINITY, total = 0.f;
                            for (int gq = 0; gq < p.group; ++gq) {
                                const float lg = stage_f[(gq * p.alpha + j) * kTile + lrow] * scale;
                                best = fmaxf(best, lg);
                                total += lg;
                            }
                            logits[(size_t)j * p.cap_pad + i] = p.gqa_mean_pool ? total / (float)p.group : best;
                        }
                    }
                }
            }
        }
    }

    // ---------------------------------------------------------------------- common exit
    tc_fence_before();
    __syncthreads();
    if (warp == 1) {
        if (*abort_flag) __nanosleep(200000);      // error path only: let copies and MMAs in flight land
        tc_fence_after();
        asm volatile("tcgen05.dealloc.cta_group::1.sync.aligned.b32 %0, %1;" ::"r"(tmem_base), "r"(kTmemCols) : "memory");
    }
    if (threadIdx.x == 0 && !is_q && !*abort_flag)
        atomicAdd(p.counters, (unsigned long long)(n_iter * num_m));
}

}  // namespace

bool scores_sm100_available() { return true; }
long long sm100_default_wait_cycles() { return sm100::kWaitCycles; }

cudaError_t launch_scores_sm100(const Params &p, cudaStream_t s)
{
    const int q_rows = p.group * p.alpha;
    const int q_rows_pad = (q_rows + 15) / 16 * 16;
    CUtensorMap map_k, map_q;
    if (!make_map(&map_k, p.k_cache, key_rows_total(p), kTile) ||
        !make_map(&map_q, p.q_window, (uint64_t)p.batch * p.hq * p.alpha, (uint32_t)q_rows_pad))
        return cudaErrorInvalidValue;
    cudaError_t e = cudaFuncSetAttribute(scores_sm100_kernel, cudaFuncAttributeMaxDynamicSharedMemorySize, kSmemBytes);
    if (e != cudaSuccess) return e;
    const int row_blocks = (p.cap + kRowsPerBlock - 1) / kRowsPerBlock;
    const unsigned grid = (unsigned)(row_blocks + 1) * (unsigned)(p.batch * p.hkv);
    scores_sm100_kernel<<<grid, kThreads, kSmemBytes, s>>>(p, map_k, map_q, row_blocks, q_rows_pad);
    return cudaGetLastError();
}

}  // namespace rkv

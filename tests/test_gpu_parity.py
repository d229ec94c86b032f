"""Parity of the CUDA path (through the C ABI) with the CPU oracle, element by element on the same seeded
inputs.  Every test here needs a B200."""
import numpy as np
import pytest
import torch

import rkv_inputs as ri
from parity_util import check_batch, from_paged, pick, random_block_table, raw_rows, to_paged

pytestmark = pytest.mark.gpu

DEFAULTS = dict(W=4, beta=1, T=0.5, eps=1e-8)


@pytest.fixture(scope="module")
def rkv():
    from paper_2505_24133_b200 import build as b
    b.build()
    import paper_2505_24133_b200 as r
    assert r.lib() is not None
    return r


def run_and_check(rkv, wl, *, flags=0, W=4, beta=1, T=0.5, eps=1e-8, lam=None, check_rows=None, stages=None,
                  budgets=None):
    """Compress wl on the GPU through the C ABI and compare with the oracle.  check_rows: indices of the
    leading (folded batch) dimension to verify (default: all)."""
    spec = wl.spec
    lam = spec.lam if lam is None else lam
    k0, v0, q0, s0 = wl.k_cache.clone(), wl.v_cache.clone(), wl.q_window.clone(), wl.seq_lens.clone()
    comp = rkv.Compressor(spec.folded_batch, spec.n_kv_heads, spec.n_q_heads, spec.budget, spec.buffer, spec.alpha,
                          lam, dtype=spec.torch_dtype, pool_w=W, beta=beta, sim_threshold=T, eps=eps, flags=flags,
                          dump_scores=True, budgets=None if budgets is None else torch.tensor(budgets),
                          head_dim=spec.head_dim)
    if stages is None:
        idx = comp.compress(wl.k_cache, wl.v_cache, wl.q_window, wl.seq_lens)
    else:
        for st in stages:
            idx = comp.compress(wl.k_cache, wl.v_cache, wl.q_window, wl.seq_lens, stages=st)
    torch.cuda.synchronize()
    rows = list(range(spec.folded_batch)) if check_rows is None else list(check_rows)
    sel = torch.tensor(rows, device=k0.device)
    rep = check_batch(pick(k0, sel), pick(v0, sel), q0[sel], s0[sel], budget=spec.budget, alpha=spec.alpha, lam=lam, W=W,
                      beta=beta, T=T, eps=eps, gpu_idx=idx[sel], gpu_k=pick(wl.k_cache, sel), gpu_v=pick(wl.v_cache, sel),
                      gpu_seq=wl.seq_lens[sel], gpu_scores=comp.scores[:, sel],
                      mean_then_pool=bool(flags & 4), head_mean=bool(flags & 8), gqa_mean_pool=bool(flags & 16),
                      budgets=None if budgets is None else [budgets[r] for r in rows])
    return rep, comp


def small_spec(name, *, layers=1, batch=2, hkv=2, hq=8, budget=256, buffer=64, alpha=8, dtype="bf16", span=16,
               copy_frac=0.3, sigma=0.05, lam=0.1, head_dim=128):
    return ri.CacheSpec(name, layers, batch, hkv, hq, head_dim, budget, buffer, alpha, lam, dtype, span, copy_frac, sigma,
                        4, 8.0)


# ----------------------------------------------------------------------------- config 1
def test_tiny_config_fp32(rkv):
    """Config 1: 1 KV head x 4 query heads, 96 cached tokens, fp32; keep 64."""
    wl = ri.make_workload(ri.SPECS["tiny"], device="cuda")
    rep, _ = run_and_check(rkv, wl)
    assert rep.ok(), rep.errors
    assert rep.compressed_heads == 1 and rep.threshold_flips == 0
    assert int(wl.seq_lens[0]) == 64


@pytest.mark.parametrize("seed", [1, 2, 3])
def test_tiny_shape_other_seeds_and_margin(rkv, seed):
    """The Tiny shape is small enough for one threshold flip to exceed 1e-3 on R, so its keys must stay clear
    of T: checked here through the oracle, for the seeds used."""
    import oracle
    wl = ri.make_workload(ri.SPECS["tiny"], device="cuda", seed=ri.BASE_SEED + 100 + seed)
    r = oracle.oracle_head(wl.k_cache[0, 0].cpu().numpy(), wl.q_window[0].cpu().numpy(), budget=64, alpha=8, lam=0.1,
                           W=4, beta=1, T=0.5, want_S=True)
    assert np.abs(r.S_raw - 0.5).min() > 1e-4
    rep, _ = run_and_check(rkv, wl)
    assert rep.ok(), rep.errors


# ----------------------------------------------------------------------------- small shapes, both score kernels
# the three scoring routes: fp32 CUDA cores; the two-pass tcgen05 kernels (default for bf16, whatever beta and T);
# the row-block tcgen05 kernel that forms the full matrix
SCORE_FLAGS = [pytest.param(1, id="simt"), pytest.param(0, id="sym"), pytest.param(2, id="rowblock")]


@pytest.mark.parametrize("flags", SCORE_FLAGS)
@pytest.mark.parametrize("hkv,hq", [(2, 2), (2, 8), (1, 7), (2, 10)])
def test_gqa_group_sizes(rkv, flags, hkv, hq):
    """G = 1 (Eq. 1), 4, 7, 5."""
    wl = ri.make_workload(small_spec(f"g{hq // hkv}", hkv=hkv, hq=hq), device="cuda", seed=11 + hq)
    rep, _ = run_and_check(rkv, wl, flags=flags)
    assert rep.ok(), rep.errors


@pytest.mark.parametrize("flags", SCORE_FLAGS)
@pytest.mark.parametrize("W", [0, 1, 4, 9])
def test_pooling_window(rkv, flags, W):
    wl = ri.make_workload(small_spec("w"), device="cuda", seed=21)
    rep, _ = run_and_check(rkv, wl, flags=flags, W=W)
    assert rep.ok(), rep.errors


@pytest.mark.parametrize("flags", SCORE_FLAGS)
@pytest.mark.parametrize("T,beta", [(0.0, 1), (0.5, 0), (0.5, 2), (0.5, 8), (0.5, 100000), (0.9, 1), (1.0, 3),
                                    (0.3, 40)])
def test_retention_threshold_and_beta(rkv, flags, T, beta):
    wl = ri.make_workload(small_spec("tb"), device="cuda", seed=31)
    rep, _ = run_and_check(rkv, wl, flags=flags, T=T, beta=beta)
    assert rep.ok(), rep.errors


@pytest.mark.parametrize("flags", SCORE_FLAGS)
@pytest.mark.parametrize("lam", [0.0, 0.5, 1.0])
def test_lambda_limits(rkv, flags, lam):
    wl = ri.make_workload(small_spec("lam"), device="cuda", seed=41)
    rep, _ = run_and_check(rkv, wl, flags=flags, lam=lam)
    assert rep.ok(), rep.errors


@pytest.mark.parametrize("flags", SCORE_FLAGS)
@pytest.mark.parametrize("budget,buffer,alpha,lens", [
    (16, 8, 1, [24, 17, 16, 3]),          # n as small as 16: one ragged tile; L = budget: guard; L < budget
    (64, 32, 8, [96, 65, 73, 0]),         # n = 88, 57, 65; an empty cache
    (120, 17, 8, [137, 129, 136, 121]),   # n = 129: one row past a tile boundary; n = 121, 128, 113
    (256, 131, 4, [387, 300, 257, 385]),  # four tiles with a ragged tail
])
def test_ragged_lengths_and_tile_edges(rkv, flags, budget, buffer, alpha, lens):
    spec = small_spec("ragged", batch=4, hkv=2, hq=4, budget=budget, buffer=buffer, alpha=alpha, span=4)
    wl = ri.make_workload(spec, device="cuda", seed=51, seq_lens=torch.tensor(lens))
    # rows beyond L are unspecified memory: fill them with a NaN pattern to prove they are never read as data
    for b, L in enumerate(lens):
        wl.k_cache[b, :, L:] = float("nan")
        wl.v_cache[b, :, L:] = float("nan")
    rep, _ = run_and_check(rkv, wl, flags=flags)
    assert rep.ok(), rep.errors
    assert rep.compressed_heads == 2 * sum(L > budget for L in lens)


@pytest.mark.parametrize("flags", [pytest.param(4 | 1, id="simt"), pytest.param(4, id="tri")])
@pytest.mark.parametrize("W,budget,buffer", [(0, 256, 64), (4, 256, 64), (9, 256, 64), (4, 1800, 128)])
def test_mean_then_pool_variant(rkv, flags, W, budget, buffer):
    """Algorithm 1's order for the importance (flag RKV_FLAG_MEAN_THEN_POOL): both forms of the select stage (one
    kernel for small caches, three for larger ones: budget 1800 + 128 is beyond the single-kernel limit)."""
    wl = ri.make_workload(small_spec("mtp", budget=budget, buffer=buffer), device="cuda", seed=151)
    rep, _ = run_and_check(rkv, wl, flags=flags, W=W)
    assert rep.ok(), rep.errors


@pytest.mark.parametrize("flags", [pytest.param(8 | 1, id="simt"), pytest.param(8, id="tri"),
                                   pytest.param(8 | 4, id="tri+mean_then_pool")])
@pytest.mark.parametrize("hkv,hq,budget,buffer", [(2, 8, 256, 64), (4, 8, 300, 75), (3, 6, 1800, 128)])
def test_head_mean_variant(rkv, flags, hkv, hq, budget, buffer):
    """Algorithm 1's aggregated selection (flag RKV_FLAG_HEAD_MEAN): one kept set per sequence from the head-averaged
    score, after both forms of the select stage; ragged lengths with one sequence left alone by the guard."""
    spec = small_spec("hm", batch=3, hkv=hkv, hq=hq, budget=budget, buffer=buffer)
    lens = torch.tensor([spec.cap, budget, budget + (buffer + 1) // 2])
    wl = ri.make_workload(spec, device="cuda", seed=171, seq_lens=lens)
    rep, comp = run_and_check(rkv, wl, flags=flags)
    assert rep.ok(), rep.errors
    assert rep.compressed_heads == 2 * hkv
    assert rkv.rkv_launch_count_for(comp.desc, budget, buffer, spec.alpha, rkv.RKV_STAGE_SELECT) == \
        (2 if budget < 1000 else 4)


@pytest.mark.parametrize("flags", [pytest.param(16 | 1, id="simt"), pytest.param(16, id="tri"),
                                   pytest.param(16 | 2, id="rowblock")])
@pytest.mark.parametrize("hkv,hq,alpha", [(2, 8, 8), (1, 7, 8), (2, 6, 5), (2, 2, 8)])
def test_gqa_mean_pool_variant(rkv, flags, hkv, hq, alpha):
    """Mean instead of max over the query heads of a group in Eq. 3 (flag RKV_FLAG_GQA_MEAN_POOL), on all three
    scoring routes: even and odd group sizes, the general query-window length, and G = 1."""
    spec = small_spec("gmp", batch=2, hkv=hkv, hq=hq, budget=256, buffer=64, alpha=alpha)
    wl = ri.make_workload(spec, device="cuda", seed=191)
    rep, _ = run_and_check(rkv, wl, flags=flags)
    assert rep.ok(), rep.errors
    assert rep.compressed_heads == 2 * hkv


def test_fp32_small_shapes(rkv):
    spec = small_spec("f32", dtype="f32", batch=3, budget=100, buffer=40)
    wl = ri.make_workload(spec, device="cuda", seed=61, seq_lens=torch.tensor([140, 101, 100]))
    rep, _ = run_and_check(rkv, wl)
    assert rep.ok(), rep.errors


@pytest.mark.parametrize("flags", SCORE_FLAGS)
def test_identical_keys_uniform_redundancy(rkv, flags):
    """All keys equal: R = 1/n exactly in the oracle; every candidate ties, and the latest k are kept."""
    spec = small_spec("same", batch=1, hkv=1, hq=4, budget=128, buffer=40, copy_frac=0.0)
    wl = ri.make_workload(spec, device="cuda", seed=71)
    wl.k_cache[:] = wl.k_cache[:, :, :1, :]
    rep, comp = run_and_check(rkv, wl, flags=flags, lam=0.0)
    assert rep.ok(), rep.errors
    n = spec.cap - spec.alpha
    R = comp.scores[2, 0, 0, :n]
    assert torch.allclose(R, torch.full_like(R, 1.0 / n), rtol=1e-5)


@pytest.mark.parametrize("flags", SCORE_FLAGS)
def test_stage_by_stage_equals_one_call(rkv, flags):
    spec = small_spec("stages", batch=3)
    wl_a = ri.make_workload(spec, device="cuda", seed=81)
    wl_b = ri.make_workload(spec, device="cuda", seed=81)
    rep, ca = run_and_check(rkv, wl_a, flags=flags)
    assert rep.ok(), rep.errors
    rep, cb = run_and_check(rkv, wl_b, flags=flags, stages=[rkv.RKV_STAGE_PREP, rkv.RKV_STAGE_SCORES,
                                                            rkv.RKV_STAGE_SELECT, rkv.RKV_STAGE_GATHER])
    assert rep.ok(), rep.errors
    assert torch.equal(ca.out_idx, cb.out_idx)
    assert torch.equal(wl_a.k_cache.view(torch.int16), wl_b.k_cache.view(torch.int16))
    assert torch.equal(ca.scores, cb.scores)     # deterministic: the same bits on a second run


# ----------------------------------------------------------------------------- compaction
@pytest.mark.parametrize("pattern", ["identity", "last_k", "every_other", "long_shift", "random"])
@pytest.mark.parametrize("dtype", ["bf16", "f32"])
def test_in_place_gather_overlap(rkv, pattern, dtype):
    """The gather stage alone, on hand-made ascending index lists that stress the in-place hazards."""
    budget, buffer, alpha = 200, 150, 8
    spec = small_spec("gather", batch=2, hkv=3, hq=3, budget=budget, buffer=buffer, alpha=alpha, dtype=dtype)
    wl = ri.make_workload(spec, device="cuda", seed=91)
    cap = spec.cap
    comp = rkv.Compressor(2, 3, 3, budget, buffer, alpha, 0.1, dtype=spec.torch_dtype, flags=1)
    comp.compress(wl.k_cache, wl.v_cache, wl.q_window, wl.seq_lens, stages=rkv.RKV_STAGE_PREP)  # records lengths
    g = torch.Generator().manual_seed(5)
    idx = torch.empty(2, 3, budget, dtype=torch.int32)
    for b in range(2):
        for h in range(3):
            if pattern == "identity":
                row = torch.arange(budget)
            elif pattern == "last_k":
                row = torch.arange(cap - budget, cap)
            elif pattern == "every_other":
                row = torch.cat([torch.arange(0, 2 * (budget - 30), 2), torch.arange(cap - 30, cap)])
            elif pattern == "long_shift":
                row = torch.cat([torch.arange(0, 70), torch.arange(cap - (budget - 70), cap)])
            else:
                row = torch.randperm(cap, generator=g)[:budget].sort().values
            idx[b, h] = row.int()
    comp.out_idx.copy_(idx)
    k0, v0 = raw_rows(wl.k_cache), raw_rows(wl.v_cache)
    comp.compress(wl.k_cache, wl.v_cache, wl.q_window, wl.seq_lens, stages=rkv.RKV_STAGE_GATHER)
    torch.cuda.synchronize()
    k1, v1 = raw_rows(wl.k_cache), raw_rows(wl.v_cache)
    for b in range(2):
        for h in range(3):
            sel = idx[b, h].long().numpy()
            assert np.array_equal(k1[b, h, :budget], k0[b, h][sel])
            assert np.array_equal(v1[b, h, :budget], v0[b, h][sel])
    assert wl.seq_lens.tolist() == [budget, budget]


def test_second_call_is_a_no_op(rkv):
    """Idempotence: after a compression L = budget, so Algorithm 1's guard leaves everything alone."""
    spec = small_spec("idem")
    wl = ri.make_workload(spec, device="cuda", seed=101)
    comp = rkv.Compressor(spec.folded_batch, 2, 8, spec.budget, spec.buffer, spec.alpha, 0.1, flags=1)
    comp.compress(wl.k_cache, wl.v_cache, wl.q_window, wl.seq_lens)
    torch.cuda.synchronize()
    k1, v1 = wl.k_cache.clone(), wl.v_cache.clone()
    idx = comp.compress(wl.k_cache, wl.v_cache, wl.q_window, wl.seq_lens)
    torch.cuda.synchronize()
    assert torch.equal(k1.view(torch.int16), wl.k_cache.view(torch.int16))
    assert torch.equal(v1.view(torch.int16), wl.v_cache.view(torch.int16))
    assert torch.equal(idx[0, 0].cpu(), torch.arange(spec.budget, dtype=torch.int32))
    comp.check_status()


@pytest.mark.parametrize("flags", SCORE_FLAGS)
def test_length_beyond_capacity_is_reported_not_clamped(rkv, flags):
    """One sequence with an impossible length: it alone is skipped and reported; the other sequences of the batch are
    compressed exactly as if it were not there (full parity on them), on every scoring route."""
    spec = small_spec("bad", batch=3)
    wl = ri.make_workload(spec, device="cuda", seed=111, seq_lens=torch.tensor([spec.cap, spec.cap, spec.cap]))
    wl.seq_lens[1] = spec.cap + 1
    k0, v0, q0, s0 = wl.k_cache.clone(), wl.v_cache.clone(), wl.q_window.clone(), wl.seq_lens.clone()
    comp = rkv.Compressor(3, 2, 8, spec.budget, spec.buffer, spec.alpha, 0.1, flags=flags, dump_scores=True)
    idx = comp.compress(wl.k_cache, wl.v_cache, wl.q_window, wl.seq_lens)
    torch.cuda.synchronize()
    assert int(comp.status.item()) == 1                      # RKV_ERR_INVALID_ARG
    assert bool((idx[1] == -1).all())
    assert torch.equal(k0[1].view(torch.int16), wl.k_cache[1].view(torch.int16))
    assert torch.equal(v0[1].view(torch.int16), wl.v_cache[1].view(torch.int16))
    assert wl.seq_lens.tolist() == [spec.budget, spec.cap + 1, spec.budget]
    sel = torch.tensor([0, 2], device="cuda")
    d = comp.desc
    rep = check_batch(k0[sel], v0[sel], q0[sel], s0[sel], budget=spec.budget, alpha=spec.alpha, lam=0.1, W=d.pool_w,
                      beta=d.beta, T=d.sim_threshold, eps=d.eps, gpu_idx=idx[sel], gpu_k=wl.k_cache[sel],
                      gpu_v=wl.v_cache[sel], gpu_seq=wl.seq_lens[sel], gpu_scores=comp.scores[:, sel])
    assert rep.ok(), rep.errors
    assert rep.compressed_heads == 4
    with pytest.raises(rkv.RkvError):
        comp.check_status()


@pytest.mark.parametrize("flags", SCORE_FLAGS)
def test_stale_status_word_does_not_disturb_a_call(rkv, flags):
    """The status word is write-only for the library: a value left over from an earlier call (here planted by hand)
    changes nothing in the next call, and stays as it is."""
    spec = small_spec("stale", batch=2, budget=384, buffer=128)
    wl = ri.make_workload(spec, device="cuda", seed=113)
    k0, v0, q0, s0 = wl.k_cache.clone(), wl.v_cache.clone(), wl.q_window.clone(), wl.seq_lens.clone()
    comp = rkv.Compressor(spec.folded_batch, 2, 8, spec.budget, spec.buffer, spec.alpha, 0.1, flags=flags)
    comp.status.fill_(5)
    idx = comp.compress(wl.k_cache, wl.v_cache, wl.q_window, wl.seq_lens)
    torch.cuda.synchronize()
    assert int(comp.status.item()) == 5
    rep = check_batch(k0, v0, q0, s0, budget=spec.budget, alpha=spec.alpha, lam=0.1, gpu_idx=idx, gpu_k=wl.k_cache,
                      gpu_v=wl.v_cache, gpu_seq=wl.seq_lens, **DEFAULTS)
    assert rep.ok(), rep.errors
    assert rep.compressed_heads == 4


def test_bounded_wait_runs_out_and_the_context_stays_usable(rkv):
    """Failure detection without a fault: a device-side wait on a barrier that nothing arrives at gives up after its
    limit (about a millisecond here), records RKV_ERR_TIMEOUT, calls off the other waiting thread of the block, and
    the kernel ends normally with its tensor memory freed.  A compression enqueued right behind it on the same stream
    is unaffected."""
    status = torch.zeros(1, dtype=torch.int32, device="cuda")
    words = torch.full((8,), 77, dtype=torch.int64, device="cuda")
    limit = 2_000_000                                       # about 1 ms at 1.9 GHz
    assert rkv.rkv_selftest_wait_expiry(status, words, 10, None) == 1       # limit out of range: refused
    assert rkv.rkv_selftest_wait_expiry(status, words, limit) == rkv.RKV_OK
    spec = small_spec("after_timeout", batch=2, budget=384, buffer=128)
    wl = ri.make_workload(spec, device="cuda", seed=115)
    rep, comp = run_and_check(rkv, wl)                      # same (current) stream, straight behind the self-test
    w = words.tolist()
    assert int(status.item()) == 5                          # RKV_ERR_TIMEOUT
    assert w[0] != 0                                        # abort recorded
    assert w[2] == 0 and limit < w[1] < 50 * limit          # the first wait failed, after its limit and not much later
    assert w[4] == 1 and w[3] < 100 * limit                 # the second was called off long before two seconds
    assert w[5] == 1                                        # the block reached its end
    assert rep.ok(), rep.errors
    comp.check_status()


# ----------------------------------------------------------------------------- symmetric route of the second pass
@pytest.mark.parametrize("T", [0.9, 0.75])
@pytest.mark.parametrize("budget,buffer,lens", [(1536, 128, [1664, 1640, 1537, 513]), (1500, 120, [1620, 1619, 1580, 1501])])
def test_symmetric_route_for_heads_with_few_partners(rkv, T, budget, buffer, lens):
    """With a high threshold nearly every token is still without a partner after the first pass, and a head is then
    scored by forming each pair of key tiles once (row and column direction of the same product).  Checked against the
    oracle and against the same call with that route switched off: same Sbar up to rounding, same kept sets; ragged
    lengths (12 and 13 key tiles, odd and even counts, ragged last tiles), rows beyond the length filled with NaN."""
    spec = small_spec("symroute", batch=4, hkv=2, hq=8, budget=budget, buffer=buffer, span=32)
    wl_a = ri.make_workload(spec, device="cuda", seed=261, seq_lens=torch.tensor(lens))
    wl_b = ri.make_workload(spec, device="cuda", seed=261, seq_lens=torch.tensor(lens))
    for wl in (wl_a, wl_b):
        for b, L in enumerate(lens):
            wl.k_cache[b, :, L:] = float("nan")
            wl.v_cache[b, :, L:] = float("nan")
    rep_a, ca = run_and_check(rkv, wl_a, T=T)
    rep_b, cb = run_and_check(rkv, wl_b, T=T, flags=rkv.RKV_FLAG_NO_SYMMETRIC)
    print(rep_a.summary())
    assert rep_a.ok(), rep_a.errors
    assert rep_b.ok(), rep_b.errors
    assert rep_a.compressed_heads == 2 * sum(L > budget for L in lens)
    ca.check_status()
    n_max = spec.cap - spec.alpha
    assert torch.allclose(ca.scores[1, :, :, :n_max], cb.scores[1, :, :, :n_max], rtol=0, atol=2e-6, equal_nan=True)
    same = (ca.out_idx == cb.out_idx).all(dim=-1).float().mean().item()
    assert same > 0.7


# ----------------------------------------------------------------------------- paged caches
@pytest.mark.parametrize("flags,dtype", [pytest.param(0, "bf16", id="sym"), pytest.param(1, "bf16", id="simt"),
                                         pytest.param(2, "bf16", id="rowblock"), pytest.param(0, "f32", id="f32")])
@pytest.mark.parametrize("budget,buffer,lens", [(384, 128, [512, 500, 384, 390]), (1920, 128, [2048, 2047, 1921, 100])])
def test_paged_caches(rkv, flags, dtype, budget, buffer, lens):
    """Paged caches (pages of 128 rows scattered over a pool, in random order, with foreign pages full of NaN in
    between): the step through the block table gives bit for bit what it gives on contiguous caches, the table is left
    as it was, pages of other owners are not touched, and the result agrees with the oracle."""
    spec = small_spec("paged", batch=4, hkv=2, hq=8, budget=budget, buffer=buffer, dtype=dtype, span=32)
    wl = ri.make_workload(spec, device="cuda", seed=251, seq_lens=torch.tensor(lens))
    k0, v0, q0, s0 = wl.k_cache.clone(), wl.v_cache.clone(), wl.q_window.clone(), wl.seq_lens.clone()
    pages = spec.cap // 128
    pool_pages = 4 * 2 * pages + 37
    table = random_block_table(4, 2, pages, pool_pages, seed=7)
    kp, vp = to_paged(k0, pool_pages, table), to_paged(v0, pool_pages, table)
    kp0 = kp.clone()
    comp = rkv.Compressor(4, 2, 8, budget, buffer, spec.alpha, spec.lam, dtype=spec.torch_dtype, flags=flags,
                          dump_scores=True, block_table=table, pool_pages=pool_pages)
    seq = s0.clone()
    idx = comp.compress(kp, vp, q0, seq)
    torch.cuda.synchronize()
    comp.check_status()
    assert torch.equal(comp.block_table, table)
    k1, v1 = from_paged(kp, table), from_paged(vp, table)
    rep = check_batch(k0, v0, q0, s0, budget=budget, alpha=spec.alpha, lam=spec.lam, gpu_idx=idx, gpu_k=k1, gpu_v=v1,
                      gpu_seq=seq, gpu_scores=comp.scores, **DEFAULTS)
    print(rep.summary())
    assert rep.ok(), rep.errors
    assert rep.compressed_heads == 2 * sum(L > budget for L in lens)
    owned = torch.zeros(pool_pages, dtype=torch.bool, device="cuda")
    owned[table.reshape(-1).long()] = True
    view = torch.int16 if dtype == "bf16" else torch.int32
    assert torch.equal(kp[~owned].view(view), kp0[~owned].view(view))          # foreign pages untouched
    # the same call on the contiguous caches: identical index lists and rows
    ref = rkv.Compressor(4, 2, 8, budget, buffer, spec.alpha, spec.lam, dtype=spec.torch_dtype, flags=flags)
    ref_idx = ref.compress(wl.k_cache, wl.v_cache, wl.q_window, wl.seq_lens)
    torch.cuda.synchronize()
    assert torch.equal(ref_idx, idx) and torch.equal(wl.seq_lens, seq)
    for b, L in enumerate(lens):
        if L > budget:
            assert torch.equal(k1[b, :, :budget].view(view), wl.k_cache[b, :, :budget].view(view))
            assert torch.equal(v1[b, :, :budget].view(view), wl.v_cache[b, :, :budget].view(view))


def test_paged_caches_need_whole_pages(rkv):
    d = rkv.rkv_desc_default()
    d.batch, d.n_kv_heads, d.n_q_heads = 2, 2, 8
    d.block_table, d.pool_pages = 0x40000, 64
    assert rkv.rkv_workspace_bytes(d, 256, 64, 8) == 0            # 320 rows: not a multiple of the 128-row page
    assert rkv.rkv_workspace_bytes(d, 256, 128, 8) > 0


# ----------------------------------------------------------------------------- other head dimensions
@pytest.mark.parametrize("dtype", ["bf16", "f32"])
@pytest.mark.parametrize("head_dim", [64, 256])
@pytest.mark.parametrize("hkv,hq,budget,buffer,lens", [(2, 8, 256, 64, [320, 300, 256]), (2, 2, 120, 17, [137, 129, 121]),
                                                       (1, 5, 1800, 128, [1928, 1900, 1801])])
def test_head_dimensions_64_and_256(rkv, dtype, head_dim, hkv, hq, budget, buffer, lens):
    """Head dimensions other than 128 (every stage: prep, scoring -- bf16 keys of 64 dimensions on the tensor-core kernels
    through a copy padded to 128, everything else on the CUDA-core kernel --, both forms of the select stage, in-place
    compaction with 128- to 1024-byte rows), grouped and multi-head (G = 1, Eq. 1) queries, ragged lengths."""
    spec = small_spec("hd", batch=3, hkv=hkv, hq=hq, budget=budget, buffer=buffer, dtype=dtype, head_dim=head_dim)
    wl = ri.make_workload(spec, device="cuda", seed=241 + head_dim, seq_lens=torch.tensor(lens))
    for b, L in enumerate(lens):
        wl.k_cache[b, :, L:] = float("nan")
        wl.v_cache[b, :, L:] = float("nan")
    rep, comp = run_and_check(rkv, wl)
    print(rep.summary())
    assert rep.ok(), rep.errors
    assert rep.compressed_heads == hkv * sum(L > budget for L in lens)
    comp.check_status()


@pytest.mark.parametrize("flags", [pytest.param(1, id="simt"), pytest.param(2, id="rowblock"), pytest.param(32, id="two-pass"),
                                   pytest.param(8, id="sym+head_mean")])
@pytest.mark.parametrize("T,beta", [(0.5, 1), (0.9, 1), (0.5, 3)])
def test_head_dimension_64_routes_and_settings(rkv, flags, T, beta):
    """bf16 keys of 64 dimensions on every scoring route (the tensor-core ones through the padded copy, the CUDA-core
    one on the cache itself) at a size where the two rounds and the symmetric route are reached; Eq. 2's scale is that
    of the cache's own head dimension."""
    spec = small_spec("hd64", batch=2, hkv=2, hq=8, budget=1536, buffer=128, head_dim=64, span=32)
    lens = [spec.cap, spec.cap - 3]
    wl = ri.make_workload(spec, device="cuda", seed=261, seq_lens=torch.tensor(lens))
    rep, comp = run_and_check(rkv, wl, flags=flags, T=T, beta=beta)
    print(rep.summary())
    assert rep.ok(), rep.errors
    assert rep.compressed_heads == 4
    comp.check_status()


@pytest.mark.parametrize("flags", [pytest.param(0, id="sym"), pytest.param(1, id="simt"), pytest.param(2, id="rowblock")])
def test_degenerate_inputs(rkv, flags):
    """The degenerate cases of the method: keys that are all zero (norm 0: Eq. 5's epsilon keeps the division finite and
    the key similar to nothing), a whole head of zero keys, queries that are all zero (Eq. 2-3 give uniform weights),
    and the smallest shapes the call takes (budget = alpha + 1: one candidate is kept; buffer = 1)."""
    spec = small_spec("degen", batch=3, hkv=2, hq=8, budget=300, buffer=84)
    wl = ri.make_workload(spec, device="cuda", seed=281)
    wl.k_cache[0, 0, 5:40] = 0                       # a run of zero keys
    wl.k_cache[0, 0, 383] = 0                        # the last position
    wl.k_cache[1, 1] = 0                             # a whole head
    wl.q_window[2] = 0                               # uniform attention for a sequence
    rep, comp = run_and_check(rkv, wl, flags=flags)
    print(rep.summary())
    assert rep.ok(), rep.errors
    assert rep.compressed_heads == 6
    comp.check_status()
    tiny = small_spec("degen_tiny", batch=2, hkv=2, hq=8, budget=9, buffer=1)
    wl = ri.make_workload(tiny, device="cuda", seed=283, seq_lens=torch.tensor([10, 9]))
    rep, comp = run_and_check(rkv, wl, flags=flags)
    assert rep.ok(), rep.errors
    assert rep.compressed_heads == 2 and wl.seq_lens.tolist() == [9, 9]
    comp.check_status()


@pytest.mark.parametrize("flags", [pytest.param(0, id="sym"), pytest.param(32, id="two-pass")])
def test_largest_supported_capacity(rkv, flags):
    """budget + buffer = 8192 rows, the largest capacity the library takes (64 key tiles: the longest second-pass scans,
    32 work items per head in the symmetric scan), a full cache and one a few rows short of full."""
    spec = small_spec("maxcap", batch=2, hkv=1, hq=4, budget=8192 - 128, buffer=128, span=32)
    lens = [8192, 8192 - 77]
    wl = ri.make_workload(spec, device="cuda", seed=271, seq_lens=torch.tensor(lens))
    rep, comp = run_and_check(rkv, wl, flags=flags)
    print(rep.summary())
    assert rep.ok(), rep.errors
    assert rep.compressed_heads == 2
    comp.check_status()


@pytest.mark.parametrize("flags", [pytest.param(0, id="sym"), pytest.param(2, id="rowblock"), pytest.param(1, id="simt")])
def test_largest_supported_query_group(rkv, flags):
    """G * alpha = 112 query rows per KV head, the most the library takes (14 query heads per KV head with alpha = 8: the
    first pass's product then has 128 + 112 + 16 = 256 columns, the widest a tensor-core product can be)."""
    spec = small_spec("maxgroup", batch=2, hkv=2, hq=28, budget=1024, buffer=128, span=32)
    wl = ri.make_workload(spec, device="cuda", seed=273, seq_lens=torch.tensor([1152, 1100]))
    rep, comp = run_and_check(rkv, wl, flags=flags)
    print(rep.summary())
    assert rep.ok(), rep.errors
    assert rep.compressed_heads == 4
    comp.check_status()


# ----------------------------------------------------------------------------- per-sequence budgets
@pytest.mark.parametrize("flags", [pytest.param(1, id="simt"), pytest.param(0, id="sym"), pytest.param(2, id="rowblock"),
                                   pytest.param(8, id="sym+head_mean")])
@pytest.mark.parametrize("budget,buffer", [(256, 64), (1800, 128)])
def test_per_sequence_budgets(rkv, flags, budget, buffer):
    """A budget of its own for every sequence (Section 4.2's budget ratios): each sequence keeps exactly its own
    budget, the rest of its index rows is -1, its new length is its budget; a sequence at or below its budget is left
    alone; both forms of the select stage."""
    spec = small_spec("pseq", batch=4, hkv=2, hq=8, budget=budget, buffer=buffer)
    lens = [spec.cap, spec.cap - 7, budget // 2 + 40, budget // 2]
    budgets = [budget, budget - 55, budget // 2, budget // 2 + 10]
    wl = ri.make_workload(spec, device="cuda", seed=231, seq_lens=torch.tensor(lens))
    rep, comp = run_and_check(rkv, wl, flags=flags, budgets=budgets)
    print(rep.summary())
    assert rep.ok(), rep.errors
    assert rep.compressed_heads == 6
    assert wl.seq_lens.tolist() == [budget, budget - 55, budget // 2, budget // 2]
    comp.check_status()


def test_per_sequence_budget_out_of_range_is_reported(rkv):
    spec = small_spec("pseq_bad", batch=3)
    wl = ri.make_workload(spec, device="cuda", seed=233)
    k0 = wl.k_cache.clone()
    comp = rkv.Compressor(3, 2, 8, spec.budget, spec.buffer, spec.alpha, 0.1,
                          budgets=torch.tensor([spec.budget, spec.budget + 1, spec.alpha]))
    idx = comp.compress(wl.k_cache, wl.v_cache, wl.q_window, wl.seq_lens)
    torch.cuda.synchronize()
    assert int(comp.status.item()) == 1
    assert bool((idx[1:] == -1).all()) and bool((idx[0] >= 0).all())
    assert torch.equal(k0[1:].view(torch.int16), wl.k_cache[1:].view(torch.int16))
    assert wl.seq_lens.tolist() == [spec.budget, spec.cap, spec.cap]


# ----------------------------------------------------------------------------- hard inputs at benchmark sizes
@pytest.mark.parametrize("flags", [pytest.param(0, id="sym"), pytest.param(32, id="rounds_only"), pytest.param(2, id="rowblock")])
@pytest.mark.parametrize("T,beta,budget", [(0.9, 1, 2048), (0.5, 8, 2048), (1.0, 1, 2048), (0.5, 400, 2048),
                                           (0.9, 1, 4096), (0.5, 8, 4096)])
def test_hard_retention_settings_at_benchmark_sizes(rkv, flags, T, beta, budget):
    """The settings that defeat the two-pass shortcut -- a high threshold (few partners: nearly every token is listed
    for the second pass), several partners per token (their r_j staged per head in shared memory), the rule switched
    off by T = 1 -- at the cache sizes of the benchmark configurations (17 and 33 key tiles), not only on small
    shapes."""
    spec = small_spec("hard", batch=1, hkv=2, hq=8, budget=budget, buffer=128, span=32)
    wl = ri.make_workload(spec, device="cuda", seed=211 + budget)
    rep, comp = run_and_check(rkv, wl, flags=flags, T=T, beta=beta)
    print(rep.summary())
    assert rep.ok(), rep.errors
    assert rep.compressed_heads == 2
    comp.check_status()


def test_host_buffer_entry_point_matches_device_entry_point(rkv):
    spec = small_spec("host", batch=3)
    wl = ri.make_workload(spec, device="cuda", seed=121, seq_lens=torch.tensor([spec.cap, 200, spec.cap - 5]))
    hk, hv, hq = (t.cpu().pin_memory() for t in (wl.k_cache, wl.v_cache, wl.q_window))
    hs = wl.seq_lens.cpu().pin_memory()
    hidx = torch.empty(3, 2, spec.budget, dtype=torch.int32).pin_memory()
    ch = rkv.Compressor(3, 2, 8, spec.budget, spec.buffer, spec.alpha, 0.1, flags=1, host_staging=True)
    ch.compress_host(hk, hv, hq, hs, hidx)
    cd = rkv.Compressor(3, 2, 8, spec.budget, spec.buffer, spec.alpha, 0.1, flags=1)
    idx = cd.compress(wl.k_cache, wl.v_cache, wl.q_window, wl.seq_lens)
    torch.cuda.synchronize()
    assert torch.equal(hidx, idx.cpu())
    assert torch.equal(hs, wl.seq_lens.cpu())
    b = spec.budget
    assert torch.equal(hk[:, :, :b].view(torch.int16), wl.k_cache[:, :, :b].cpu().view(torch.int16))
    assert torch.equal(hv[:, :, :b].view(torch.int16), wl.v_cache[:, :, :b].cpu().view(torch.int16))


def test_thread_current_descriptor_entry_point(rkv):
    """rkv_compress, the 10-argument form, with the descriptor installed by rkv_set_desc."""
    spec = small_spec("tls")
    wl_a = ri.make_workload(spec, device="cuda", seed=131)
    wl_b = ri.make_workload(spec, device="cuda", seed=131)
    comp = rkv.Compressor(spec.folded_batch, 2, 8, spec.budget, spec.buffer, spec.alpha, 0.1, flags=1)
    ref = comp.compress(wl_a.k_cache, wl_a.v_cache, wl_a.q_window, wl_a.seq_lens).clone()
    assert rkv.rkv_set_desc(comp.desc) == 0
    out = torch.empty_like(ref)
    rc = rkv.rkv_compress(wl_b.k_cache, wl_b.v_cache, wl_b.q_window, wl_b.seq_lens, spec.budget, spec.buffer,
                          spec.alpha, 0.1, out)
    torch.cuda.synchronize()
    assert rc == 0 and torch.equal(out, ref)
    assert torch.equal(wl_a.k_cache.view(torch.int16), wl_b.k_cache.view(torch.int16))


def test_call_is_capturable_in_a_cuda_graph_and_replays(rkv):
    """The call only enqueues work on its stream (no synchronisation, no allocation), so a decode loop can capture
    it in a CUDA graph: the replayed graph gives bit for bit what the eager call gives, also when replayed again on
    restored inputs, and the result agrees with the oracle."""
    spec = small_spec("graph", batch=2, budget=384, buffer=128)          # four key tiles: all eight kernels run
    wl = ri.make_workload(spec, device="cuda", seed=181)
    k0, v0, s0 = wl.k_cache.clone(), wl.v_cache.clone(), wl.seq_lens.clone()
    comp = rkv.Compressor(spec.folded_batch, spec.n_kv_heads, spec.n_q_heads, spec.budget, spec.buffer, spec.alpha,
                          spec.lam)
    idx_eager = comp.compress(wl.k_cache, wl.v_cache, wl.q_window, wl.seq_lens).clone()
    torch.cuda.synchronize()
    comp.check_status()
    k_eager, v_eager, s_eager = wl.k_cache.clone(), wl.v_cache.clone(), wl.seq_lens.clone()

    def restore():
        wl.k_cache.copy_(k0)
        wl.v_cache.copy_(v0)
        wl.seq_lens.copy_(s0)

    restore()
    graph = torch.cuda.CUDAGraph()
    side = torch.cuda.Stream()
    side.wait_stream(torch.cuda.current_stream())
    with torch.cuda.graph(graph, stream=side):
        comp.compress(wl.k_cache, wl.v_cache, wl.q_window, wl.seq_lens, stream=torch.cuda.current_stream())
    torch.cuda.synchronize()
    for _ in range(2):
        restore()
        comp.out_idx.fill_(-5)
        graph.replay()
        torch.cuda.synchronize()
        comp.check_status()
        assert torch.equal(comp.out_idx, idx_eager)
        assert torch.equal(wl.seq_lens, s_eager)
        nb = spec.budget
        assert torch.equal(wl.k_cache[:, :, :nb].view(torch.int16), k_eager[:, :, :nb].view(torch.int16))
        assert torch.equal(wl.v_cache[:, :, :nb].view(torch.int16), v_eager[:, :, :nb].view(torch.int16))
    rep = check_batch(k0, v0, wl.q_window, s0, budget=spec.budget, alpha=spec.alpha, lam=spec.lam, W=4, beta=1, T=0.5,
                      eps=1e-8, gpu_idx=comp.out_idx, gpu_k=wl.k_cache, gpu_v=wl.v_cache, gpu_seq=wl.seq_lens)
    assert rep.ok(), rep.errors


def test_kernel_events_and_executed_tile_counter(rkv):
    """The profiling hooks of the descriptor: nine event boundaries give eight non-negative kernel times, and the
    tensor-core kernels report how many 128 x 128 x 128 tile products they executed: at least one key tile per row
    tile (pass 1), at most the full matrix."""
    spec = small_spec("events", batch=4, budget=512, buffer=128)
    wl = ri.make_workload(spec, device="cuda", seed=141)
    comp = rkv.Compressor(spec.folded_batch, 2, 8, spec.budget, spec.buffer, spec.alpha, 0.1, stage_events=True)
    comp.compress(wl.k_cache, wl.v_cache, wl.q_window, wl.seq_lens)
    torch.cuda.synchronize()
    comp.check_status()
    ms = comp.kernel_ms()
    assert len(ms) == len(comp.KERNEL_NAMES) == 8 and all(t >= 0.0 for t in ms) and sum(ms) > 0.0
    heads, T = spec.head_problems, -(-(spec.cap - spec.alpha) // 128)
    tiles = int(comp.counters[0].item())
    assert heads * T <= tiles <= heads * T * T
    assert rkv.rkv_launch_count_for(comp.desc, spec.budget, spec.buffer, spec.alpha, rkv.RKV_STAGE_ALL) == 7

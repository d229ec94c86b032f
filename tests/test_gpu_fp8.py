"""GPU parity for 8-bit (E4M3) K/V caches: the stored codes are scored as the values they stand for, the compaction
moves bytes.  The oracle decodes the codes itself (from the format's definition) and evaluates Eq. 1-7 in double."""
import numpy as np
import pytest
import torch

import rkv_inputs as ri
from parity_util import check_batch, from_paged, random_block_table, to_paged
from test_gpu_parity import DEFAULTS, run_and_check, small_spec

pytestmark = pytest.mark.gpu

FP8 = torch.float8_e4m3fn
NAN_CODE = 0x7F


@pytest.fixture(scope="module")
def rkv():
    import paper_2505_24133_b200 as m
    m.lib()
    return m


def _stale_rows_to_nan(wl, lens):
    """Rows at or beyond a sequence's length hold the NaN code: nothing of them may reach a score."""
    for b, L in enumerate(lens):
        wl.k_cache.view(torch.uint8)[b, :, L:] = NAN_CODE
        wl.v_cache.view(torch.uint8)[b, :, L:] = NAN_CODE


@pytest.mark.parametrize("flags", [pytest.param(0, id="sym"), pytest.param(32, id="two-pass"), pytest.param(1, id="simt"),
                                   pytest.param(2, id="rowblock")])
@pytest.mark.parametrize("budget,buffer,lens", [(256, 64, [320, 300, 256, 257]), (1800, 128, [1928, 1900, 1801, 40]),
                                                (1536, 128, [1664, 1664, 1663, 1600])])
def test_fp8_caches_against_the_oracle(rkv, flags, budget, buffer, lens):
    """Every scoring route on 8-bit caches with bf16 queries, ragged lengths, stale rows full of NaN codes: scores and
    kept sets within the tolerances of the bf16 tests (the arithmetic is the same: bf16 products of exactly widened
    values, fp32 accumulation), compacted rows byte for byte."""
    spec = small_spec("fp8", batch=4, hkv=2, hq=8, budget=budget, buffer=buffer, dtype="fp8", span=32)
    wl = ri.make_workload(spec, device="cuda", seed=301 + budget, seq_lens=torch.tensor(lens))
    assert wl.k_cache.dtype == FP8 and wl.q_window.dtype == torch.bfloat16
    _stale_rows_to_nan(wl, lens)
    rep, comp = run_and_check(rkv, wl, flags=flags)
    print(rep.summary())
    assert rep.ok(), rep.errors
    assert rep.compressed_heads == 2 * sum(L > budget for L in lens)
    comp.check_status()


@pytest.mark.parametrize("T,beta", [(0.9, 1), (0.5, 8), (1.0, 1), (0.7, 3)])
def test_fp8_threshold_and_beta(rkv, T, beta):
    spec = small_spec("fp8_tb", batch=2, hkv=2, hq=8, budget=1024, buffer=128, dtype="fp8", span=32)
    wl = ri.make_workload(spec, device="cuda", seed=311)
    rep, comp = run_and_check(rkv, wl, T=T, beta=beta)
    print(rep.summary())
    assert rep.ok(), rep.errors
    comp.check_status()


@pytest.mark.parametrize("head_dim,hkv,hq", [(64, 2, 8), (256, 2, 8), (256, 3, 3)])
def test_fp8_head_dimensions(rkv, head_dim, hkv, hq):
    """64- to 256-byte rows: the CUDA-core scoring route on the widened keys, 4 to 16 vectors per row in the gather."""
    lens = [320, 299, 256]
    spec = small_spec("fp8_hd", batch=3, hkv=hkv, hq=hq, budget=256, buffer=64, dtype="fp8", head_dim=head_dim)
    wl = ri.make_workload(spec, device="cuda", seed=321 + head_dim, seq_lens=torch.tensor(lens))
    _stale_rows_to_nan(wl, lens)
    rep, comp = run_and_check(rkv, wl)
    print(rep.summary())
    assert rep.ok(), rep.errors
    assert rep.compressed_heads == 2 * hkv
    comp.check_status()


def test_fp8_call_equals_the_bf16_call_on_the_widened_values(rkv):
    """The 8-bit route differs from the bf16 route only in where the keys come from: on caches holding the same values
    both calls return the same index lists, the same scores and move the same rows."""
    spec = small_spec("fp8_eq", batch=3, hkv=2, hq=8, budget=1100, buffer=100, dtype="fp8", span=32)
    lens = [1200, 1150, 1101]
    wl = ri.make_workload(spec, device="cuda", seed=331, seq_lens=torch.tensor(lens))
    k16, v16 = wl.k_cache.to(torch.bfloat16), wl.v_cache.to(torch.bfloat16)
    seq16 = wl.seq_lens.clone()
    c8 = rkv.Compressor(3, 2, 8, spec.budget, spec.buffer, spec.alpha, 0.1, dtype=FP8, dump_scores=True)
    c16 = rkv.Compressor(3, 2, 8, spec.budget, spec.buffer, spec.alpha, 0.1, dtype=torch.bfloat16, dump_scores=True)
    k8_before = wl.k_cache.clone()
    i8 = c8.compress(wl.k_cache, wl.v_cache, wl.q_window, wl.seq_lens)
    i16 = c16.compress(k16, v16, wl.q_window, seq16)
    torch.cuda.synchronize()
    c8.check_status()
    assert torch.equal(i8, i16) and torch.equal(wl.seq_lens, seq16)
    n = spec.cap - spec.alpha
    # (column sums are accumulated with floating-point atomics: equal up to their order)
    assert torch.allclose(c8.scores[:, :, :, :n], c16.scores[:, :, :, :n], rtol=1e-5, atol=2e-6, equal_nan=True)
    b = spec.budget
    assert torch.equal(wl.k_cache[:, :, :b].to(torch.bfloat16).view(torch.int16), k16[:, :, :b].view(torch.int16))
    assert torch.equal(wl.v_cache[:, :, :b].to(torch.bfloat16).view(torch.int16), v16[:, :, :b].view(torch.int16))
    # rows beyond the budget are not touched
    assert torch.equal(wl.k_cache.view(torch.uint8)[:, :, b:], k8_before.view(torch.uint8)[:, :, b:])
    # workspace: the bf16 call's plus the widened keys
    extra = (3 * 2 * spec.cap + 128) * 128 * 2
    w8 = rkv.rkv_workspace_bytes(c8.desc, spec.budget, spec.buffer, spec.alpha)
    w16 = rkv.rkv_workspace_bytes(c16.desc, spec.budget, spec.buffer, spec.alpha)
    assert w8 == w16 + extra
    assert rkv.rkv_launch_count_for(c8.desc, spec.budget, spec.buffer, spec.alpha, rkv.RKV_STAGE_ALL) == \
        rkv.rkv_launch_count_for(c16.desc, spec.budget, spec.buffer, spec.alpha, rkv.RKV_STAGE_ALL) + 1


def test_fp8_paged_caches(rkv):
    """8-bit page pools (128 rows of head_dim bytes per page) behind a block table, foreign pages full of NaN codes."""
    budget, buffer, lens = 1920, 128, [2048, 2047, 1921, 100]
    spec = small_spec("fp8_paged", batch=4, hkv=2, hq=8, budget=budget, buffer=buffer, dtype="fp8", span=32)
    wl = ri.make_workload(spec, device="cuda", seed=341, seq_lens=torch.tensor(lens))
    k0, v0, q0, s0 = wl.k_cache.clone(), wl.v_cache.clone(), wl.q_window.clone(), wl.seq_lens.clone()
    pages = spec.cap // 128
    pool_pages = 4 * 2 * pages + 23
    table = random_block_table(4, 2, pages, pool_pages, seed=9)
    kp = to_paged(k0.view(torch.uint8), pool_pages, table, fill=NAN_CODE)
    vp = to_paged(v0.view(torch.uint8), pool_pages, table, fill=NAN_CODE)
    kp0 = kp.clone()
    comp = rkv.Compressor(4, 2, 8, budget, buffer, spec.alpha, spec.lam, dtype=FP8, dump_scores=True, block_table=table,
                          pool_pages=pool_pages)
    seq = s0.clone()
    idx = comp.compress(kp.view(FP8), vp.view(FP8), q0, seq)
    torch.cuda.synchronize()
    comp.check_status()
    k1, v1 = from_paged(kp, table).view(FP8), from_paged(vp, table).view(FP8)
    rep = check_batch(k0, v0, q0, s0, budget=budget, alpha=spec.alpha, lam=spec.lam, gpu_idx=idx, gpu_k=k1, gpu_v=v1,
                      gpu_seq=seq, gpu_scores=comp.scores, **DEFAULTS)
    print(rep.summary())
    assert rep.ok(), rep.errors
    assert rep.compressed_heads == 2 * 3
    owned = torch.zeros(pool_pages, dtype=torch.bool, device="cuda")
    owned[table.reshape(-1).long()] = True
    assert torch.equal(kp[~owned], kp0[~owned])
    ref = rkv.Compressor(4, 2, 8, budget, buffer, spec.alpha, spec.lam, dtype=FP8)
    ref_idx = ref.compress(wl.k_cache, wl.v_cache, wl.q_window, wl.seq_lens)
    torch.cuda.synchronize()
    assert torch.equal(ref_idx, idx) and torch.equal(wl.seq_lens, seq)


def test_fp8_append_push_and_host_entry_points(rkv):
    """Rows of head_dim bytes through rkv_append, bf16 queries through rkv_push_query, and the host-buffer entry."""
    spec = small_spec("fp8_io", batch=3, hkv=2, hq=8, budget=256, buffer=64, dtype="fp8")
    lens = [300, 256, 319]
    wl = ri.make_workload(spec, device="cuda", seed=351, seq_lens=torch.tensor(lens))
    comp = rkv.Compressor(3, 2, 8, spec.budget, spec.buffer, spec.alpha, 0.1, dtype=FP8)
    g = torch.Generator(device="cuda").manual_seed(5)
    k_new = torch.randn(3, 2, 128, device="cuda", generator=g).to(FP8)
    v_new = torch.randn(3, 2, 128, device="cuda", generator=g).to(FP8)
    k_before = wl.k_cache.view(torch.uint8).clone()
    assert rkv.rkv_append(comp.desc, wl.k_cache, wl.v_cache, k_new, v_new, wl.seq_lens, spec.budget, spec.buffer) == 0
    torch.cuda.synchronize()
    assert wl.seq_lens.tolist() == [L + 1 for L in lens]
    kb = wl.k_cache.view(torch.uint8)
    for b, L in enumerate(lens):
        assert torch.equal(kb[b, :, L], k_new.view(torch.uint8)[b])
        assert torch.equal(wl.v_cache.view(torch.uint8)[b, :, L], v_new.view(torch.uint8)[b])
        assert torch.equal(kb[b, :, :L], k_before[b, :, :L]) and torch.equal(kb[b, :, L + 1:], k_before[b, :, L + 1:])
    q_new = torch.randn(3, 8, 128, device="cuda", generator=g).to(torch.bfloat16)
    qw = wl.q_window.clone()
    assert rkv.rkv_push_query(comp.desc, qw, q_new, spec.alpha, 3) == 0
    torch.cuda.synchronize()
    assert torch.equal(qw[:, :, 3].view(torch.int16), q_new.view(torch.int16))
    assert torch.equal(qw[:, :, :3].view(torch.int16), wl.q_window[:, :, :3].view(torch.int16))
    # the host-buffer entry point against the device one
    hk, hv = (t.view(torch.uint8).cpu().pin_memory() for t in (wl.k_cache, wl.v_cache))
    hq, hs = wl.q_window.cpu().pin_memory(), wl.seq_lens.cpu().pin_memory()
    hidx = torch.empty(3, 2, spec.budget, dtype=torch.int32).pin_memory()
    ch = rkv.Compressor(3, 2, 8, spec.budget, spec.buffer, spec.alpha, 0.1, dtype=FP8, host_staging=True)
    ch.compress_host(hk, hv, hq, hs, hidx)
    idx = comp.compress(wl.k_cache, wl.v_cache, wl.q_window, wl.seq_lens)
    torch.cuda.synchronize()
    assert torch.equal(hidx, idx.cpu()) and torch.equal(hs, wl.seq_lens.cpu())
    b = spec.budget
    assert torch.equal(hk[:, :, :b], wl.k_cache.view(torch.uint8)[:, :, :b].cpu())
    assert torch.equal(hv[:, :, :b], wl.v_cache.view(torch.uint8)[:, :, :b].cpu())


@pytest.mark.parametrize("hkv,hq,budget,buffer,lens", [(2, 8, 300, 84, [384, 1, 0, 200, 129]),
                                                       (1, 7, 4096, 128, [4224, 1, 0, 3000, 129]),
                                                       (2, 10, 1920, 128, [2048, 2047, 1921, 100, 128])])
def test_fp8_decode_attention_matches_the_oracle(rkv, hkv, hq, budget, buffer, lens):
    """Section 3.1's decode step over 8-bit caches (bf16 queries): the codes are widened on their way to the tensor
    cores, so the result is the attention over the values they stand for; ragged lengths, an empty and a one-token
    cache, stale rows full of NaN codes, one to several splits per head."""
    import oracle
    spec = small_spec("fp8_att", batch=5, hkv=hkv, hq=hq, budget=budget, buffer=buffer, dtype="fp8")
    wl = ri.make_workload(spec, device="cuda", seed=361 + hq, seq_lens=torch.tensor(lens))
    _stale_rows_to_nan(wl, lens)
    g = torch.Generator(device="cuda").manual_seed(7)
    q_new = torch.randn(5, hq, 128, generator=g, device="cuda").to(torch.bfloat16)
    comp = rkv.Compressor(5, hkv, hq, budget, buffer, spec.alpha, 0.1, dtype=FP8)
    assert rkv.rkv_decode_workspace_bytes(comp.desc, budget, buffer) <= comp.workspace.numel()
    out = torch.full((5, hq, 128), 7.0, dtype=torch.float32, device="cuda")
    rc = rkv.rkv_decode_attention(comp.desc, wl.k_cache, wl.v_cache, q_new, wl.seq_lens, out, budget, buffer)
    assert rc == rkv.RKV_OK, rkv.rkv_status_string(rc)
    torch.cuda.synchronize()
    comp.check_status()
    K = np.nan_to_num(oracle.e4m3_to_f32(wl.k_cache.view(torch.uint8).cpu().numpy()), nan=0.0)
    V = np.nan_to_num(oracle.e4m3_to_f32(wl.v_cache.view(torch.uint8).cpu().numpy()), nan=0.0)
    ref = oracle.oracle_decode_attention(K, V, q_new.float().cpu().numpy(), np.array(lens, dtype=np.int32))
    got = out.cpu().numpy().astype(np.float64)
    assert np.isfinite(got).all()
    scale = np.maximum(np.abs(ref).max(axis=-1, keepdims=True), 1e-30)
    assert (np.abs(got - ref) <= 1e-3 * scale + 1e-7).all(), float((np.abs(got - ref) / scale).max())
    for b, L in enumerate(lens):
        if L == 0:
            assert not got[b].any()                           # empty cache: zero rows


def test_fp8_decode_attention_paged_equals_contiguous(rkv):
    """The same call through a block table over 8-bit page pools: bit for bit the result on the contiguous caches."""
    spec = small_spec("fp8_att_paged", batch=4, hkv=1, hq=8, budget=896, buffer=128, dtype="fp8")
    lens = [1024, 127, 129, 700]
    wl = ri.make_workload(spec, device="cuda", seed=371, seq_lens=torch.tensor(lens))
    pages, pool_pages = spec.cap // 128, 4 * 8 + 5
    table = random_block_table(4, 1, pages, pool_pages, seed=14)
    kp = to_paged(wl.k_cache.view(torch.uint8), pool_pages, table, fill=NAN_CODE).view(FP8)
    vp = to_paged(wl.v_cache.view(torch.uint8), pool_pages, table, fill=NAN_CODE).view(FP8)
    g = torch.Generator(device="cuda").manual_seed(4)
    q_new = torch.randn(4, 8, 128, generator=g, device="cuda").to(torch.bfloat16)
    outs = []
    for k, v, kw in ((wl.k_cache, wl.v_cache, {}), (kp, vp, dict(block_table=table, pool_pages=pool_pages))):
        comp = rkv.Compressor(4, 1, 8, spec.budget, spec.buffer, spec.alpha, 0.1, dtype=FP8, **kw)
        out = torch.empty(4, 8, 128, dtype=torch.float32, device="cuda")
        assert rkv.rkv_decode_attention(comp.desc, k, v, q_new, wl.seq_lens, out, spec.budget, spec.buffer) == rkv.RKV_OK
        torch.cuda.synchronize()
        comp.check_status()
        outs.append(out)
    assert torch.equal(outs[0], outs[1])


def test_fp8_every_code_through_the_attention_and_the_widening_kernels(rkv):
    """All 254 finite E4M3 codes, subnormals and both zeros included, pass through the kernels' own decode exactly:
    with a one-token cache the attention's output row IS the value row (weight 1), and a compression call on keys made
    of every code agrees with the oracle's decode of them (the widening kernel feeds every scoring stage)."""
    import oracle
    codes = torch.arange(256, dtype=torch.uint8)
    codes[0x7F], codes[0xFF] = 0x7E, 0xFE                     # the two NaN codes: replaced by the largest finite ones
    v = torch.zeros(2, 1, 128, 128, dtype=torch.uint8)
    v[0, 0, 0], v[1, 0, 0] = codes[:128], codes[128:]
    k = torch.full((2, 1, 128, 128), 0x38, dtype=torch.uint8)                 # keys: all ones
    lens = torch.tensor([1, 1], dtype=torch.int32, device="cuda")
    d = rkv.rkv_desc_default()
    d.batch, d.n_kv_heads, d.n_q_heads, d.dtype = 2, 1, 4, rkv.RKV_FP8_E4M3
    q_new = torch.randn(2, 4, 128, device="cuda").to(torch.bfloat16)
    out = torch.empty(2, 4, 128, dtype=torch.float32, device="cuda")
    need = rkv.rkv_decode_workspace_bytes(d, 100, 28)
    ws = torch.empty(max(need, 256), dtype=torch.uint8, device="cuda")
    d.workspace, d.workspace_bytes = ws.data_ptr(), ws.numel()
    rc = rkv.rkv_decode_attention(d, k.cuda().view(FP8), v.cuda().view(FP8), q_new, lens, out, 100, 28)
    assert rc == rkv.RKV_OK
    torch.cuda.synchronize()
    want = oracle.e4m3_to_f32(codes.numpy())
    got = out.cpu().numpy()
    for g in range(4):
        assert np.array_equal(got[0, g], want[:128]) and np.array_equal(got[1, g], want[128:])
    # keys holding every code, through the widening kernel and a whole compression call
    spec = small_spec("fp8_codes", batch=1, hkv=1, hq=4, budget=200, buffer=56, dtype="fp8")
    wl = ri.make_workload(spec, device="cuda", seed=381)
    kb = wl.k_cache.view(torch.uint8)
    gen = torch.Generator().manual_seed(3)
    kb[0, 0, :64] = codes[torch.randint(0, 256, (64, 128), generator=gen)].cuda()
    rep, comp = run_and_check(rkv, wl)
    assert rep.ok(), rep.errors


@pytest.mark.parametrize("dtype,head_dim", [("fp8", 128), ("bf16", 64)])
def test_scoring_copy_with_budgets_and_pages(rkv, dtype, head_dim):
    """The prep kernel that writes the scoring copy itself (8-bit codes of 128 dimensions, bf16 keys of 64; capacity a
    whole number of tiles), together with per-sequence budgets and a block table: the stored tiles are fetched through
    the table, the copy is contiguous, the compaction moves the stored rows page by page."""
    budget, buffer = 896, 128
    lens = [1024, 1000, 600, 1024]
    budgets = [896, 700, 896, 512]
    spec = small_spec("copy_bp", batch=4, hkv=2, hq=8, budget=budget, buffer=buffer, dtype=dtype, head_dim=head_dim, span=32)
    wl = ri.make_workload(spec, device="cuda", seed=391 + head_dim, seq_lens=torch.tensor(lens))
    k0, v0, q0, s0 = wl.k_cache.clone(), wl.v_cache.clone(), wl.q_window.clone(), wl.seq_lens.clone()
    pages, pool_pages = spec.cap // 128, 4 * 2 * 8 + 9
    table = random_block_table(4, 2, pages, pool_pages, seed=15)
    raw = torch.uint8 if dtype == "fp8" else torch.int16
    fill = NAN_CODE if dtype == "fp8" else 0x7FC0                    # NaN patterns in the pages nobody owns
    kp = to_paged(k0.view(raw), pool_pages, table, fill=fill).view(k0.dtype)
    vp = to_paged(v0.view(raw), pool_pages, table, fill=fill).view(v0.dtype)
    comp = rkv.Compressor(4, 2, 8, budget, buffer, spec.alpha, spec.lam, dtype=spec.torch_dtype, head_dim=head_dim,
                          dump_scores=True, block_table=table, pool_pages=pool_pages, budgets=torch.tensor(budgets))
    seq = s0.clone()
    idx = comp.compress(kp, vp, q0, seq)
    torch.cuda.synchronize()
    comp.check_status()
    k1 = from_paged(kp.view(raw), table).view(k0.dtype)
    v1 = from_paged(vp.view(raw), table).view(v0.dtype)
    rep = check_batch(k0, v0, q0, s0, budget=budget, alpha=spec.alpha, lam=spec.lam, gpu_idx=idx, gpu_k=k1, gpu_v=v1,
                      gpu_seq=seq, gpu_scores=comp.scores, budgets=budgets, **DEFAULTS)
    print(rep.summary())
    assert rep.ok(), rep.errors
    assert rep.compressed_heads == 2 * 3
    assert seq.tolist() == [896, 700, 600, 512]

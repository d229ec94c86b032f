"""The decode-step updates around the compression (rkv_append, rkv_push_query) against the oracle, and one whole
decode segment -- appends until the buffer is full, then the compression -- eagerly and as one CUDA graph."""
import numpy as np
import pytest
import torch

import oracle
import rkv_inputs as ri
from parity_util import check_batch, from_paged, random_block_table, raw_rows, to_paged

pytestmark = pytest.mark.gpu


@pytest.fixture(scope="module")
def rkv():
    from paper_2505_24133_b200 import build as b
    b.build()
    import paper_2505_24133_b200 as r
    assert r.lib() is not None
    return r


def _spec(dtype="bf16", batch=3, budget=256, buffer=64, alpha=8):
    return ri.CacheSpec("decode", 1, batch, 2, 8, 128, budget, buffer, alpha, 0.1, dtype, 16, 0.3, 0.05, 4, 8.0)


def _desc(rkv, spec, status):
    d = rkv.rkv_desc_default()
    d.batch, d.n_kv_heads, d.n_q_heads = spec.folded_batch, spec.n_kv_heads, spec.n_q_heads
    d.dtype = rkv.RKV_BF16 if spec.dtype == "bf16" else rkv.RKV_F32
    d.device_status = status.data_ptr()
    return d


@pytest.mark.parametrize("dtype", ["bf16", "f32"])
def test_append_matches_oracle_bit_for_bit(rkv, dtype):
    spec = _spec(dtype)
    lens = torch.tensor([spec.budget, spec.cap, 17])                 # the second cache is full: refused, flagged
    wl = ri.make_workload(spec, device="cuda", seed=211, seq_lens=lens)
    gen = torch.Generator(device="cuda").manual_seed(5)
    k_new = torch.randn(spec.folded_batch, spec.n_kv_heads, 128, device="cuda", generator=gen).to(wl.k_cache.dtype)
    v_new = torch.randn(spec.folded_batch, spec.n_kv_heads, 128, device="cuda", generator=gen).to(wl.k_cache.dtype)
    status = torch.zeros(1, dtype=torch.int32, device="cuda")
    want_k, want_v, want_s = oracle.oracle_append(raw_rows(wl.k_cache), raw_rows(wl.v_cache), raw_rows(k_new),
                                                  raw_rows(v_new), wl.seq_lens.cpu().numpy())
    rc = rkv.rkv_append(_desc(rkv, spec, status), wl.k_cache, wl.v_cache, k_new, v_new, wl.seq_lens, spec.budget,
                        spec.buffer)
    assert rc == rkv.RKV_OK, rkv.rkv_status_string(rc)
    torch.cuda.synchronize()
    assert np.array_equal(raw_rows(wl.k_cache), want_k) and np.array_equal(raw_rows(wl.v_cache), want_v)
    assert wl.seq_lens.cpu().numpy().tolist() == want_s.tolist() == [spec.budget + 1, spec.cap, 18]
    assert int(status.item()) == 1                                    # RKV_ERR_INVALID_ARG: a full cache was met


def test_push_query_matches_oracle_and_rejects_bad_slots(rkv):
    spec = _spec()
    wl = ri.make_workload(spec, device="cuda", seed=212)
    status = torch.zeros(1, dtype=torch.int32, device="cuda")
    d = _desc(rkv, spec, status)
    gen = torch.Generator(device="cuda").manual_seed(6)
    want = raw_rows(wl.q_window)
    for step in range(spec.alpha + 3):
        q_new = torch.randn(spec.folded_batch, spec.n_q_heads, 128, device="cuda", generator=gen).to(torch.bfloat16)
        want = oracle.oracle_push_query(want, raw_rows(q_new), step % spec.alpha)
        assert rkv.rkv_push_query(d, wl.q_window, q_new, spec.alpha, step % spec.alpha) == rkv.RKV_OK
    torch.cuda.synchronize()
    assert np.array_equal(raw_rows(wl.q_window), want)
    assert rkv.rkv_push_query(d, wl.q_window, q_new, spec.alpha, spec.alpha) == 1       # slot out of range
    assert rkv.rkv_push_query(d, wl.q_window, q_new, spec.alpha, -1) == 1


def test_decode_segment_eager_and_as_one_cuda_graph(rkv):
    """budget cached tokens, then `buffer` decode steps (append + query push), then the compression: the state after
    the segment agrees with the oracle driven by the same inputs, and a CUDA graph of the whole segment replays to
    the same bits."""
    spec = _spec(batch=2, budget=256, buffer=32)
    steps = spec.buffer
    wl = ri.make_workload(spec, device="cuda", seed=213, seq_lens=torch.tensor([spec.budget, spec.budget]))
    gen = torch.Generator(device="cuda").manual_seed(7)
    B, H, Hq = spec.folded_batch, spec.n_kv_heads, spec.n_q_heads
    # new tokens: every fourth repeats an earlier key with a little noise, so that the redundancy term has work to do
    k_steps = torch.randn(steps, B, H, 128, device="cuda", generator=gen)
    k_steps[3::4] = k_steps[0:steps:4][: k_steps[3::4].shape[0]] + 0.05 * torch.randn_like(k_steps[3::4])
    k_steps = k_steps.to(torch.bfloat16)
    v_steps = torch.randn(steps, B, H, 128, device="cuda", generator=gen).to(torch.bfloat16)
    q_steps = (2.0 * torch.randn(steps, B, Hq, 128, device="cuda", generator=gen)).to(torch.bfloat16)
    k0, v0, q0, s0 = wl.k_cache.clone(), wl.v_cache.clone(), wl.q_window.clone(), wl.seq_lens.clone()
    comp = rkv.Compressor(B, H, Hq, spec.budget, spec.buffer, spec.alpha, spec.lam)

    def segment():
        for t in range(steps):
            assert rkv.rkv_append(comp.desc, wl.k_cache, wl.v_cache, k_steps[t], v_steps[t], wl.seq_lens, spec.budget,
                                  spec.buffer) == rkv.RKV_OK
            assert rkv.rkv_push_query(comp.desc, wl.q_window, q_steps[t], spec.alpha, t % spec.alpha) == rkv.RKV_OK
        comp.compress(wl.k_cache, wl.v_cache, wl.q_window, wl.seq_lens)

    segment()
    torch.cuda.synchronize()
    comp.check_status()
    # the oracle's view of the same segment, up to the compression's inputs
    ok_, ov_, os_ = raw_rows(k0), raw_rows(v0), s0.cpu().numpy()
    oq = raw_rows(q0)
    for t in range(steps):
        ok_, ov_, os_ = oracle.oracle_append(ok_, ov_, raw_rows(k_steps[t]), raw_rows(v_steps[t]), os_)
        oq = oracle.oracle_push_query(oq, raw_rows(q_steps[t]), t % spec.alpha)
    assert os_.tolist() == [spec.cap, spec.cap]
    as_bf16 = lambda a: torch.from_numpy(a.view(np.int16).copy()).view(torch.bfloat16).cuda()
    rep = check_batch(as_bf16(ok_), as_bf16(ov_), as_bf16(oq), torch.from_numpy(os_), budget=spec.budget,
                      alpha=spec.alpha, lam=spec.lam, W=4, beta=1, T=0.5, eps=1e-8, gpu_idx=comp.out_idx,
                      gpu_k=wl.k_cache, gpu_v=wl.v_cache, gpu_seq=wl.seq_lens)
    assert rep.ok(), rep.errors
    assert rep.compressed_heads == B * H and wl.seq_lens.tolist() == [spec.budget, spec.budget]
    eager = (comp.out_idx.clone(), wl.k_cache.clone(), wl.v_cache.clone(), wl.q_window.clone())

    # the same segment as one graph
    def restore():
        wl.k_cache.copy_(k0), wl.v_cache.copy_(v0), wl.q_window.copy_(q0), wl.seq_lens.copy_(s0)

    restore()
    graph, side = torch.cuda.CUDAGraph(), torch.cuda.Stream()
    side.wait_stream(torch.cuda.current_stream())
    with torch.cuda.graph(graph, stream=side):
        segment()
    torch.cuda.synchronize()
    restore()
    graph.replay()
    torch.cuda.synchronize()
    comp.check_status()
    nb = spec.budget
    assert torch.equal(comp.out_idx, eager[0]) and wl.seq_lens.tolist() == [spec.budget, spec.budget]
    assert torch.equal(wl.k_cache[:, :, :nb].view(torch.int16), eager[1][:, :, :nb].view(torch.int16))
    assert torch.equal(wl.v_cache[:, :, :nb].view(torch.int16), eager[2][:, :, :nb].view(torch.int16))
    assert torch.equal(wl.q_window.view(torch.int16), eager[3].view(torch.int16))


# ----------------------------------------------------------------------------- decode-step attention over the cache
@pytest.mark.parametrize("dtype", ["bf16", "f32"])
@pytest.mark.parametrize("hkv,hq", [(2, 2), (2, 8), (2, 10), (1, 7), (1, 8), (3, 9)])
def test_decode_attention_matches_the_oracle(rkv, dtype, hkv, hq):
    """Section 3.1's decode step, Eq. 1 with one query row: all group sizes the kernel serves, ragged lengths (a full
    cache, a single token, an empty cache, a length that ends inside a tile), rows beyond the length filled with NaN
    to prove they are never read.  Few head-problems: the rows of a head are cut into splits and merged."""
    spec = ri.CacheSpec("att", 1, 5, hkv, hq, 128, 300, 84, 8, 0.1, dtype, 16, 0.3, 0.05, 4, 8.0)
    lens = [spec.cap, 1, 0, 200, 129]
    wl = ri.make_workload(spec, device="cuda", seed=301 + hq, seq_lens=torch.tensor(lens))
    for b, L in enumerate(lens):
        wl.k_cache[b, :, L:] = float("nan")
        wl.v_cache[b, :, L:] = float("nan")
    g = torch.Generator(device="cuda").manual_seed(5)
    q_new = torch.randn(5, hq, 128, generator=g, device="cuda").to(spec.torch_dtype)
    comp = rkv.Compressor(5, hkv, hq, spec.budget, spec.buffer, spec.alpha, 0.1, dtype=spec.torch_dtype)
    assert rkv.rkv_decode_workspace_bytes(comp.desc, spec.budget, spec.buffer) <= comp.workspace.numel()
    out = torch.full((5, hq, 128), 7.0, dtype=torch.float32, device="cuda")
    rc = rkv.rkv_decode_attention(comp.desc, wl.k_cache, wl.v_cache, q_new, wl.seq_lens, out, spec.budget, spec.buffer)
    assert rc == rkv.RKV_OK, rkv.rkv_status_string(rc)
    torch.cuda.synchronize()
    comp.check_status()
    K, V = (torch.nan_to_num(t.float(), nan=0.0).cpu().numpy() for t in (wl.k_cache, wl.v_cache))
    ref = oracle.oracle_decode_attention(K, V, q_new.float().cpu().numpy(), np.array(lens, dtype=np.int32))
    got = out.cpu().numpy().astype(np.float64)
    assert np.isfinite(got).all()
    scale = np.maximum(np.abs(ref).max(axis=-1, keepdims=True), 1e-30)
    assert (np.abs(got - ref) <= 1e-3 * scale + 1e-7).all(), float((np.abs(got - ref) / scale).max())
    assert not got[2].any()                                   # empty cache: zero rows


def test_decode_attention_large_batch_single_split(rkv):
    """Enough head-problems for one block per head (no splits, no workspace): the Llama-8B group size at the cache
    size of the first benchmark configuration, checked on sampled sequences."""
    spec = ri.scaled(ri.SPECS["llama8b_b1"], layers=1, batch=80)
    lens = torch.randint(1, spec.cap + 1, (80,), generator=torch.Generator().manual_seed(9))
    lens[0], lens[1] = spec.cap, 1
    wl = ri.make_workload(spec, device="cuda", seed=311, seq_lens=lens)
    g = torch.Generator(device="cuda").manual_seed(6)
    q_new = torch.randn(80, spec.n_q_heads, 128, generator=g, device="cuda").to(torch.bfloat16)
    d = rkv.rkv_desc_default()
    d.batch, d.n_kv_heads, d.n_q_heads = 80, spec.n_kv_heads, spec.n_q_heads
    assert rkv.rkv_decode_workspace_bytes(d, spec.budget, spec.buffer) == 0
    out = torch.empty(80, spec.n_q_heads, 128, dtype=torch.float32, device="cuda")
    rc = rkv.rkv_decode_attention(d, wl.k_cache, wl.v_cache, q_new, wl.seq_lens, out, spec.budget, spec.buffer)
    assert rc == rkv.RKV_OK, rkv.rkv_status_string(rc)
    torch.cuda.synchronize()
    rows = [0, 1, 17, 42, 79]
    ref = oracle.oracle_decode_attention(wl.k_cache[rows].float().cpu().numpy(), wl.v_cache[rows].float().cpu().numpy(),
                                         q_new[rows].float().cpu().numpy(), lens[rows].numpy().astype(np.int32))
    got = out[rows].cpu().numpy().astype(np.float64)
    scale = np.maximum(np.abs(ref).max(axis=-1, keepdims=True), 1e-30)
    assert (np.abs(got - ref) <= 1e-3 * scale + 1e-7).all()


@pytest.mark.parametrize("hkv,hq,batch", [(2, 10, 3), (1, 7, 40), (4, 32, 2), (1, 6, 600)])
def test_decode_attention_tensor_core_route_large_cache(rkv, hkv, hq, batch):
    """Query groups of 5 to 8 at the largest cache size of the configurations (33 key tiles, so every head is cut into
    three or more splits, whatever the batch), random lengths with a full, a one-token and an empty cache among them,
    stale rows full of NaN; checked on sampled sequences."""
    spec = ri.CacheSpec("att_tc", 1, batch, hkv, hq, 128, 4096, 128, 8, 0.1, "bf16", 32, 0.3, 0.05, 4, 8.0)
    lens = torch.randint(1, spec.cap + 1, (batch,), generator=torch.Generator().manual_seed(13 + hq))
    lens[0], lens[1] = spec.cap, 1
    if batch > 2:
        lens[2] = 0
    wl = ri.make_workload(spec, device="cuda", seed=341 + hq, seq_lens=lens)
    for b in range(batch):
        wl.k_cache[b, :, int(lens[b]):] = float("nan")
        wl.v_cache[b, :, int(lens[b]):] = float("nan")
    g = torch.Generator(device="cuda").manual_seed(8)
    q_new = torch.randn(batch, hq, 128, generator=g, device="cuda").to(torch.bfloat16)
    d = rkv.rkv_desc_default()
    d.batch, d.n_kv_heads, d.n_q_heads = batch, hkv, hq
    status = torch.zeros(1, dtype=torch.int32, device="cuda")
    d.device_status = status.data_ptr()
    need = rkv.rkv_decode_workspace_bytes(d, spec.budget, spec.buffer)
    assert need > 0                                    # 33 tiles never fit one block's 15
    ws = torch.empty(need, dtype=torch.uint8, device="cuda")
    d.workspace, d.workspace_bytes = ws.data_ptr(), need
    out = torch.full((batch, hq, 128), 7.0, dtype=torch.float32, device="cuda")
    rc = rkv.rkv_decode_attention(d, wl.k_cache, wl.v_cache, q_new, wl.seq_lens, out, spec.budget, spec.buffer)
    assert rc == rkv.RKV_OK, rkv.rkv_status_string(rc)
    torch.cuda.synchronize()
    assert int(status.item()) == 0
    rows = sorted(set([0, 1, min(2, batch - 1), batch // 2, batch - 1]))
    K, V = (torch.nan_to_num(t[rows].float(), nan=0.0).cpu().numpy() for t in (wl.k_cache, wl.v_cache))
    ref = oracle.oracle_decode_attention(K, V, q_new[rows].float().cpu().numpy(), lens[rows].numpy().astype(np.int32))
    got = out[rows].cpu().numpy().astype(np.float64)
    assert np.isfinite(out.cpu().numpy()).all()
    scale = np.maximum(np.abs(ref).max(axis=-1, keepdims=True), 1e-30)
    assert (np.abs(got - ref) <= 1e-3 * scale + 1e-7).all(), float((np.abs(got - ref) / scale).max())
    if batch > 2:
        assert not out[2].any()


def test_decode_attention_tensor_core_route_paged(rkv):
    """The tensor-core kernel through a block table (G = 8)."""
    spec = ri.CacheSpec("att_tc_paged", 1, 4, 1, 8, 128, 896, 128, 8, 0.1, "bf16", 16, 0.3, 0.05, 4, 8.0)
    lens = [1024, 127, 129, 700]
    wl = ri.make_workload(spec, device="cuda", seed=351, seq_lens=torch.tensor(lens))
    pages, pool_pages = spec.cap // 128, 4 * 8 + 5
    table = random_block_table(4, 1, pages, pool_pages, seed=12)
    kp, vp = to_paged(wl.k_cache, pool_pages, table), to_paged(wl.v_cache, pool_pages, table)     # foreign pages: NaN
    comp = rkv.Compressor(4, 1, 8, spec.budget, spec.buffer, spec.alpha, 0.1, block_table=table, pool_pages=pool_pages)
    g = torch.Generator(device="cuda").manual_seed(4)
    q_new = torch.randn(4, 8, 128, generator=g, device="cuda").to(torch.bfloat16)
    need = rkv.rkv_decode_workspace_bytes(comp.desc, spec.budget, spec.buffer)
    ws = torch.empty(max(need, 256), dtype=torch.uint8, device="cuda")
    comp.desc.workspace, comp.desc.workspace_bytes = ws.data_ptr(), ws.numel()
    out = torch.empty(4, 8, 128, dtype=torch.float32, device="cuda")
    assert rkv.rkv_decode_attention(comp.desc, kp, vp, q_new, wl.seq_lens, out, spec.budget, spec.buffer) == rkv.RKV_OK
    torch.cuda.synchronize()
    comp.check_status()
    ref = oracle.oracle_decode_attention(wl.k_cache.float().cpu().numpy(), wl.v_cache.float().cpu().numpy(),
                                         q_new.float().cpu().numpy(), np.array(lens, dtype=np.int32))
    got = out.cpu().numpy().astype(np.float64)
    scale = np.maximum(np.abs(ref).max(axis=-1, keepdims=True), 1e-30)
    assert (np.abs(got - ref) <= 1e-3 * scale + 1e-7).all(), float((np.abs(got - ref) / scale).max())


@pytest.mark.parametrize("hkv,hq,budget,buffer,lens", [(2, 8, 300, 84, [384, 1, 0, 200, 129]),
                                                       (1, 7, 4096, 128, [4224, 1, 0, 3000, 129]),
                                                       (8, 32, 1024, 128, [1152, 1151, 1000, 7, 128])])
def test_decode_attention_head_dimension_64(rkv, hkv, hq, budget, buffer, lens):
    """bf16 caches with 64-dimensional heads: the tensor-core kernel pads the tiles (and the queries) to 128 dimensions on
    their way to the tensor cores; Eq. 1's scale is 1 / sqrt(64); one to several splits; stale rows full of NaN."""
    spec = ri.CacheSpec("att64", 1, 5, hkv, hq, 64, budget, buffer, 8, 0.1, "bf16", 16, 0.3, 0.05, 4, 8.0)
    wl = ri.make_workload(spec, device="cuda", seed=361 + hq, seq_lens=torch.tensor(lens))
    for b, L in enumerate(lens):
        wl.k_cache[b, :, L:] = float("nan")
        wl.v_cache[b, :, L:] = float("nan")
    g = torch.Generator(device="cuda").manual_seed(9)
    q_new = torch.randn(5, hq, 64, generator=g, device="cuda").to(torch.bfloat16)
    comp = rkv.Compressor(5, hkv, hq, budget, buffer, spec.alpha, 0.1, head_dim=64)
    assert rkv.rkv_decode_workspace_bytes(comp.desc, budget, buffer) <= comp.workspace.numel()
    out = torch.full((5, hq, 64), 7.0, dtype=torch.float32, device="cuda")
    rc = rkv.rkv_decode_attention(comp.desc, wl.k_cache, wl.v_cache, q_new, wl.seq_lens, out, budget, buffer)
    assert rc == rkv.RKV_OK, rkv.rkv_status_string(rc)
    torch.cuda.synchronize()
    comp.check_status()
    K, V = (torch.nan_to_num(t.float(), nan=0.0).cpu().numpy() for t in (wl.k_cache, wl.v_cache))
    ref = oracle.oracle_decode_attention(K, V, q_new.float().cpu().numpy(), np.array(lens, dtype=np.int32))
    got = out.cpu().numpy().astype(np.float64)
    assert np.isfinite(got).all()
    scale = np.maximum(np.abs(ref).max(axis=-1, keepdims=True), 1e-30)
    assert (np.abs(got - ref) <= 1e-3 * scale + 1e-7).all(), float((np.abs(got - ref) / scale).max())
    for b, L in enumerate(lens):
        if L == 0:
            assert not got[b].any()
    # fp32 caches of 64 dimensions are not served
    d = rkv.rkv_desc_default()
    d.batch, d.n_kv_heads, d.n_q_heads, d.head_dim, d.dtype = 5, hkv, hq, 64, rkv.RKV_F32
    assert rkv.rkv_decode_attention(d, wl.k_cache, wl.v_cache, q_new, wl.seq_lens, out, budget, buffer) == 2


def test_decode_attention_argument_checks(rkv):
    d = rkv.rkv_desc_default()
    d.batch, d.n_kv_heads, d.n_q_heads = 2, 1, 9           # G = 9: beyond what one block serves
    assert rkv.rkv_decode_attention(d, 0x20000, 0x20000, 0x20000, 0x30000, 0x40000, 256, 64, 0) == 2
    d.n_q_heads = 4
    assert rkv.rkv_decode_attention(d, 0x20000, 0x20000, 0x20000, 0x30000, 0, 256, 64, 0) == 1       # null output
    assert rkv.rkv_decode_attention(d, 0x20000, 0x20000, 0x20000, 0x30000, 0x40000, 256, 64, 0) == 3  # splits need a workspace


# ----------------------------------------------------------------------------- paged caches in the decode-step calls
@pytest.mark.parametrize("dtype", ["bf16", "f32"])
def test_paged_append_and_attention(rkv, dtype):
    """rkv_append and rkv_decode_attention through a block table: the appended rows land in the right pages (compared
    with the oracle's append after un-paging), and the attention over the paged caches equals the oracle's over the
    same rows (tiles of 56 rows cross the 128-row pages)."""
    spec = ri.CacheSpec("paged_dec", 1, 4, 2, 8, 128, 256, 128, 8, 0.1, dtype, 16, 0.3, 0.05, 4, 8.0)
    lens = [300, 127, 128, 383]
    wl = ri.make_workload(spec, device="cuda", seed=331, seq_lens=torch.tensor(lens))
    pages, pool_pages = spec.cap // 128, 4 * 2 * 3 + 11
    table = random_block_table(4, 2, pages, pool_pages, seed=11)
    kp, vp = to_paged(wl.k_cache, pool_pages, table, fill=0.0), to_paged(wl.v_cache, pool_pages, table, fill=0.0)
    comp = rkv.Compressor(4, 2, 8, spec.budget, spec.buffer, spec.alpha, 0.1, dtype=spec.torch_dtype, block_table=table,
                          pool_pages=pool_pages)
    g = torch.Generator(device="cuda").manual_seed(3)
    k_new = torch.randn(4, 2, 128, generator=g, device="cuda").to(spec.torch_dtype)
    v_new = torch.randn(4, 2, 128, generator=g, device="cuda").to(spec.torch_dtype)
    q_new = torch.randn(4, 8, 128, generator=g, device="cuda").to(spec.torch_dtype)
    seq = wl.seq_lens.clone()
    assert rkv.rkv_append(comp.desc, kp, vp, k_new, v_new, seq, spec.budget, spec.buffer) == rkv.RKV_OK
    torch.cuda.synchronize()
    k_ref, v_ref, s_ref = oracle.oracle_append(raw_rows(wl.k_cache), raw_rows(wl.v_cache), raw_rows(k_new), raw_rows(v_new),
                                               np.array(lens, dtype=np.int32))
    assert seq.tolist() == s_ref.tolist() == [301, 128, 129, 384]
    for b, L in enumerate(s_ref.tolist()):
        assert np.array_equal(raw_rows(from_paged(kp, table))[b, :, :L], k_ref[b, :, :L])
        assert np.array_equal(raw_rows(from_paged(vp, table))[b, :, :L], v_ref[b, :, :L])
    out = torch.empty(4, 8, 128, dtype=torch.float32, device="cuda")
    assert rkv.rkv_decode_attention(comp.desc, kp, vp, q_new, seq, out, spec.budget, spec.buffer) == rkv.RKV_OK
    torch.cuda.synchronize()
    comp.check_status()
    ref = oracle.oracle_decode_attention(from_paged(kp, table).float().cpu().numpy(), from_paged(vp, table).float().cpu().numpy(),
                                         q_new.float().cpu().numpy(), seq.cpu().numpy())
    got = out.cpu().numpy().astype(np.float64)
    scale = np.maximum(np.abs(ref).max(axis=-1, keepdims=True), 1e-30)
    assert (np.abs(got - ref) <= 1e-3 * scale + 1e-7).all()

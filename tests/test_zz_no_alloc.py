"""rkv_compress_static: the compression step for callers that cannot allocate a workspace.

Some users of this library are not allowed to call cudaMalloc when the decode buffer fills: a serving engine
whose block pool already owns the whole GPU, code running inside another framework's callback, a latency-bound
loop that must stay off the driver's allocation lock.  rkv_compress_static serves them from a 32 MiB scratch
array that is part of the library itself.  This file checks, through the C ABI, that it gives exactly what
rkv_compress_ex gives with a caller-allocated workspace -- on two calls in a row, because the array keeps the
first call's contents and the second must not be disturbed by them.

The file name sorts last on purpose: in a run that stops at the first failure every other test has already run.
It passes on its own in a fresh process as well (the first call on a device does the entry point's set-up).
"""
import pytest
import torch

import rkv_inputs as ri

pytestmark = pytest.mark.gpu


@pytest.fixture(scope="module")
def rkv():
    from paper_2505_24133_b200 import build as b
    b.build()
    import paper_2505_24133_b200 as r
    assert r.lib() is not None
    return r


def _spec(name, batch, budget, buffer):
    return ri.CacheSpec(name, 1, batch, 2, 8, 128, budget, buffer, 8, 0.1, "bf16", 16, 0.3, 0.05, 4, 8.0)


def _run_both(rkv, spec, seed, seq_lens, check_memory=False):
    """One compression of the same seeded caches through rkv_compress_ex (torch-allocated workspace) and through
    rkv_compress_static (no workspace); returns both results."""
    a = ri.make_workload(spec, device="cuda", seed=seed, seq_lens=seq_lens)
    b = ri.make_workload(spec, device="cuda", seed=seed, seq_lens=seq_lens)
    ref = rkv.Compressor(spec.folded_batch, spec.n_kv_heads, spec.n_q_heads, spec.budget, spec.buffer, spec.alpha,
                         spec.lam)
    ref_idx = ref.compress(a.k_cache, a.v_cache, a.q_window, a.seq_lens)
    torch.cuda.synchronize()
    ref.check_status()

    d = rkv.rkv_desc_default()
    d.batch, d.n_kv_heads, d.n_q_heads = spec.folded_batch, spec.n_kv_heads, spec.n_q_heads
    status = torch.zeros(1, dtype=torch.int32, device="cuda")
    d.device_status = status.data_ptr()
    assert d.workspace is None and d.workspace_bytes == 0          # nothing allocated for scratch
    idx = torch.full((spec.folded_batch, spec.n_kv_heads, spec.budget), -7, dtype=torch.int32, device="cuda")
    if check_memory:
        # the descriptor's workspace fields are ignored: a bogus, far too small one must make no difference, and
        # the pointer is never dereferenced
        d.workspace, d.workspace_bytes = 0x1000, 16
        torch.cuda.synchronize()
        free_before, _ = torch.cuda.mem_get_info()
    rc = rkv.rkv_compress_static(d, b.k_cache, b.v_cache, b.q_window, b.seq_lens, spec.budget, spec.buffer,
                                 spec.alpha, spec.lam, idx)
    assert rc == rkv.RKV_OK, rkv.rkv_status_string(rc)
    torch.cuda.synchronize()
    if check_memory:
        # a warm call (the device image is loaded, the array's address cached) takes no device memory at all
        free_after, _ = torch.cuda.mem_get_info()
        assert free_after == free_before
    assert int(status.item()) == 0
    return (ref_idx, a), (idx, b)


def _assert_same(spec, ref, got):
    (ref_idx, a), (idx, b) = ref, got
    # the two entry points run the same kernels on the same inputs: index lists, new lengths and the compacted
    # rows agree bit for bit (the tolerance the stage-by-stage parity test uses)
    assert torch.equal(idx, ref_idx)
    assert torch.equal(b.seq_lens, a.seq_lens)
    nb = spec.budget
    assert torch.equal(b.k_cache[:, :, :nb].view(torch.int16), a.k_cache[:, :, :nb].view(torch.int16))
    assert torch.equal(b.v_cache[:, :, :nb].view(torch.int16), a.v_cache[:, :, :nb].view(torch.int16))


def test_static_scratch_matches_workspace_entry_point_twice_in_a_row(rkv):
    # first call: four tiles per head, every cache full
    big = _spec("static_a", batch=3, budget=384, buffer=128)
    ref, got = _run_both(rkv, big, seed=201, seq_lens=torch.tensor([512, 512, 512]))
    _assert_same(big, ref, got)
    assert got[1].seq_lens.tolist() == [384, 384, 384]
    # second call, straight after: another shape with shorter and ragged lengths (one sequence below the
    # budget, so Algorithm 1's guard leaves it alone), so that stale scores of the first call sit right
    # behind the rows this one uses
    small = _spec("static_b", batch=4, budget=200, buffer=60)
    ref, got = _run_both(rkv, small, seed=202, seq_lens=torch.tensor([260, 201, 150, 233]), check_memory=True)
    _assert_same(small, ref, got)
    assert got[1].seq_lens.tolist() == [200, 200, 150, 200]


def test_static_scratch_refuses_shapes_beyond_its_size(rkv):
    """A shape that needs more than the built-in array is turned down with RKV_ERR_WORKSPACE before any launch
    (the fake pointers below are never dereferenced)."""
    d = rkv.rkv_desc_default()
    d.batch, d.n_kv_heads, d.n_q_heads = 512, 8, 32
    assert rkv.rkv_workspace_bytes(d, 4096, 128, 8) > rkv.RKV_STATIC_SCRATCH_BYTES
    rc = rkv.rkv_compress_static(d, 0x20000, 0x20000, 0x20000, 0x30000, 4096, 128, 8, 0.1, 0x30000, 0)
    assert rc == 3, rkv.rkv_status_string(rc)
    d.n_q_heads = 30                                                   # an invalid shape keeps its own error code
    rc = rkv.rkv_compress_static(d, 0x20000, 0x20000, 0x20000, 0x30000, 4096, 128, 8, 0.1, 0x30000, 0)
    assert rc == 1, rkv.rkv_status_string(rc)

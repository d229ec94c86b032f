"""Host-side checks of the C-ABI library that need no GPU: it loads, exports every declared symbol, and
rejects host-detectable errors before any launch."""
import ctypes
import os
import re

import pytest

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))


@pytest.fixture(scope="module")
def rkv():
    from paper_2505_24133_b200 import build as b
    b.build()
    import paper_2505_24133_b200 as r
    return r


def test_library_exports_every_declared_symbol(rkv):
    header = open(os.path.join(ROOT, "include", "rkv.h")).read()
    names = re.findall(r"RKV_API\s+[\w\s\*]+?\b(rkv_\w+)\s*\(", header)
    assert len(names) >= 13
    lib = ctypes.CDLL(rkv.lib_path())
    for name in names:
        assert hasattr(lib, name), f"{name} is declared in include/rkv.h but not exported"


def test_desc_mirror_matches_the_c_struct(rkv):
    d = rkv.rkv_desc_default()
    assert (d.head_dim, d.dtype, d.pool_w, d.beta) == (128, rkv.RKV_BF16, 4, 1)
    assert abs(d.sim_threshold - 0.5) < 1e-7 and abs(d.eps - 1e-8) < 1e-15
    assert d.workspace is None and d.stage_events is None and d.flags == 0


def _desc(rkv, **kw):
    d = rkv.rkv_desc_default()
    d.batch, d.n_kv_heads, d.n_q_heads = 2, 8, 32
    for k, v in kw.items():
        setattr(d, k, v)
    return d


def test_workspace_size_rules(rkv):
    d = _desc(rkv)
    a = rkv.rkv_workspace_bytes(d, 1024, 128, 8)
    assert a > 0 and a % 256 == 0
    d2 = _desc(rkv, batch=4)
    assert rkv.rkv_workspace_bytes(d2, 1024, 128, 8) > a
    assert rkv.rkv_host_workspace_bytes(d, 1024, 128, 8) > a + 2 * 2 * 8 * 1152 * 256
    # invalid shapes give 0
    assert rkv.rkv_workspace_bytes(_desc(rkv, n_q_heads=30), 1024, 128, 8) == 0      # G not integral
    assert rkv.rkv_workspace_bytes(_desc(rkv, head_dim=96), 1024, 128, 8) == 0
    # (on the CUDA-core route; on the default route head dimension 64 carries a padded copy of the keys)
    assert 0 < rkv.rkv_workspace_bytes(_desc(rkv, head_dim=64, flags=rkv.RKV_FLAG_SIMT_SCORES), 1024, 128, 8) < \
        rkv.rkv_workspace_bytes(_desc(rkv, head_dim=256), 1024, 128, 8)
    assert rkv.rkv_workspace_bytes(d, 8, 128, 8) == 0                                # budget <= alpha
    assert rkv.rkv_workspace_bytes(d, 8192, 128, 8) == 0                             # cap > RKV_MAX_CAP
    assert rkv.rkv_workspace_bytes(_desc(rkv, n_q_heads=8 * 17), 1024, 128, 8) == 0  # G * alpha = 136 > 112


@pytest.mark.parametrize("case,want", [
    ("null_k", 1), ("misaligned_q", 1), ("lambda", 1), ("alpha0", 1), ("budget_le_alpha", 1), ("buffer0", 1),
    ("threshold", 1), ("group", 1), ("head_dim", 2), ("dtype", 2), ("no_workspace", 3), ("small_workspace", 3),
    ("stage_mask", 1),
])
def test_host_detectable_errors_return_before_any_launch(rkv, case, want):
    """No CUDA call is made on these paths, so they run without a GPU; fake non-null pointers are never
    dereferenced."""
    d = _desc(rkv)
    d.workspace, d.workspace_bytes = 0x10000, 1 << 40
    k = v = q = 0x20000
    seq = idx = 0x30000
    budget, buffer, alpha, lam, mask = 1024, 128, 8, 0.1, rkv.RKV_STAGE_ALL
    if case == "null_k":
        k = None
    elif case == "misaligned_q":
        q = 0x20008
    elif case == "lambda":
        lam = 1.5
    elif case == "alpha0":
        alpha = 0
    elif case == "budget_le_alpha":
        budget = 8
    elif case == "buffer0":
        buffer = 0
    elif case == "threshold":
        d.sim_threshold = -0.1
    elif case == "group":
        d.n_q_heads = 30
    elif case == "head_dim":
        d.head_dim = 96
    elif case == "dtype":
        d.dtype = 7
    elif case == "no_workspace":
        d.workspace = None
    elif case == "small_workspace":
        d.workspace_bytes = 1024
    elif case == "stage_mask":
        mask = 32
    rc = rkv.rkv_compress_stages(d, k, v, q, seq, budget, buffer, alpha, lam, idx, 0, mask)
    assert rc == want, rkv.rkv_status_string(rc)


def test_rkv_compress_needs_a_current_descriptor(rkv):
    import threading
    out = {}

    def fresh_thread():     # the current descriptor is per thread
        out["rc"] = rkv.rkv_compress(0x20000, 0x20000, 0x20000, 0x30000, 1024, 128, 8, 0.1, 0x30000, 0)
    t = threading.Thread(target=fresh_thread)
    t.start()
    t.join()
    assert out["rc"] == 1
    assert rkv.rkv_status_string(5) == "RKV_ERR_TIMEOUT"
    assert rkv.rkv_launch_count(_desc(rkv), rkv.RKV_STAGE_ALL) == 13     # prep + head sums, first pass + 2 x (list, scan), symmetric scan + finish, 3 select kernels, gather
    assert rkv.rkv_launch_count(_desc(rkv, flags=rkv.RKV_FLAG_NO_SYMMETRIC), rkv.RKV_STAGE_ALL) == 11
    assert rkv.rkv_launch_count(_desc(rkv, flags=rkv.RKV_FLAG_SIMT_SCORES), rkv.RKV_STAGE_ALL) == 7
    # exact counts for given sizes: small caches run the select stage as one kernel
    assert rkv.rkv_launch_count_for(_desc(rkv), 4096, 128, 8, rkv.RKV_STAGE_ALL) == 13
    assert rkv.rkv_launch_count_for(_desc(rkv), 2048, 128, 8, rkv.RKV_STAGE_ALL) == 13         # 17 key tiles: two rounds as well
    assert rkv.rkv_launch_count_for(_desc(rkv), 1024, 128, 8, rkv.RKV_STAGE_ALL) == 7          # 9 key tiles: no symmetric route
    assert rkv.rkv_launch_count_for(_desc(rkv), 64, 32, 8, rkv.RKV_STAGE_ALL) == 5          # one key tile: no second pass
    assert rkv.rkv_launch_count_for(_desc(rkv), 8, 128, 8, rkv.RKV_STAGE_ALL) == 0           # invalid sizes
    assert rkv.rkv_launch_count_for(_desc(rkv, flags=rkv.RKV_FLAG_HEAD_MEAN), 1024, 128, 8, rkv.RKV_STAGE_ALL) == 8


def test_product_package_does_not_touch_the_oracle():
    pkg = os.path.join(ROOT, "paper_2505_24133_b200")
    for dirpath, _, files in os.walk(pkg):
        for f in files:
            if f.endswith((".py", ".cu", ".cuh", ".h")):
                text = open(os.path.join(dirpath, f)).read()
                assert "oracle" not in text.lower(), f"{f} mentions the oracle"
    for f in os.listdir(os.path.join(ROOT, "oracle")):
        if f.endswith((".py", ".c")):
            text = open(os.path.join(ROOT, "oracle", f)).read()
            assert "paper_2505_24133_b200" not in text and "librkv_b200" not in text


def test_eight_bit_cache_type_sizes_and_counts(rkv):
    """RKV_FP8_E4M3: the workspace grows by the bf16 copy of the keys, the host-buffer staging shrinks to one byte per
    cache element (queries stay bf16), one more kernel (the widening) is launched; an unknown type is refused."""
    P, cap, alpha = 2 * 8, 1024 + 128, 8
    for hd in (64, 128, 256):
        b16 = _desc(rkv, head_dim=hd)
        f8 = _desc(rkv, head_dim=hd, dtype=rkv.RKV_FP8_E4M3)
        w16, w8 = rkv.rkv_workspace_bytes(b16, 1024, 128, alpha), rkv.rkv_workspace_bytes(f8, 1024, 128, alpha)
        # head dimension 64: bf16 caches are scored on a copy padded to 128 dimensions as well, so nothing is added
        assert w8 == w16 + (0 if hd == 64 else (P * cap + 128) * hd * 2)
        h16, h8 = rkv.rkv_host_workspace_bytes(b16, 1024, 128, alpha), rkv.rkv_host_workspace_bytes(f8, 1024, 128, alpha)
        assert (h16 - w16) - (h8 - w8) == 2 * P * cap * hd            # K and V staging: two bytes per element less one
        assert rkv.rkv_launch_count_for(f8, 1024, 128, alpha, rkv.RKV_STAGE_ALL) == \
            rkv.rkv_launch_count_for(b16, 1024, 128, alpha, rkv.RKV_STAGE_ALL) + (1 if hd == 256 else 0)
        # (d = 128 with a capacity of whole tiles: the prep kernel writes the widened copy itself; otherwise one more launch)
        assert rkv.rkv_launch_count_for(f8, 1000, 100, alpha, rkv.RKV_STAGE_ALL) == \
            rkv.rkv_launch_count_for(b16, 1000, 100, alpha, rkv.RKV_STAGE_ALL) + (0 if hd == 64 else 1)
        assert rkv.rkv_launch_count_for(f8, 1024, 128, alpha, rkv.RKV_STAGE_GATHER) == 1
    # head dimension 64 takes the kernels of head dimension 128 plus the one that writes the padded copy; on the
    # CUDA-core route (on request) it needs neither the copy nor the extra launches
    d64, d128 = _desc(rkv, head_dim=64), _desc(rkv)
    assert rkv.rkv_launch_count_for(d64, 1024, 128, alpha, rkv.RKV_STAGE_ALL) == \
        rkv.rkv_launch_count_for(d128, 1024, 128, alpha, rkv.RKV_STAGE_ALL) + 1
    w64, w128 = rkv.rkv_workspace_bytes(d64, 1024, 128, alpha), rkv.rkv_workspace_bytes(d128, 1024, 128, alpha)
    assert w64 == w128 + (P * cap + 128) * 128 * 2 + 2 * 32 * alpha * 128 * 2
    s64 = _desc(rkv, head_dim=64, flags=rkv.RKV_FLAG_SIMT_SCORES)
    assert rkv.rkv_workspace_bytes(s64, 1024, 128, alpha) < w128
    assert rkv.rkv_launch_count_for(s64, 1024, 128, alpha, rkv.RKV_STAGE_ALL) == 4      # prep, scores, select, gather
    assert rkv.rkv_workspace_bytes(_desc(rkv, dtype=3), 1024, 128, alpha) == 0
    assert rkv.rkv_decode_workspace_bytes(_desc(rkv, dtype=rkv.RKV_FP8_E4M3), 1024, 128) == \
        rkv.rkv_decode_workspace_bytes(_desc(rkv), 1024, 128) > 0       # the attention takes 8-bit caches like bf16 ones

"""ctypes binding of include/rkv.h: same names, argument marshalling only.

torch is used for device memory and streams; tensors cross the boundary as raw pointers.
"""
from __future__ import annotations

import ctypes
import os
from typing import Optional, Sequence

import torch

_PKG = os.path.dirname(os.path.abspath(__file__))
_LIB_PATH = os.path.join(_PKG, "librkv_b200.so")
_lib = None

RKV_OK = 0
RKV_BF16, RKV_F32, RKV_FP8_E4M3 = 0, 1, 2
RKV_FLAG_SIMT_SCORES = 1
RKV_FLAG_ROWBLOCK_SCORES = 2
RKV_FLAG_MEAN_THEN_POOL = 4
RKV_FLAG_HEAD_MEAN = 8
RKV_FLAG_GQA_MEAN_POOL = 16
RKV_FLAG_NO_SYMMETRIC = 32
RKV_STAGE_PREP, RKV_STAGE_SCORES, RKV_STAGE_SELECT, RKV_STAGE_GATHER, RKV_STAGE_ALL = 1, 2, 4, 8, 15


class RkvError(RuntimeError):
    def __init__(self, status: int, where: str):
        self.status = status
        detail = lib().rkv_last_cuda_error().decode() if status == 4 else ""
        super().__init__(f"{where}: {rkv_status_string(status)}" + (f" ({detail})" if detail else ""))


class RkvDesc(ctypes.Structure):
    """Mirror of rkv_desc_t."""
    _fields_ = [
        ("batch", ctypes.c_int32), ("n_kv_heads", ctypes.c_int32), ("n_q_heads", ctypes.c_int32),
        ("head_dim", ctypes.c_int32), ("dtype", ctypes.c_int32), ("pool_w", ctypes.c_int32),
        ("beta", ctypes.c_int32), ("sim_threshold", ctypes.c_float), ("eps", ctypes.c_float),
        ("flags", ctypes.c_uint32), ("workspace", ctypes.c_void_p), ("workspace_bytes", ctypes.c_size_t),
        ("device_status", ctypes.c_void_p), ("dbg_I", ctypes.c_void_p), ("dbg_Sbar", ctypes.c_void_p),
        ("dbg_R", ctypes.c_void_p), ("dbg_Z", ctypes.c_void_p), ("stage_events", ctypes.c_void_p),
        ("kernel_events", ctypes.c_void_p), ("dbg_counters", ctypes.c_void_p),
        ("wait_limit_cycles", ctypes.c_int64), ("budgets", ctypes.c_void_p), ("block_table", ctypes.c_void_p),
        ("pool_pages", ctypes.c_int64),
    ]


def lib_path() -> str:
    return _LIB_PATH


def lib():
    """Load librkv_b200.so (built in-tree by paper_2505_24133_b200/build.py).  No fallback."""
    global _lib
    if _lib is None:
        if not os.path.exists(_LIB_PATH):
            raise ImportError(f"{_LIB_PATH} is missing: run `python paper_2505_24133_b200/build.py` "
                              "(or __graft_entry__.build()); there is no CPU fallback")
        L = ctypes.CDLL(_LIB_PATH)
        P, I32, F, VP, U32, SZ = (ctypes.POINTER(RkvDesc), ctypes.c_int32, ctypes.c_float, ctypes.c_void_p,
                                  ctypes.c_uint32, ctypes.c_size_t)
        ten = [VP, VP, VP, VP, I32, I32, I32, F, VP, VP]     # the 10 arguments of rkv_compress
        L.rkv_desc_default.restype, L.rkv_desc_default.argtypes = None, [P]
        L.rkv_workspace_bytes.restype, L.rkv_workspace_bytes.argtypes = SZ, [P, I32, I32, I32]
        L.rkv_host_workspace_bytes.restype, L.rkv_host_workspace_bytes.argtypes = SZ, [P, I32, I32, I32]
        L.rkv_set_desc.restype, L.rkv_set_desc.argtypes = ctypes.c_int, [P]
        L.rkv_compress.restype, L.rkv_compress.argtypes = ctypes.c_int, ten
        L.rkv_compress_ex.restype, L.rkv_compress_ex.argtypes = ctypes.c_int, [P] + ten
        L.rkv_compress_stages.restype, L.rkv_compress_stages.argtypes = ctypes.c_int, [P] + ten + [U32]
        L.rkv_compress_host.restype, L.rkv_compress_host.argtypes = ctypes.c_int, [P] + ten
        L.rkv_compress_static.restype, L.rkv_compress_static.argtypes = ctypes.c_int, [P] + ten
        L.rkv_append.restype, L.rkv_append.argtypes = ctypes.c_int, [P, VP, VP, VP, VP, VP, I32, I32, VP]
        L.rkv_push_query.restype, L.rkv_push_query.argtypes = ctypes.c_int, [P, VP, VP, I32, I32, VP]
        L.rkv_decode_workspace_bytes.restype, L.rkv_decode_workspace_bytes.argtypes = SZ, [P, I32, I32]
        L.rkv_decode_attention.restype, L.rkv_decode_attention.argtypes = ctypes.c_int, [P, VP, VP, VP, VP, VP, I32, I32, VP]
        L.rkv_selftest_wait_expiry.restype, L.rkv_selftest_wait_expiry.argtypes = ctypes.c_int, [VP, VP, ctypes.c_int64, VP]
        L.rkv_launch_count.restype, L.rkv_launch_count.argtypes = ctypes.c_int, [P, U32]
        L.rkv_launch_count_for.restype, L.rkv_launch_count_for.argtypes = ctypes.c_int, [P, I32, I32, I32, U32]
        L.rkv_status_string.restype, L.rkv_status_string.argtypes = ctypes.c_char_p, [ctypes.c_int]
        L.rkv_last_cuda_error.restype, L.rkv_last_cuda_error.argtypes = ctypes.c_char_p, []
        _lib = L
    return _lib


def _ptr(t) -> Optional[int]:
    if t is None:
        return None
    if isinstance(t, int):
        return t
    assert t.is_contiguous(), "tensors must be contiguous"
    return t.data_ptr()


def _stream(stream) -> Optional[int]:
    if stream is None:
        return torch.cuda.current_stream().cuda_stream if torch.cuda.is_available() else None
    return stream.cuda_stream if hasattr(stream, "cuda_stream") else int(stream)


def rkv_status_string(status: int) -> str:
    return lib().rkv_status_string(int(status)).decode()


def rkv_desc_default() -> RkvDesc:
    d = RkvDesc()
    lib().rkv_desc_default(ctypes.byref(d))
    return d


def rkv_workspace_bytes(desc: RkvDesc, budget: int, buffer: int, alpha: int) -> int:
    return int(lib().rkv_workspace_bytes(ctypes.byref(desc), budget, buffer, alpha))


def rkv_host_workspace_bytes(desc: RkvDesc, budget: int, buffer: int, alpha: int) -> int:
    return int(lib().rkv_host_workspace_bytes(ctypes.byref(desc), budget, buffer, alpha))


def rkv_set_desc(desc: RkvDesc) -> int:
    return lib().rkv_set_desc(ctypes.byref(desc))


def rkv_launch_count(desc: RkvDesc, stage_mask: int = RKV_STAGE_ALL) -> int:
    return lib().rkv_launch_count(ctypes.byref(desc), stage_mask)


def rkv_launch_count_for(desc: RkvDesc, budget: int, buffer: int, alpha: int, stage_mask: int = RKV_STAGE_ALL) -> int:
    return lib().rkv_launch_count_for(ctypes.byref(desc), budget, buffer, alpha, stage_mask)


def rkv_compress(k_cache, v_cache, q_window, seq_lens, budget, buffer, alpha, lam, out_idx, stream=None) -> int:
    return lib().rkv_compress(_ptr(k_cache), _ptr(v_cache), _ptr(q_window), _ptr(seq_lens), budget, buffer, alpha,
                              float(lam), _ptr(out_idx), _stream(stream))


def rkv_compress_ex(desc, k_cache, v_cache, q_window, seq_lens, budget, buffer, alpha, lam, out_idx,
                    stream=None) -> int:
    return lib().rkv_compress_ex(ctypes.byref(desc), _ptr(k_cache), _ptr(v_cache), _ptr(q_window), _ptr(seq_lens),
                                 budget, buffer, alpha, float(lam), _ptr(out_idx), _stream(stream))


def rkv_compress_stages(desc, k_cache, v_cache, q_window, seq_lens, budget, buffer, alpha, lam, out_idx,
                        stream=None, stage_mask: int = RKV_STAGE_ALL) -> int:
    return lib().rkv_compress_stages(ctypes.byref(desc), _ptr(k_cache), _ptr(v_cache), _ptr(q_window),
                                     _ptr(seq_lens), budget, buffer, alpha, float(lam), _ptr(out_idx),
                                     _stream(stream), stage_mask)


def rkv_compress_host(desc, host_k, host_v, host_q, host_seq_lens, budget, buffer, alpha, lam, host_out_idx,
                      stream=None) -> int:
    return lib().rkv_compress_host(ctypes.byref(desc), _ptr(host_k), _ptr(host_v), _ptr(host_q),
                                   _ptr(host_seq_lens), budget, buffer, alpha, float(lam), _ptr(host_out_idx),
                                   _stream(stream))


RKV_STATIC_SCRATCH_BYTES = 32 << 20


def rkv_compress_static(desc, k_cache, v_cache, q_window, seq_lens, budget, buffer, alpha, lam, out_idx,
                        stream=None) -> int:
    """rkv_compress_ex with the scratch taken from the library's built-in 32 MiB device array, for callers that
    cannot allocate a workspace; desc.workspace is ignored.  Calls on one device share that array: do not let
    two of them overlap on the GPU."""
    return lib().rkv_compress_static(ctypes.byref(desc), _ptr(k_cache), _ptr(v_cache), _ptr(q_window),
                                     _ptr(seq_lens), budget, buffer, alpha, float(lam), _ptr(out_idx),
                                     _stream(stream))


def rkv_append(desc, k_cache, v_cache, k_new, v_new, seq_lens, budget, buffer, stream=None) -> int:
    """The new token of every sequence enters its cache at row seq_lens[b]; seq_lens[b] += 1 (Section 3.1)."""
    return lib().rkv_append(ctypes.byref(desc), _ptr(k_cache), _ptr(v_cache), _ptr(k_new), _ptr(v_new), _ptr(seq_lens),
                            budget, buffer, _stream(stream))


def rkv_push_query(desc, q_window, q_new, alpha, slot, stream=None) -> int:
    """q_new becomes row `slot` of every query head's observation window (Algorithm 1's M_alpha as a ring)."""
    return lib().rkv_push_query(ctypes.byref(desc), _ptr(q_window), _ptr(q_new), alpha, slot, _stream(stream))


def rkv_decode_workspace_bytes(desc, budget: int, buffer: int) -> int:
    return int(lib().rkv_decode_workspace_bytes(ctypes.byref(desc), budget, buffer))


def rkv_decode_attention(desc, k_cache, v_cache, q_new, seq_lens, out, budget, buffer, stream=None) -> int:
    """The new token's queries attend over the cached keys and values of their KV heads (Section 3.1, Eq. 1);
    out [batch, n_q_heads, head_dim] float32."""
    return lib().rkv_decode_attention(ctypes.byref(desc), _ptr(k_cache), _ptr(v_cache), _ptr(q_new), _ptr(seq_lens),
                                      _ptr(out), budget, buffer, _stream(stream))


def rkv_selftest_wait_expiry(device_status, report_words, limit_cycles: int, stream=None) -> int:
    """Make a bounded device-side wait run out on purpose in a tiny kernel of its own (failure-detection self-test)."""
    return lib().rkv_selftest_wait_expiry(_ptr(device_status), _ptr(report_words), int(limit_cycles), _stream(stream))


class Compressor:
    """Convenience holder of a descriptor, its workspace and optional score dumps for one cache shape.

    It owns device memory through torch and forwards to the C ABI; it computes nothing itself.
    """

    def __init__(self, batch: int, n_kv_heads: int, n_q_heads: int, budget: int, buffer: int, alpha: int = 8,
                 lam: float = 0.1, dtype: torch.dtype = torch.bfloat16, pool_w: Optional[int] = None,
                 beta: Optional[int] = None, sim_threshold: Optional[float] = None, eps: Optional[float] = None,
                 flags: int = 0, device="cuda", dump_scores: bool = False, host_staging: bool = False,
                 stage_events: bool = False, budgets: Optional[torch.Tensor] = None, head_dim: int = 128,
                 block_table: Optional[torch.Tensor] = None, pool_pages: int = 0):
        self.budget, self.buffer, self.alpha, self.lam = budget, buffer, alpha, lam
        self.cap = budget + buffer
        self.device = torch.device(device)
        d = rkv_desc_default()
        d.batch, d.n_kv_heads, d.n_q_heads = batch, n_kv_heads, n_q_heads
        d.head_dim = head_dim
        if dtype not in (torch.bfloat16, torch.float32, torch.float8_e4m3fn):
            raise ValueError("dtype must be bfloat16, float32 or float8_e4m3fn")
        d.dtype = {torch.bfloat16: RKV_BF16, torch.float32: RKV_F32, torch.float8_e4m3fn: RKV_FP8_E4M3}[dtype]
        if pool_w is not None:
            d.pool_w = pool_w
        if beta is not None:
            d.beta = beta
        if sim_threshold is not None:
            d.sim_threshold = sim_threshold
        if eps is not None:
            d.eps = eps
        d.flags = flags
        nbytes = (rkv_host_workspace_bytes if host_staging else rkv_workspace_bytes)(d, budget, buffer, alpha)
        if nbytes == 0:
            raise RkvError(1, "rkv_workspace_bytes (invalid or unsupported shape)")
        self.workspace = torch.empty(nbytes, dtype=torch.uint8, device=self.device)
        assert self.workspace.data_ptr() % 256 == 0
        d.workspace, d.workspace_bytes = self.workspace.data_ptr(), nbytes
        self.status = torch.zeros(1, dtype=torch.int32, device=self.device)
        d.device_status = self.status.data_ptr()
        self.scores = None
        if dump_scores:
            self.scores = torch.zeros(4, batch, n_kv_heads, self.cap, dtype=torch.float32, device=self.device)
            d.dbg_I, d.dbg_Sbar, d.dbg_R, d.dbg_Z = (self.scores[i].data_ptr() for i in range(4))
        self.events = self.kevents = self.counters = None
        if stage_events:
            self.events = [torch.cuda.Event(enable_timing=True) for _ in range(5)]
            self.kevents = [torch.cuda.Event(enable_timing=True) for _ in range(4)]
            for ev in self.events + self.kevents:      # torch creates the handle lazily, on first record
                ev.record()
            self._event_array = (ctypes.c_void_p * 5)(*[ev.cuda_event for ev in self.events])
            self._kevent_array = (ctypes.c_void_p * 4)(*[ev.cuda_event for ev in self.kevents])
            d.stage_events = ctypes.cast(self._event_array, ctypes.c_void_p)
            d.kernel_events = ctypes.cast(self._kevent_array, ctypes.c_void_p)
            self.counters = torch.zeros(8, dtype=torch.int64, device=self.device)
            d.dbg_counters = self.counters.data_ptr()
        self.budgets = None
        if budgets is not None:          # per-sequence budgets (device int32 [batch]); `budget` stays the maximum
            self.budgets = budgets.to(device=self.device, dtype=torch.int32).contiguous()
            assert self.budgets.shape == (batch,)
            d.budgets = self.budgets.data_ptr()
        self.block_table = None
        if block_table is not None:      # paged caches: [batch, n_kv_heads, cap / 128] page ids into pools of pool_pages pages
            self.block_table = block_table.to(device=self.device, dtype=torch.int32).contiguous()
            assert self.block_table.shape == (batch, n_kv_heads, self.cap // 128)
            d.block_table, d.pool_pages = self.block_table.data_ptr(), pool_pages
        self.desc = d
        self.out_idx = torch.empty(batch, n_kv_heads, budget, dtype=torch.int32, device=self.device)

    def compress(self, k_cache, v_cache, q_window, seq_lens, stream=None, stages: int = RKV_STAGE_ALL):
        """Enqueue one compression; returns out_idx (device tensor, valid once the stream has run)."""
        rc = rkv_compress_stages(self.desc, k_cache, v_cache, q_window, seq_lens, self.budget, self.buffer,
                                 self.alpha, self.lam, self.out_idx, stream, stages)
        if rc != RKV_OK:
            raise RkvError(rc, "rkv_compress")
        return self.out_idx

    def compress_host(self, host_k, host_v, host_q, host_seq_lens, host_out_idx, stream=None):
        rc = rkv_compress_host(self.desc, host_k, host_v, host_q, host_seq_lens, self.budget, self.buffer,
                               self.alpha, self.lam, host_out_idx, stream)
        if rc != RKV_OK:
            raise RkvError(rc, "rkv_compress_host")

    def stage_ms(self) -> Sequence[float]:
        """Milliseconds of prep, scores, select, gather of the last call (after a synchronise)."""
        return [self.events[i].elapsed_time(self.events[i + 1]) for i in range(4)]

    KERNEL_NAMES = ("prep", "scores_pass1", "scores_list", "scores_pass2", "row_stats", "importance", "select", "gather")

    def kernel_ms(self) -> Sequence[float]:
        """Milliseconds of the eight kernels of the last call (KERNEL_NAMES), after a synchronise.  With a
        single-launch scoring kernel its time is under scores_pass2."""
        s, k = self.events, self.kevents
        order = [s[0], s[1], k[0], k[1], s[2], k[2], k[3], s[3], s[4]]
        return [order[i].elapsed_time(order[i + 1]) for i in range(8)]

    def check_status(self):
        s = int(self.status.item())
        if s != 0:
            self.status.zero_()
            raise RkvError(s, "device status")

"""Comparison of the CUDA path's outputs with the CPU oracle (used by the -m gpu tests and the smoke check).

Tolerances (fp32 scores "within 1e-3 relative"; selection exact except for ties within 1e-3 relative of the
k-th score) are written out here:
  I, R   |x - ref| <= 1e-3 * max(|ref|, 1/n)
  Sbar   |x - ref| <= 1e-3 * max(|ref|, 1e-2); a larger gap is accepted only when the oracle's own similarity
         column holds an entry within 1e-5 of the threshold T (the retention rule is discontinuous there) and
         the gap is at most one entry's worth, 1/n
  Z      |x - ref| <= 1e-3 * (lam |I_ref| + (1 - lam) |R_ref|)
  kept   with z_k the oracle's k-th largest Z and tau = 1e-3 |z_k|: every candidate with Z_ref > z_k + tau is
         kept, every one with Z_ref < z_k - tau is evicted, exactly k are kept, ascending, then the alpha
         observation positions
         (head_mean: the same rule on the head-averaged Z, and one list per sequence)
  K, V   rows [0, budget) bit-identical to the oracle's gather applied to the kept positions
"""
from __future__ import annotations

from dataclasses import dataclass, field
from typing import List, Optional

import numpy as np
import torch

import oracle


def to_numpy_f32(t: torch.Tensor) -> np.ndarray:
    if t.dtype == torch.float8_e4m3fn:          # 8-bit caches: the oracle's own decode of the stored codes
        return oracle.e4m3_to_f32(t.detach().view(torch.uint8).cpu().numpy())
    return t.detach().to("cpu", torch.float32).numpy()


def pick(t: torch.Tensor, sel: torch.Tensor) -> torch.Tensor:
    """t[sel] along the leading dimension (8-bit tensors are indexed through their byte view)."""
    if t.dtype == torch.float8_e4m3fn:
        return t.view(torch.uint8)[sel].view(torch.float8_e4m3fn)
    return t[sel]


def raw_rows(t: torch.Tensor) -> np.ndarray:
    """Bit pattern view (uint8 for E4M3 codes, uint16 for bf16, uint32 for fp32) on the CPU."""
    t = t.detach().cpu().contiguous()
    if t.dtype == torch.float8_e4m3fn:
        return t.view(torch.uint8).numpy()
    return t.view(torch.int16).numpy().view(np.uint16) if t.dtype == torch.bfloat16 else \
        t.view(torch.int32).numpy().view(np.uint32)


@dataclass
class ParityReport:
    heads: int = 0
    compressed_heads: int = 0
    max_rel_I: float = 0.0
    max_rel_R: float = 0.0
    max_rel_Z: float = 0.0
    max_abs_Sbar: float = 0.0
    threshold_flips: int = 0
    band_members: int = 0          # candidates inside the tie band, summed over heads
    sets_identical: int = 0        # heads whose kept set equals the oracle's exactly
    errors: List[str] = field(default_factory=list)

    def ok(self) -> bool:
        return not self.errors

    def summary(self) -> str:
        return (f"heads={self.heads} compressed={self.compressed_heads} identical_sets={self.sets_identical} "
                f"band={self.band_members} flips={self.threshold_flips} relI={self.max_rel_I:.2e} "
                f"relR={self.max_rel_R:.2e} relZ={self.max_rel_Z:.2e} absSbar={self.max_abs_Sbar:.2e} "
                f"errors={len(self.errors)}")


def _column_near_threshold(Kc: np.ndarray, i: int, T: float, eps: float, width: float = 1e-5) -> bool:
    Kd = Kc.astype(np.float64)
    Kb = Kd / (np.linalg.norm(Kd, axis=1, keepdims=True) + eps)
    col = Kb @ Kb[i]
    col[i] = 0.0
    return bool(np.any(np.abs(col - T) < width))


def check_batch(k_in: torch.Tensor, v_in: torch.Tensor, q_in: torch.Tensor, seq_in: torch.Tensor, *,
                budget: int, alpha: int, lam: float, W: int, beta: int, T: float, eps: float,
                gpu_idx: torch.Tensor, gpu_k: Optional[torch.Tensor] = None, gpu_v: Optional[torch.Tensor] = None,
                gpu_seq: Optional[torch.Tensor] = None, gpu_scores: Optional[torch.Tensor] = None,
                max_errors: int = 10, mean_then_pool: bool = False, head_mean: bool = False,
                gqa_mean_pool: bool = False, budgets=None) -> ParityReport:
    """All tensors are for the same (sub)batch: k_in/v_in [B,H,cap,d] and q_in [B,Hq,alpha,d] BEFORE the call,
    gpu_* AFTER it.  gpu_scores is [4,B,H,cap] (I, Sbar, R, Z) or None."""
    rep = ParityReport()
    K = to_numpy_f32(k_in)
    Q = to_numpy_f32(q_in)
    seq = seq_in.detach().cpu().numpy().astype(np.int32)
    B, H, cap, d = K.shape
    nb_all = np.full(B, budget, np.int32) if budgets is None else np.asarray(budgets, dtype=np.int32)
    res = oracle.oracle_batch(K, Q, seq, budget=budget, alpha=alpha, lam=lam, W=W, beta=beta, T=T, eps=eps,
                              mean_then_pool=mean_then_pool, head_mean=head_mean, gqa_mean_pool=gqa_mean_pool,
                              budgets=None if budgets is None else nb_all)
    gidx = gpu_idx.detach().cpu().numpy()
    k_raw_in, v_raw_in = raw_rows(k_in), raw_rows(v_in)
    k_raw_out = raw_rows(gpu_k) if gpu_k is not None else None
    v_raw_out = raw_rows(gpu_v) if gpu_v is not None else None
    sc = gpu_scores.detach().cpu().numpy().astype(np.float64) if gpu_scores is not None else None

    def err(msg):
        if len(rep.errors) < max_errors:
            rep.errors.append(msg)

    if gpu_seq is not None:
        want = np.where(seq > nb_all, nb_all, seq)
        got = gpu_seq.detach().cpu().numpy()
        if not np.array_equal(got, want):
            err(f"seq_lens after the call: got {got[:8]}, want {want[:8]}")

    for b in range(B):
        L = int(seq[b])
        nb = int(nb_all[b])            # this sequence's budget (Section 4.2's per-sequence budgets; else the call's)
        kk = nb - alpha
        for h in range(H):
            rep.heads += 1
            tag = f"[b={b},h={h},L={L}]"
            gi = gidx[b, h]
            if L > nb and not np.all(gi[nb:] == -1):
                err(f"{tag} index entries beyond the sequence's budget {nb} are not -1")
            if L > nb:
                gi = gi[:nb]
            if L <= nb:
                if not np.array_equal(gi, res.idx[b, h]):
                    err(f"{tag} no-op index list differs")
                if k_raw_out is not None and not (np.array_equal(k_raw_out[b, h], k_raw_in[b, h]) and
                                                  np.array_equal(v_raw_out[b, h], v_raw_in[b, h])):
                    err(f"{tag} cache changed although L <= budget")
                continue
            rep.compressed_heads += 1
            n = L - alpha
            Zr, Ir, Rr, Sr = res.Z[b, h, :n], res.I[b, h, :n], res.R[b, h, :n], res.Sbar[b, h, :n]
            if sc is not None:
                gI, gS, gR, gZ = (sc[t, b, h, :n] for t in range(4))
                if not (np.all(np.isfinite(gI)) and np.all(np.isfinite(gS)) and np.all(np.isfinite(gR))):
                    err(f"{tag} non-finite scores")
                    continue
                relI = np.abs(gI - Ir) / np.maximum(np.abs(Ir), 1.0 / n)
                rep.max_rel_I = max(rep.max_rel_I, float(relI.max()))
                if relI.max() > 1e-3:
                    err(f"{tag} I off by {relI.max():.3e} rel at i={int(relI.argmax())}")
                dS = np.abs(gS - Sr)
                bad = np.nonzero(dS > 1e-3 * np.maximum(np.abs(Sr), 1e-2))[0]
                flips = 0
                for i in bad:
                    if dS[i] <= 1.0 / n + 1e-6 and _column_near_threshold(K[b, h, :n], int(i), T, eps):
                        flips += 1
                    else:
                        err(f"{tag} Sbar[{int(i)}] = {gS[i]:.8f}, oracle {Sr[i]:.8f}")
                rep.threshold_flips += flips
                ok_rows = np.ones(n, bool)
                ok_rows[bad] = False
                if ok_rows.any():
                    rep.max_abs_Sbar = max(rep.max_abs_Sbar, float(dS[ok_rows].max()))
                relR = np.abs(gR - Rr) / np.maximum(np.abs(Rr), 1.0 / n)
                relR_lim = np.where(ok_rows, 1e-3, 1e-3 + 1.5 / n)       # a flipped row moves R by ~1/n relative
                rep.max_rel_R = max(rep.max_rel_R, float(relR[ok_rows].max()) if ok_rows.any() else 0.0)
                if np.any(relR > relR_lim):
                    i = int((relR - relR_lim).argmax())
                    err(f"{tag} R off by {relR[i]:.3e} rel at i={i}")
                scaleZ = lam * np.abs(Ir) + (1 - lam) * np.abs(Rr)
                relZ = np.abs(gZ - Zr) / np.maximum(scaleZ, 1e-300)
                rep.max_rel_Z = max(rep.max_rel_Z, float(relZ[ok_rows].max()) if ok_rows.any() else 0.0)
                if np.any(relZ > np.where(ok_rows, 1e-3, 1e-3 + 1.5 / n)):
                    i = int(relZ.argmax())
                    err(f"{tag} Z off by {relZ[i]:.3e} (scaled) at i={i}")
            # ---- kept positions
            cand = gi[:kk]
            if not (np.all(np.diff(gi) > 0) and gi[0] >= 0 and np.array_equal(gi[kk:], np.arange(n, L))):
                err(f"{tag} index list not ascending / observation tail wrong: {gi[:4]}..{gi[-alpha - 1:]}")
                continue
            ref_set = res.idx[b, h, :kk]
            if head_mean:
                # Algorithm 1's aggregated selection: the kept set is judged on the head-averaged score, and every
                # head of the sequence carries the same list
                Zr = res.Z[b, :, :n].mean(axis=0)
                if not np.array_equal(gi, gidx[b, 0][:nb]):
                    err(f"{tag} index list differs from head 0's although one set per sequence was asked for")
            z_k = Zr[ref_set].min()
            tau = 1e-3 * abs(z_k)
            must_keep = np.nonzero(Zr > z_k + tau)[0]
            must_evict = np.nonzero(Zr < z_k - tau)[0]
            rep.band_members += int(n - must_keep.size - must_evict.size)
            kept = np.zeros(n, bool)
            kept[cand] = True
            if not kept[must_keep].all():
                miss = must_keep[~kept[must_keep]]
                err(f"{tag} evicted {miss.size} tokens whose score is clearly above the k-th, e.g. i={int(miss[0])} "
                    f"Z={Zr[miss[0]]:.6e} z_k={z_k:.6e}")
            if kept[must_evict].any():
                wrong = must_evict[kept[must_evict]]
                err(f"{tag} kept {wrong.size} tokens whose score is clearly below the k-th, e.g. i={int(wrong[0])} "
                    f"Z={Zr[wrong[0]]:.6e} z_k={z_k:.6e}")
            if np.array_equal(cand, ref_set):
                rep.sets_identical += 1
            # ---- compacted rows: the oracle's gather on the positions the GPU kept
            if k_raw_out is not None:
                if not np.array_equal(k_raw_out[b, h, :nb], oracle.oracle_gather(k_raw_in[b, h], gi)):
                    err(f"{tag} compacted K rows differ from the gather of the kept positions")
                if not np.array_equal(v_raw_out[b, h, :nb], oracle.oracle_gather(v_raw_in[b, h], gi)):
                    err(f"{tag} compacted V rows differ from the gather of the kept positions")
    return rep


# ----------------------------------------------------------------------------- paged caches (layout only)
def to_paged(cache: torch.Tensor, pool_pages: int, table: torch.Tensor, fill=float("nan")) -> torch.Tensor:
    """cache [B, H, cap, d] (cap a multiple of 128) scattered into a page pool [pool_pages, 128, d]: rows
    [128 t, 128 t + 128) of head (b, h) go to page table[b, h, t].  Pages nobody owns hold `fill`."""
    B, H, cap, d = cache.shape
    pool = torch.full((pool_pages, 128, d), fill, dtype=cache.dtype, device=cache.device)
    pool[table.reshape(-1).long()] = cache.reshape(B * H * (cap // 128), 128, d)
    return pool


def from_paged(pool: torch.Tensor, table: torch.Tensor) -> torch.Tensor:
    """The inverse view: [B, H, cap, d] gathered from the pool through the table."""
    B, H, T = table.shape
    return pool[table.reshape(-1).long()].reshape(B, H, T * 128, pool.shape[-1])


def random_block_table(B: int, H: int, pages_per_head: int, pool_pages: int, seed: int, device="cuda") -> torch.Tensor:
    """Distinct page ids in random order, with unused pages in between."""
    g = torch.Generator().manual_seed(seed)
    ids = torch.randperm(pool_pages, generator=g)[:B * H * pages_per_head]
    return ids.reshape(B, H, pages_per_head).to(torch.int32).to(device)

"""Pins of the CPU oracle against what the paper and the mathematics fix (no GPU).

Each test ties one part of the oracle to something other than the oracle itself:
library routines in the special cases where the method reduces to them, closed forms,
invariants, and an independent brute force on tiny inputs.  Citations are to the paper's
equations / sections.
"""
import itertools

import numpy as np
import pytest
from scipy.ndimage import maximum_filter1d
from scipy.special import softmax as sp_softmax
from sklearn.metrics.pairwise import cosine_similarity

import oracle

D = 128


def _rand(rng, *shape):
    return rng.standard_normal(shape).astype(np.float32)


def _run(K, Q, budget, alpha, **kw):
    args = dict(lam=0.1, W=4, beta=1, T=0.5, eps=1e-8)
    args.update(kw)
    return oracle.oracle_head(K, Q, budget=budget, alpha=alpha, want_S=True, **args)


# ----------------------------------------------------------------------------- Eq. 1-3
def test_mha_equals_textbook_softmax_attention():
    """Eq. 1: with G = 1 the weights are softmax(Q K^T / sqrt(d)) over the candidate keys."""
    rng = np.random.default_rng(1)
    L, alpha = 50, 8
    K, Q = _rand(rng, L, D), _rand(rng, 1, alpha, D)
    r = _run(K, Q, budget=20, alpha=alpha)
    n = L - alpha
    ref = sp_softmax(Q[0].astype(np.float64) @ K[:n].astype(np.float64).T / np.sqrt(D), axis=1)
    np.testing.assert_allclose(r.A, ref, rtol=1e-12, atol=1e-300)


def test_gqa_maxpool_on_logits_then_one_softmax():
    """Eq. 2-3: max over the group on the scaled logits, then softmax.  Rows sum to 1 (softmax per head
    followed by a max would not), and the result equals the library softmax of the pooled logits."""
    rng = np.random.default_rng(2)
    L, alpha, G = 70, 8, 4
    K, Q = _rand(rng, L, D), _rand(rng, G, alpha, D) * 2.0
    r = _run(K, Q, budget=30, alpha=alpha)
    n = L - alpha
    np.testing.assert_allclose(r.A.sum(axis=1), 1.0, rtol=1e-12)
    logits = np.einsum("gjd,nd->gjn", Q.astype(np.float64), K[:n].astype(np.float64)) / np.sqrt(D)
    np.testing.assert_allclose(r.A, sp_softmax(logits.max(axis=0), axis=1), rtol=1e-12)
    # the wrong order (softmax per query head, then max) differs and does not sum to 1
    wrong = sp_softmax(logits, axis=2).max(axis=0)
    assert np.abs(wrong.sum(axis=1) - 1.0).min() > 1e-3
    assert np.abs(wrong - r.A).max() > 1e-4


def test_duplicate_query_head_changes_nothing():
    """max over the group is idempotent: repeating a query head leaves A and I unchanged."""
    rng = np.random.default_rng(3)
    K, Q = _rand(rng, 60, D), _rand(rng, 3, 8, D)
    a = _run(K, Q, budget=24, alpha=8)
    b = _run(K, np.concatenate([Q, Q[1:2]], axis=0), budget=24, alpha=8)
    np.testing.assert_array_equal(a.A, b.A)
    np.testing.assert_array_equal(a.I, b.I)


def test_query_group_order_is_irrelevant_but_row_order_is_not():
    rng = np.random.default_rng(4)
    K, Q = _rand(rng, 60, D), _rand(rng, 4, 8, D)
    a = _run(K, Q, budget=24, alpha=8)
    b = _run(K, Q[::-1].copy(), budget=24, alpha=8)
    np.testing.assert_allclose(a.A, b.A, rtol=1e-14)
    c = _run(K, Q[:, ::-1].copy(), budget=24, alpha=8)   # reversing the alpha rows permutes A's rows
    np.testing.assert_allclose(a.A, c.A[::-1], rtol=1e-14)


def test_observation_tokens_are_not_candidates():
    """Section 3.1: the last alpha cached tokens are observation tokens; scores cover n = L - alpha keys,
    and changing the observation KEYS changes no score."""
    rng = np.random.default_rng(5)
    L, alpha = 64, 8
    K, Q = _rand(rng, L, D), _rand(rng, 2, alpha, D)
    a = _run(K, Q, budget=32, alpha=alpha)
    K2 = K.copy()
    K2[L - alpha:] = _rand(rng, alpha, D)
    b = _run(K2, Q, budget=32, alpha=alpha)
    assert a.I.shape == (L - alpha,)
    np.testing.assert_array_equal(a.Z, b.Z)
    np.testing.assert_array_equal(a.idx, b.idx)


# ----------------------------------------------------------------------------- Eq. 4
@pytest.mark.parametrize("W", [0, 1, 2, 4, 7])
def test_sliding_max_matches_library_filter_and_bounds(W):
    """Eq. 4: window {i-W .. i+W-1} clipped to the candidates, max per query row, mean over rows."""
    rng = np.random.default_rng(6)
    L, alpha = 90, 8
    K, Q = _rand(rng, L, D), _rand(rng, 4, alpha, D) * 3.0
    r = _run(K, Q, budget=40, alpha=alpha, W=W)
    n = L - alpha
    if W == 0:
        pooled = r.A
        np.testing.assert_allclose(r.I.sum(), 1.0, rtol=1e-12)       # mean of rows that each sum to 1
    else:
        # scipy's even-size window for output i covers i - size//2 .. i + size//2 - 1
        pooled = maximum_filter1d(r.A, size=2 * W, axis=1, mode="constant", cval=0.0, origin=0)
        brute = np.array([[r.A[j, max(0, i - W):min(n, i + W)].max() for i in range(n)]
                          for j in range(alpha)])
        np.testing.assert_array_equal(pooled, brute)
        assert 1.0 <= r.I.sum() <= 2 * W
    np.testing.assert_allclose(r.I, pooled.mean(axis=0), rtol=1e-13)
    base = _run(K, Q, budget=40, alpha=alpha, W=0)
    assert np.all(r.I >= base.I - 1e-18)


def test_single_spike_spreads_over_the_asymmetric_window():
    """Eq. 4: a spike at position p raises exactly positions p-W+1 .. p+W (the window of position i reaches
    one further to the left than to the right)."""
    n, alpha, W, p = 40, 8, 3, 17
    L = n + alpha
    K = np.zeros((L, D), np.float32)
    K[:, 1] = 1.0                      # keeps every key non-zero; orthogonal to the queries
    K[p, 0] = 50.0                     # the only key with a component along the queries
    Q = np.zeros((1, alpha, D), np.float32)
    Q[0, :, 0] = 10.0
    r = _run(K, Q, budget=20, alpha=alpha, W=W)
    assert r.A[:, p].min() > 0.999999
    raised = np.nonzero(r.I > 0.5)[0]
    np.testing.assert_array_equal(raised, np.arange(p - W + 1, p + W + 1))


# ----------------------------------------------------------------------------- Eq. 5
def test_cosine_matrix_matches_library_and_its_invariants():
    rng = np.random.default_rng(7)
    L, alpha = 80, 8
    K, Q = _rand(rng, L, D), _rand(rng, 1, alpha, D)
    r = _run(K, Q, budget=30, alpha=alpha)
    n = L - alpha
    ref = cosine_similarity(K[:n].astype(np.float64))
    np.fill_diagonal(ref, 0.0)
    np.testing.assert_allclose(r.S_raw, ref, atol=1e-12)
    np.testing.assert_array_equal(np.diag(r.S_raw), 0.0)
    np.testing.assert_allclose(r.S_raw, r.S_raw.T, atol=1e-15)
    assert np.abs(r.S_raw).max() <= 1.0
    # scaling a key by c > 0 changes nothing (up to the eps in the denominator)
    K2 = K.copy()
    K2[3] *= 7.5
    r2 = _run(K2, Q, budget=30, alpha=alpha)
    np.testing.assert_allclose(r2.S_raw, r.S_raw, atol=1e-8)


def test_eps_is_added_to_the_norm_and_zero_keys_are_safe():
    """Eq. 5: Kbar = K / (||K|| + eps).  A large eps makes the effect visible: S_ij = k_i.k_j /
    ((|k_i|+eps)(|k_j|+eps)); an all-zero key gives a zero row, not NaN."""
    rng = np.random.default_rng(8)
    L, alpha, eps = 40, 8, 0.75
    K, Q = _rand(rng, L, D), _rand(rng, 1, alpha, D)
    K[5] = 0.0
    r = _run(K, Q, budget=16, alpha=alpha, eps=eps)
    n = L - alpha
    Kd = K[:n].astype(np.float64)
    nr = np.linalg.norm(Kd, axis=1) + eps
    ref = (Kd @ Kd.T) / np.outer(nr, nr)
    np.fill_diagonal(ref, 0.0)
    np.testing.assert_allclose(r.S_raw, ref, atol=1e-13)
    assert np.all(r.S_raw[5] == 0.0) and np.all(np.isfinite(r.R))


def test_orthonormal_keys_give_uniform_redundancy():
    n, alpha = 88, 8
    L = n + alpha
    K = np.zeros((L, D), np.float32)
    K[np.arange(n), np.arange(n)] = 1.0
    K[n:, 0] = 1.0
    Q = _rand(np.random.default_rng(9), 2, alpha, D)
    r = _run(K, Q, budget=64, alpha=alpha)
    np.testing.assert_allclose(r.S_raw, 0.0, atol=1e-15)
    np.testing.assert_allclose(r.R, 1.0 / n, rtol=1e-12)


# ----------------------------------------------------------------------------- Eq. 6 without the rule
@pytest.mark.parametrize("mode", ["beta0", "T1"])
def test_row_mean_closed_form_without_retention(mode):
    """With beta = 0 (or T = 1: nothing exceeds it) Eq. 6 is linear:
    Sbar_i = (Kbar_i . s - Kbar_i . Kbar_i) / n with s = sum_j Kbar_j.  Checks the whole matrix + mean
    in O(n d), at a size with a ragged tail."""
    rng = np.random.default_rng(10)
    L, alpha = 300 + 8 + 37, 8
    K, Q = _rand(rng, L, D), _rand(rng, 1, alpha, D)
    K[:, :3] *= 6.0
    kw = dict(beta=0) if mode == "beta0" else dict(T=1.0, beta=5)
    r = _run(K, Q, budget=100, alpha=alpha, **kw)
    n = L - alpha
    Kd = K[:n].astype(np.float64)
    Kb = Kd / (np.linalg.norm(Kd, axis=1, keepdims=True) + 1e-8)
    s = Kb.sum(axis=0)
    ref = (Kb @ s - (Kb * Kb).sum(axis=1)) / n
    np.testing.assert_allclose(r.Sbar, ref, atol=1e-13)
    np.testing.assert_allclose(r.R, sp_softmax(ref), rtol=1e-11)
    np.testing.assert_allclose(r.R.sum(), 1.0, rtol=1e-12)


# ----------------------------------------------------------------------------- retention rule
@pytest.mark.parametrize("beta", [0, 1, 2, 8, 200])
def test_identical_keys_give_uniform_redundancy(beta):
    """All keys equal: every off-diagonal similarity is 1 > T, so each token loses min(beta, n-1) entries:
    Sbar_i = (n - 1 - min(beta, n-1)) / n for every i and R = 1/n."""
    n, alpha = 88, 8
    L = n + alpha
    rng = np.random.default_rng(11)
    K = np.tile(_rand(rng, 1, D), (L, 1))
    Q = _rand(rng, 4, alpha, D)
    r = _run(K, Q, budget=64, alpha=alpha, beta=beta, T=0.5)
    # eps = 1e-8 in the denominator lowers each similarity by ~2e-8 / ||k||
    np.testing.assert_allclose(r.Sbar, (n - 1 - min(beta, n - 1)) / n, rtol=1e-7, atol=1e-9)
    np.testing.assert_allclose(r.R, 1.0 / n, rtol=1e-12)


@pytest.mark.parametrize("beta", [0, 1, 3, 10])
def test_cluster_closed_form(beta):
    """m copies of e_0 scattered among distinct orthogonal keys: Sbar = (m-1-min(beta, m-1))/n on the
    copies and 0 elsewhere; R follows in closed form."""
    n, alpha, m = 60, 8, 6
    L = n + alpha
    K = np.zeros((L, D), np.float32)
    copies = np.array([2, 9, 10, 31, 47, 59])
    free_axis = 1
    for i in range(L):
        if i in copies:
            K[i, 0] = 3.0
        else:
            K[i, free_axis] = 1.0 + 0.1 * i
            free_axis += 1
    Q = _rand(np.random.default_rng(12), 1, alpha, D)
    r = _run(K, Q, budget=40, alpha=alpha, beta=beta, T=0.5)
    sbar = np.zeros(n)
    sbar[copies] = (m - 1 - min(beta, m - 1)) / n
    np.testing.assert_allclose(r.Sbar, sbar, atol=1e-9)       # eps = 1e-8 shows at the 1e-9 level
    e = np.exp(sbar)
    np.testing.assert_allclose(r.R, e / e.sum(), rtol=1e-8)


def _retention_brute(S, T, beta):
    """Independent statement of Section 3.3's rule: per token i, sort the partner set by position."""
    S = S.copy()
    n = S.shape[0]
    for i in range(n):
        partners = sorted((j for j in range(n) if S[j, i] > T), reverse=True)
        for j in partners[:beta]:
            S[j, i] = 0.0
    return S


@pytest.mark.parametrize("T,beta", list(itertools.product([0.0, 0.3, 0.5, 0.9, 1.0], [0, 1, 2, 8, 1000])))
def test_retention_rule_brute_force(T, beta):
    """Random keys with planted near-duplicates; the rule zeroes, per token, the beta largest positions among
    the partners above T (strict >), deciding on the unmodified matrix."""
    rng = np.random.default_rng(13)
    L, alpha = 56, 8
    n = L - alpha
    K = _rand(rng, L, D)
    K[:, :2] *= 5.0
    for p in (7, 20, 21, 33, 40, 47):
        K[p] = K[rng.integers(0, p)] + 0.05 * _rand(rng, D)
    Q = _rand(rng, 2, alpha, D)
    r = _run(K, Q, budget=30, alpha=alpha, T=T, beta=beta)
    ref = _retention_brute(r.S_raw, T, beta)
    np.testing.assert_array_equal(r.S_mod, ref)
    np.testing.assert_allclose(r.Sbar, ref.sum(axis=0) / n, atol=1e-15)
    if beta >= n:      # every above-threshold entry vanishes
        np.testing.assert_array_equal(r.S_mod, np.where(r.S_raw > T, 0.0, r.S_raw))
    if T == 0.0 and beta > 0:
        assert (r.S_raw > 0).sum() > (r.S_mod > 0).sum()   # strict '>' at T = 0: zeros never count
    # the diagonal (zero) is never a partner for T in [0, 1]
    assert np.all(np.diag(r.S_mod) == 0.0)


def test_retention_prefers_the_most_recent_partner():
    """Three identical keys at positions 4 < 11 < 30 among orthogonal ones, beta = 1: token 4 loses its link
    to 30, token 11 loses 30, token 30 loses 11."""
    n, alpha = 40, 8
    L = n + alpha
    K = np.zeros((L, D), np.float32)
    ax = 1
    for i in range(L):
        if i in (4, 11, 30):
            K[i, 0] = 2.0
        else:
            K[i, ax] = 1.0
            ax += 1
    Q = _rand(np.random.default_rng(14), 1, alpha, D)
    r = _run(K, Q, budget=20, alpha=alpha, beta=1, T=0.5)
    assert r.S_mod[30, 4] == 0 and r.S_mod[11, 4] > 0.999
    assert r.S_mod[30, 11] == 0 and r.S_mod[4, 11] > 0.999
    assert r.S_mod[11, 30] == 0 and r.S_mod[4, 30] > 0.999


def test_redundancy_is_a_softmax_monotone_in_sbar():
    rng = np.random.default_rng(15)
    K, Q = _rand(rng, 100, D), _rand(rng, 1, 8, D)
    K[:, 0] += 4.0
    r = _run(K, Q, budget=50, alpha=8)
    np.testing.assert_allclose(r.R, sp_softmax(r.Sbar), rtol=1e-12)
    order = np.argsort(r.Sbar)
    assert np.all(np.diff(r.R[order]) >= 0)


# ----------------------------------------------------------------------------- Eq. 7 and selection
def _dup_workload(rng, L, alpha, G):
    K = _rand(rng, L, D)
    K[:, :4] *= 8.0
    for p in range(5, L - alpha, 7):
        K[p] = K[rng.integers(0, p)] + 0.05 * _rand(rng, D)
    return K, _rand(rng, G, alpha, D)


@pytest.mark.parametrize("lam", [0.0, 0.1, 0.5, 1.0])
def test_joint_score_and_topk_against_full_sort(lam):
    """Eq. 7 and per-head top-k: Z = lam I - (1-lam) R; kept = the k = budget - alpha best candidates in
    ascending position, then the alpha observation positions.  lam = 1 is attention-only selection,
    lam = 0 keeps the k least redundant."""
    rng = np.random.default_rng(16)
    L, alpha, budget = 96, 8, 64
    K, Q = _dup_workload(rng, L, alpha, 4)
    r = _run(K, Q, budget=budget, alpha=alpha, lam=lam)
    n, k = L - alpha, budget - alpha
    np.testing.assert_allclose(r.Z, lam * r.I - (1 - lam) * r.R, rtol=1e-15, atol=1e-18)
    assert r.idx.shape == (budget,) and np.all(np.diff(r.idx) > 0) and r.idx.max() == L - 1
    np.testing.assert_array_equal(r.idx[k:], np.arange(n, L))
    key = {1.0: r.I, 0.0: -r.R}.get(lam, r.Z)
    # the sliding max makes exact ties in I; among equals the later position is kept
    best = np.sort(np.lexsort((-np.arange(n), -key))[:k])
    np.testing.assert_array_equal(r.idx[:k], best)
    # nothing evicted outranks anything kept
    evicted = np.setdiff1d(np.arange(n), r.idx[:k])
    assert r.Z[evicted].max() <= r.Z[r.idx[:k]].min()


def test_exact_ties_keep_the_later_position():
    """Identical keys and queries orthogonal to them: all candidates share one score; the k latest stay."""
    n, alpha, budget = 30, 4, 16
    L = n + alpha
    K = np.zeros((L, D), np.float32)
    K[:, 0] = 1.5
    Q = np.zeros((2, alpha, D), np.float32)
    Q[:, :, 1] = 1.0
    r = _run(K, Q, budget=budget, alpha=alpha, W=0)
    assert np.ptp(r.Z) == 0.0
    k = budget - alpha
    np.testing.assert_array_equal(r.idx, np.concatenate([np.arange(n - k, n), np.arange(n, L)]))


def test_guard_and_idempotence():
    """Algorithm 1's guard: with L <= budget nothing is compressed; compressing the compacted cache again
    is therefore a no-op."""
    rng = np.random.default_rng(17)
    L, alpha, budget = 96, 8, 64
    K, Q = _dup_workload(rng, L, alpha, 4)
    V = _rand(rng, L, D)
    r = _run(K, Q, budget=budget, alpha=alpha)
    assert r.compressed
    K2, V2 = oracle.oracle_gather(K, r.idx), oracle.oracle_gather(V, r.idx)
    np.testing.assert_array_equal(K2.view(np.uint32), K[r.idx].view(np.uint32))
    np.testing.assert_array_equal(V2.view(np.uint32), V[r.idx].view(np.uint32))
    r2 = oracle.oracle_head(K2, Q, budget=budget, alpha=alpha, lam=0.1, W=4, beta=1, T=0.5)
    assert not r2.compressed
    np.testing.assert_array_equal(r2.idx, np.arange(budget))
    r3 = oracle.oracle_head(K, Q, budget=budget, alpha=alpha, lam=0.1, W=4, beta=1, T=0.5, L=40)
    assert not r3.compressed
    np.testing.assert_array_equal(r3.idx, np.concatenate([np.arange(40), -np.ones(24, np.int32)]))


def test_gather_copies_bytes_for_16_bit_rows():
    rng = np.random.default_rng(18)
    rows = rng.integers(0, 2 ** 16, size=(50, 128), dtype=np.uint16)   # any bit pattern, NaNs included
    idx = np.array([0, 3, 4, 17, 49, -1], np.int32)
    out = oracle.oracle_gather(rows, idx)
    np.testing.assert_array_equal(out[:5], rows[idx[:5]])
    assert np.all(out[5] == 0)


# ----------------------------------------------------------------------------- batch driver
def test_batch_driver_equals_head_by_head_with_ragged_lengths():
    rng = np.random.default_rng(19)
    B, Hkv, G, cap, alpha, budget = 3, 2, 3, 48, 4, 32
    K = _rand(rng, B, Hkv, cap, D)
    Q = _rand(rng, B, Hkv * G, alpha, D)
    seq = np.array([48, 30, 41], np.int32)
    res = oracle.oracle_batch(K, Q, seq, budget=budget, alpha=alpha, lam=0.1, W=2, beta=1, T=0.2)
    np.testing.assert_array_equal(res.compressed, [True, False, True])
    for b in range(B):
        for h in range(Hkv):
            one = oracle.oracle_head(K[b, h], Q[b, h * G:(h + 1) * G], budget=budget, alpha=alpha, lam=0.1,
                                     W=2, beta=1, T=0.2, L=int(seq[b]))
            np.testing.assert_array_equal(res.idx[b, h], one.idx)
            if one.compressed:
                n = int(seq[b]) - alpha
                np.testing.assert_array_equal(res.Z[b, h, :n], one.Z)
                np.testing.assert_array_equal(res.I[b, h, :n], one.I)
    with pytest.raises(ValueError):
        oracle.oracle_batch(K, Q, np.array([49, 1, 1], np.int32), budget=budget, alpha=alpha, lam=0.1, W=2,
                            beta=1, T=0.2)


# ----------------------------------------------------------------------------- planted mistakes
def test_pins_catch_planted_mistakes():
    """Sanity of the pins themselves: plausible wrong variants (written here, on the CPU) differ from the
    oracle by far more than the tolerances used above."""
    rng = np.random.default_rng(20)
    L, alpha = 64, 8
    K, Q = _dup_workload(rng, L, alpha, 4)
    r = _run(K, Q, budget=32, alpha=alpha, beta=1, T=0.5, W=2)
    n = L - alpha
    # (a) symmetric window i-W..i+W instead of i-W..i+W-1
    sym = np.array([[r.A[j, max(0, i - 2):min(n, i + 3)].max() for i in range(n)] for j in range(alpha)]).mean(0)
    assert np.abs(sym - r.I).max() > 1e-6
    # (b) zeroing the beta SMALLEST positions instead of the largest
    wrong = r.S_raw.copy()
    for i in range(n):
        for j in [j for j in range(n) if r.S_raw[j, i] > 0.5][:1]:
            wrong[j, i] = 0.0
    assert np.abs(wrong.sum(0) / n - r.Sbar).max() > 1e-4
    # (c) mean over the 1/(n-1) off-diagonal entries instead of 1/n
    assert np.abs(r.S_mod.sum(0) / (n - 1) - r.Sbar).max() > 1e-6
    # (d) plus instead of minus in Eq. 7
    assert np.abs((0.1 * r.I + 0.9 * r.R) - r.Z).max() > 1e-4


# ----------------------------------------------------------------------------- hand-worked fixture
def test_handworked_three_copies_fixture():
    """tests/golden/handworked_three_copies.json: every stage worked by hand from the equations."""
    import json
    import os
    with open(os.path.join(os.path.dirname(__file__), "golden", "handworked_three_copies.json")) as f:
        g = json.load(f)
    K = np.array(g["K"], np.float32)
    Q = np.array([[[np.sqrt(2.0) * np.log(g["q_scale_ln"]), 0.0]]], np.float32)
    r = oracle.oracle_head(K, Q, budget=g["budget"], alpha=g["alpha"], lam=g["lam"], W=g["W"], beta=g["beta"],
                           T=g["T"])
    np.testing.assert_allclose(r.I, g["I"], rtol=1e-6)
    np.testing.assert_allclose(r.Sbar, g["Sbar"], atol=1e-7)
    np.testing.assert_allclose(r.R, g["R"], rtol=1e-6)
    np.testing.assert_allclose(r.Z, g["Z"], atol=2e-7)
    np.testing.assert_array_equal(r.idx, g["idx"])


# ----------------------------------------------------------------------------- Algorithm 1's order (variant)
@pytest.mark.parametrize("W", [0, 1, 3, 6])
def test_mean_then_pool_variant_against_numpy_and_eq4(W):
    """Algorithm 1 takes the mean over the alpha query rows first and pools afterwards (read as Eq. 4's max over
    the same window).  Pinned by a numpy recomputation from the attention weights, by a library max filter, and by
    max-of-means <= mean-of-maxes against the Eq. 4 order; with W = 0 the two orders coincide."""
    rng = np.random.default_rng(40 + W)
    L, alpha = 150, 8
    K, Q = _rand(rng, L, D), _rand(rng, 4, alpha, D) * 2.5
    eq4 = _run(K, Q, budget=60, alpha=alpha, W=W)
    var = _run(K, Q, budget=60, alpha=alpha, W=W, mean_then_pool=True)
    n = L - alpha
    np.testing.assert_array_equal(var.A, eq4.A)                       # only the last two steps differ
    mean = var.A.mean(axis=0)
    if W == 0:
        brute = mean
        np.testing.assert_allclose(var.I, eq4.I, rtol=1e-13)
    else:
        brute = np.array([mean[max(0, i - W):min(n, i + W)].max() for i in range(n)])
        lib = maximum_filter1d(mean, size=2 * W, mode="constant", cval=0.0, origin=0)
        np.testing.assert_allclose(lib, brute, rtol=0, atol=0)
    np.testing.assert_allclose(var.I, brute, rtol=1e-13)
    assert np.all(var.I <= eq4.I + 1e-18)
    # the scores downstream follow: Z = lambda I - (1 - lambda) R with the same R
    np.testing.assert_array_equal(var.R, eq4.R)
    np.testing.assert_allclose(var.Z, 0.1 * var.I - 0.9 * var.R, rtol=1e-12, atol=1e-18)


def test_head_mean_aggregated_selection_variant():
    """Algorithm 1 averages the heads' scores and keeps ONE set of positions per sequence.  Pinned by recomputing
    the selection from the oracle's own per-head Z with numpy (stable sort: score descending, later position first
    among equals), by H_kv = 1 reducing to the per-head selection, and by all heads sharing the set."""
    rng = np.random.default_rng(77)
    B, Hkv, Hq, cap, alpha, budget = 2, 3, 6, 90, 8, 50
    K = _rand(rng, B, Hkv, cap, D)
    K[:, :, 40:48] = K[:, :, 8:16] + 0.05 * _rand(rng, B, Hkv, 8, D)         # some redundancy
    Q = _rand(rng, B, Hq, alpha, D) * 2.0
    seq = np.array([90, 77], np.int32)
    kw = dict(budget=budget, alpha=alpha, lam=0.1, W=4, beta=1, T=0.5)
    per = oracle.oracle_batch(K, Q, seq, **kw)
    agg = oracle.oracle_batch(K, Q, seq, head_mean=True, **kw)
    np.testing.assert_array_equal(agg.Z, per.Z)                               # the scores themselves do not change
    k = budget - alpha
    for b in range(B):
        n = int(seq[b]) - alpha
        zbar = per.Z[b, :, :n].mean(axis=0)
        order = sorted(range(n), key=lambda i: (-zbar[i], -i))
        want = np.array(sorted(order[:k]) + list(range(n, n + alpha)), np.int32)
        for h in range(Hkv):
            np.testing.assert_array_equal(agg.idx[b, h], want)
    # the per-head sets do differ on this input (otherwise the pin above would not tell the variants apart)
    assert any(not np.array_equal(per.idx[b, 0], per.idx[b, 1]) for b in range(B))
    one = oracle.oracle_batch(K[:, :1], Q[:, :2], seq, head_mean=True, **kw)
    ref = oracle.oracle_batch(K[:, :1], Q[:, :2], seq, **kw)
    np.testing.assert_array_equal(one.idx, ref.idx)


def test_gqa_mean_pool_variant():
    """Mean instead of max over the query heads of a group (the pooling the paper's appendix ascribes to earlier work),
    read as Eq. 3 with the max replaced: the attention weights are softmax(mean_g Q^g K^T / sqrt(d)), recomputed here
    with numpy/scipy; G = 1 and a group of identical query heads give the max-pooled result; and on generic inputs
    the two poolings differ (otherwise the pins above would not tell them apart)."""
    from scipy.special import softmax
    rng = np.random.default_rng(91)
    L, alpha, G = 70, 8, 4
    K, Q = _rand(rng, L, D), _rand(rng, G, alpha, D) * 2.0
    n = L - alpha
    mx = _run(K, Q, budget=40, alpha=alpha)
    mp = _run(K, Q, budget=40, alpha=alpha, gqa_mean_pool=True)
    logits = np.einsum("gjc,ic->gji", Q.astype(np.float64), K[:n].astype(np.float64)) / np.sqrt(D)
    np.testing.assert_allclose(mp.A, softmax(logits.mean(axis=0), axis=1), rtol=1e-12, atol=1e-300)
    np.testing.assert_allclose(mx.A, softmax(logits.max(axis=0), axis=1), rtol=1e-12, atol=1e-300)
    np.testing.assert_allclose(mp.A.sum(axis=1), 1.0, rtol=1e-12)
    assert np.abs(mp.A - mx.A).max() > 1e-3
    np.testing.assert_array_equal(mp.S_raw, mx.S_raw)                        # the redundancy side does not change
    one = _rand(rng, 1, alpha, D)
    a = _run(K, one, budget=40, alpha=alpha)
    b = _run(K, one, budget=40, alpha=alpha, gqa_mean_pool=True)
    np.testing.assert_array_equal(a.idx, b.idx)
    np.testing.assert_allclose(a.A, b.A, rtol=1e-15)
    same = np.repeat(one, 3, axis=0)
    c = _run(K, same, budget=40, alpha=alpha, gqa_mean_pool=True)
    np.testing.assert_allclose(c.A, a.A, rtol=1e-12)


def test_append_and_query_ring_semantics():
    """Section 3.1's decode step and Algorithm 1's observation buffer, pinned by what they must leave behind:
    only row seq_lens[b] of each head changes and holds the new token, a full cache stays as it is, alpha pushes
    with slots 0..alpha-1 rebuild the window from the pushed rows, and the scores do not depend on the slot order
    (Eq. 4 averages over the window's rows)."""
    rng = np.random.default_rng(101)
    B, H, cap, alpha = 3, 2, 12, 4
    K, V = _rand(rng, B, H, cap, D), _rand(rng, B, H, cap, D)
    kn, vn = _rand(rng, B, H, D), _rand(rng, B, H, D)
    seq = np.array([5, 12, 0], np.int32)
    k2, v2, s2 = oracle.oracle_append(K, V, kn, vn, seq)
    assert s2.tolist() == [6, 12, 1]
    for b, L in enumerate(seq):
        changed = np.any(k2[b] != K[b], axis=-1) | np.any(v2[b] != V[b], axis=-1)          # [H, cap]
        if L < cap:
            assert changed[:, L].all() and changed.sum() == H
            np.testing.assert_array_equal(k2[b, :, L], kn[b])
            np.testing.assert_array_equal(v2[b, :, L], vn[b])
        else:
            assert not changed.any()
    Hq = 4
    Qw = _rand(rng, B, Hq, alpha, D)
    pushed = [_rand(rng, B, Hq, D) for _ in range(alpha)]
    q = Qw
    for step, row in enumerate(pushed):
        q = oracle.oracle_push_query(q, row, step % alpha)
    np.testing.assert_array_equal(q, np.stack(pushed, axis=2))
    # a rotated window gives the same scores
    Kh = _rand(rng, 40, D)
    a = _run(Kh, q[0], budget=20, alpha=alpha)
    b_ = _run(Kh, np.roll(q[0], 1, axis=1), budget=20, alpha=alpha)
    np.testing.assert_allclose(a.I, b_.I, rtol=1e-12)
    np.testing.assert_array_equal(a.idx, b_.idx)


def test_decode_attention_against_library_softmax_and_closed_forms():
    """Section 3.1's decode step (Eq. 1 with one query row) pinned to what fixes it from outside: scipy's softmax and
    numpy's matrix product per query head with the GQA head mapping written out; one cached token returns its value
    row; identical keys give the mean of the values; adding a constant vector's worth of logit to every key changes
    nothing; tokens at and beyond the cached length are never read (NaN there)."""
    from scipy.special import softmax
    import oracle
    rng = np.random.default_rng(17)
    B, Hkv, Hq, cap, d = 3, 2, 6, 37, 16
    G = Hq // Hkv
    K = rng.standard_normal((B, Hkv, cap, d)).astype(np.float32)
    V = rng.standard_normal((B, Hkv, cap, d)).astype(np.float32)
    q = rng.standard_normal((B, Hq, d)).astype(np.float32)
    seq = np.array([37, 1, 20], dtype=np.int32)
    K[2, :, 20:] = np.nan
    V[2, :, 20:] = np.nan
    out = oracle.oracle_decode_attention(K, V, q, seq)
    for b in range(B):
        L = int(seq[b])
        for h in range(Hq):
            kv = h // G
            w = softmax(q[b, h].astype(np.float64) @ K[b, kv, :L].astype(np.float64).T / np.sqrt(d))
            want = w @ V[b, kv, :L].astype(np.float64)
            assert np.allclose(out[b, h], want, rtol=1e-12, atol=1e-14)
    assert np.allclose(out[1], np.repeat(V[1, :, 0].astype(np.float64), G, axis=0))          # one token: its value row
    Ks = K.copy()
    Ks[0] = Ks[0, :, :1]                                                                     # identical keys
    same = oracle.oracle_decode_attention(Ks, V, q, seq)
    assert np.allclose(same[0], np.repeat(V[0].astype(np.float64).mean(axis=1), G, axis=0))
    # softmax is shift-invariant: a key component that is the same for every token moves every logit alike
    Kc, qc = np.concatenate([K, np.full((B, Hkv, cap, 1), 3.0, np.float32)], -1), \
        np.concatenate([q * np.sqrt((d + 1) / d), np.full((B, Hq, 1), 0.7, np.float32)], -1).astype(np.float32)
    Vc = np.concatenate([V, np.zeros((B, Hkv, cap, 1), np.float32)], -1)
    Kc[2, :, 20:] = np.nan
    shifted = oracle.oracle_decode_attention(Kc, Vc, qc, seq)
    assert np.allclose(shifted[..., :d], out, rtol=1e-5, atol=1e-6)
    empty = oracle.oracle_decode_attention(K, V, q, np.array([0, 0, 0], dtype=np.int32))
    assert not empty.any()


def test_per_sequence_budgets_equal_independent_calls():
    """Budgets of their own per sequence (Section 4.2's budget ratios): every sequence's result is the one a call with
    that budget alone gives, index rows are padded with -1 beyond the sequence's budget, and a sequence at or below its
    budget is left alone."""
    import oracle
    rng = np.random.default_rng(23)
    B, Hkv, Hq, cap, d, alpha = 3, 2, 4, 60, 16, 4
    K = rng.standard_normal((B, Hkv, cap, d)).astype(np.float32)
    Q = rng.standard_normal((B, Hq, alpha, d)).astype(np.float32)
    seq = np.array([60, 50, 33], dtype=np.int32)
    budgets = np.array([40, 24, 33], dtype=np.int32)
    kw = dict(alpha=alpha, lam=0.1, W=2, beta=1, T=0.3)
    res = oracle.oracle_batch(K, Q, seq, budget=40, budgets=budgets, **kw)
    assert res.compressed.tolist() == [True, True, False]
    for b in range(B):
        one = oracle.oracle_batch(K[b:b + 1], Q[b:b + 1], seq[b:b + 1], budget=int(budgets[b]), **kw)
        nb = int(budgets[b])
        assert np.array_equal(res.idx[b, :, :nb], one.idx[0])
        assert (res.idx[b, :, nb:] == -1).all()
        assert np.array_equal(res.Z[b], one.Z[0])
    kept = res.idx[1, 0, :24]
    assert np.all(np.diff(kept) > 0) and np.array_equal(kept[-alpha:], np.arange(46, 50))    # 24 kept, observation tail
    assert np.array_equal(res.idx[2, 0, :33], np.arange(33))                                 # L = budget: the guard


# ----------------------------------------------------------------------------- 8-bit (E4M3) cache codes
def test_e4m3_decode_against_the_format_and_the_library_cast():
    """An 8-bit cache holds E4M3 codes; the oracle scores the values they stand for.  The decode is pinned to the
    format's own landmarks (1.0, the largest finite value 448, the smallest subnormal 2^-9, the smallest normal 2^-6,
    the NaN code), to the library's cast for all 256 codes, and to the ordering of the positive codes."""
    import torch
    vals = oracle.e4m3_to_f32(np.arange(256, dtype=np.uint8))
    assert vals[0x00] == 0.0 and vals[0x80] == 0.0 and np.signbit(vals[0x80])
    assert vals[0x38] == 1.0 and vals[0xB8] == -1.0 and vals[0x40] == 2.0 and vals[0x3C] == 1.5
    assert vals[0x7E] == 448.0 and vals[0x01] == 2.0 ** -9 and vals[0x07] == 7 * 2.0 ** -9 and vals[0x08] == 2.0 ** -6
    assert np.isnan(vals[0x7F]) and np.isnan(vals[0xFF])
    lib = torch.arange(256, dtype=torch.uint8).view(torch.float8_e4m3fn).to(torch.float32).numpy()
    finite = ~np.isnan(lib)
    assert np.array_equal(np.isnan(vals), np.isnan(lib))
    assert np.array_equal(vals[finite].view(np.uint32), lib[finite].view(np.uint32))       # bit for bit, -0 included
    assert np.all(np.diff(vals[:0x7F]) > 0)           # positive codes are ordered like their values


def test_e4m3_cache_scores_are_the_scores_of_the_decoded_values():
    """Nothing of Eq. 1-7 changes for an 8-bit cache: the head result on codes decoded by the oracle equals the
    result on the same values given as float32 by the library's cast, and the kept rows are moved as bytes."""
    import torch
    rng = np.random.default_rng(77)
    L, alpha, budget = 96, 8, 40
    K32 = _rand(rng, L, D)
    codes = torch.from_numpy(K32).to(torch.float8_e4m3fn).view(torch.uint8).numpy()
    Kd = oracle.e4m3_to_f32(codes)
    Kl = torch.from_numpy(codes).view(torch.float8_e4m3fn).to(torch.float32).numpy()
    Q = _rand(rng, 2, alpha, D)
    a, b = _run(Kd, Q, budget=budget, alpha=alpha), _run(Kl, Q, budget=budget, alpha=alpha)
    assert np.array_equal(a.idx, b.idx) and np.array_equal(a.Z, b.Z)
    moved = oracle.oracle_gather(codes, a.idx)
    assert moved.dtype == np.uint8 and np.array_equal(moved, codes[a.idx])
    # quantisation is not a no-op on these inputs: the 8-bit values differ from the float32 ones they came from
    assert np.abs(Kd - K32).max() > 1e-3

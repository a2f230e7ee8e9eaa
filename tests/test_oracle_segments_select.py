"""Pins for the oracle's packed-segment statistics and the Delta-IFD rule
(Eq. 3, Eq. 4, three-zone rule): unpacked per-sequence runs, a hand-worked
table, invariances and edge cases.  CPU only."""

import math
import os

import numpy as np
import pytest

from oracle import npd_oracle as orc

GOLDEN = os.path.join(os.path.dirname(__file__), "golden", "delta_ifd_table.txt")


def _packed(seed=0):
    rng = np.random.default_rng(seed)
    lens = [5, 1, 9, 3, 7]
    cu = np.concatenate([[0], np.cumsum(lens)]).astype(np.int32)
    T, d, V = int(cu[-1]), 4, 10
    H = rng.standard_normal((T, d))
    W = rng.standard_normal((V, d))
    Zt = rng.standard_normal((T, V)) * 2
    y = rng.integers(0, V, size=T)
    m = (rng.random(T) < 0.6).astype(np.uint8)
    for s in range(len(lens)):
        y[cu[s + 1] - 1] = -100
        m[cu[s + 1] - 1] = 0
    y[2] = -100            # an ignored label on a token that still carries KL
    m[2] = 1
    return cu, H, W, Zt, y, m


def test_segment_sums_equal_unpacked_per_sequence_runs():
    cu, H, W, Zt, y, m = _packed()
    kl, ns, nt = orc.kd_token_losses(H, W, Zt, y, m, 1.5)
    kl_sum, s_sum, t_sum, cnt = orc.segment_stats(cu, m, y, kl, ns, nt)
    for s in range(len(cu) - 1):
        sl = slice(cu[s], cu[s + 1])
        k1, s1, t1 = orc.kd_token_losses(H[sl], W, Zt[sl], y[sl], m[sl], 1.5)
        assert math.isclose(kl_sum[s], k1.sum(), rel_tol=1e-13, abs_tol=1e-15)
        assert math.isclose(s_sum[s], s1.sum(), rel_tol=1e-13, abs_tol=1e-15)
        assert math.isclose(t_sum[s], t1.sum(), rel_tol=1e-13, abs_tol=1e-15)
        assert cnt[s] == int(((m[sl] == 1) & (y[sl] >= 0)).sum())
    assert cnt.dtype == np.int32
    assert cnt.sum() == int(((m == 1) & (y >= 0)).sum())
    assert math.isclose(kl_sum.sum(), kl.sum(), rel_tol=1e-13)


def test_count_excludes_ignored_labels_but_kl_sum_does_not():
    cu, H, W, Zt, y, m = _packed()
    kl, ns, nt = orc.kd_token_losses(H, W, Zt, y, m, 1.0)
    kl_sum, _, _, cnt = orc.segment_stats(cu, m, y, kl, ns, nt)
    seg0 = slice(cu[0], cu[1])
    assert cnt[0] == int(((m[seg0] == 1) & (y[seg0] >= 0)).sum())
    assert kl[2] > 0 and ns[2] == 0          # token 2: KL but no label
    assert kl_sum[0] >= kl[2]


def test_permuting_segments_permutes_statistics():
    cu, H, W, Zt, y, m = _packed(3)
    kl, ns, nt = orc.kd_token_losses(H, W, Zt, y, m, 1.0)
    base = orc.segment_stats(cu, m, y, kl, ns, nt)
    perm = [3, 0, 4, 2, 1]
    idx = np.concatenate([np.arange(cu[s], cu[s + 1]) for s in perm])
    cu_p = np.concatenate([[0], np.cumsum([cu[s + 1] - cu[s] for s in perm])])
    got = orc.segment_stats(cu_p, m[idx], y[idx], kl[idx], ns[idx], nt[idx])
    for a, b in zip(base, got):
        assert np.allclose(np.asarray(a)[perm], b, rtol=1e-14)


def test_segment_ids_and_validation():
    cu = np.array([0, 2, 3, 7], dtype=np.int32)
    assert orc.segment_ids(cu, 7).tolist() == [0, 0, 1, 2, 2, 2, 2]
    assert orc.segment_ids(cu, 7).dtype == np.int32
    assert orc.validate_cu_seqlens(cu, 7)
    assert not orc.validate_cu_seqlens(cu, 8)                  # does not end at T
    assert not orc.validate_cu_seqlens([1, 2, 7], 7)           # does not start at 0
    assert not orc.validate_cu_seqlens([0, 3, 3, 7], 7)        # empty segment
    assert not orc.validate_cu_seqlens([0, 5, 4, 7], 7)        # not increasing
    assert not orc.validate_cu_seqlens([0], 0)


def _read_golden():
    rows = []
    with open(GOLDEN) as f:
        for line in f:
            line = line.strip()
            if not line or line.startswith("#"):
                continue
            left, right = line.split("|")
            l, r = left.split(), right.split()
            rows.append(dict(cc=int(l[1]), cu=int(l[2]), tc=float(l[3]), tu=float(l[4]),
                             sc=float(l[5]), su=float(l[6]), ifd_t=float(r[0]), ifd_s=float(r[1]),
                             delta=float(r[2]), keep=int(r[3]), keep2=int(r[4])))
    return rows


@pytest.mark.parametrize("dtype", [np.float64, np.float32])
def test_hand_worked_table(dtype):
    rows = _read_golden()
    n = len(rows)
    count = np.zeros(2 * n, dtype=np.int32)
    t_sum = np.zeros(2 * n)
    s_sum = np.zeros(2 * n)
    for i, r in enumerate(rows):
        count[2 * i], count[2 * i + 1] = r["cc"], r["cu"]
        t_sum[2 * i], t_sum[2 * i + 1] = r["tc"], r["tu"]
        s_sum[2 * i], s_sum[2 * i + 1] = r["sc"], r["su"]
    cond = np.arange(n) * 2
    unc = cond + 1
    it, is_, dl, keep, nk = orc.delta_ifd_select(cond, unc, s_sum, t_sum, count, 0.0, 1.0,
                                                 dtype=dtype)
    assert it.dtype == dtype and dl.dtype == dtype and keep.dtype == np.uint8
    for i, r in enumerate(rows):
        for got, want in ((it[i], r["ifd_t"]), (is_[i], r["ifd_s"]), (dl[i], r["delta"])):
            assert (math.isnan(got) and math.isnan(want)) or got == want
        assert keep[i] == r["keep"]
    assert nk == sum(r["keep"] for r in rows)
    _, _, _, keep2, nk2 = orc.delta_ifd_select(cond, unc, s_sum, t_sum, count, 0.0, 1.0,
                                               require_teacher_ifd_le_1=True, dtype=dtype)
    assert keep2.tolist() == [r["keep2"] for r in rows]
    assert nk2 == sum(r["keep2"] for r in rows)


def test_teacher_equal_to_student_is_kept_and_scaling_leaves_delta_unchanged():
    rng = np.random.default_rng(0)
    n = 8
    count = rng.integers(1, 20, size=2 * n).astype(np.int32)
    s_sum = rng.random(2 * n) * 10 + 0.1
    cond, unc = np.arange(n) * 2, np.arange(n) * 2 + 1
    _, _, dl, keep, nk = orc.delta_ifd_select(cond, unc, s_sum, s_sum, count, 0.0, 0.8)
    assert np.all(dl == 0) and np.all(keep == 1) and nk == n
    t_sum = rng.random(2 * n) * 10 + 0.1
    base = orc.delta_ifd_select(cond, unc, s_sum, t_sum, count, 0.0, 0.8)
    scale = np.repeat(rng.random(n) * 5 + 0.5, 2)       # one constant per sample
    scaled = orc.delta_ifd_select(cond, unc, s_sum * scale, t_sum * scale, count, 0.0, 0.8)
    assert np.allclose(base[2], scaled[2], rtol=1e-12)
    assert np.array_equal(base[3], scaled[3])


def test_ifd_is_ratio_of_token_means_not_sums():
    # cond: 4 tokens summing to 8 (mean 2); uncond: 2 tokens summing to 8 (mean 4)
    ifd = orc.ifd_scores([0], [1], [8.0, 8.0], [4, 2])
    assert ifd[0] == 0.5


def test_pair_maps_are_arbitrary_indices():
    count = np.array([2, 4, 1, 8], dtype=np.int32)
    s = np.array([2.0, 4.0, 3.0, 8.0])
    t = np.array([4.0, 4.0, 1.0, 4.0])
    it, is_, dl, keep, nk = orc.delta_ifd_select([3, 0], [2, 1], s, t, count, 0.0, 1.0)
    # sample 0: cond=3, unc=2 -> T: (4/8)/(1/1)=0.5 ; S: (8/8)/(3/1)=1/3
    assert it[0] == 0.5 and math.isclose(is_[0], 1 / 3)
    # sample 1: cond=0, unc=1 -> T: (4/2)/(4/4)=2 ; S: (2/2)/(4/4)=1
    assert it[1] == 2.0 and is_[1] == 1.0 and dl[1] == 1.0 and keep[1] == 1
    assert nk == 2


def test_zero_denominator_and_empty_are_rejected():
    count = np.array([3, 3, 0, 2], dtype=np.int32)
    z = np.array([1.0, 0.0, 0.0, 1.0])
    it, is_, dl, keep, nk = orc.delta_ifd_select([0, 2], [1, 3], z, z, count, -10, 10)
    assert np.all(np.isnan(dl)) and keep.tolist() == [0, 0] and nk == 0


def test_nearest_rank_percentile():
    assert orc.nearest_rank_percentile([5, 1, 3, 2, 4], 0.8) == 4
    assert orc.nearest_rank_percentile([5, 1, 3, 2, 4], 0.81) == 5
    assert orc.nearest_rank_percentile([1, float("nan"), 2, 3, 4, 5], 0.2) == 1
    assert orc.nearest_rank_percentile(np.arange(1, 11), 0.8) == 8


def test_filter_ablation_scopes_on_the_hand_worked_table():
    rows = _read_golden()
    n = len(rows)
    count = np.zeros(2 * n, dtype=np.int32)
    t_sum, s_sum = np.zeros(2 * n), np.zeros(2 * n)
    for i, r in enumerate(rows):
        count[2 * i], count[2 * i + 1] = r["cc"], r["cu"]
        t_sum[2 * i], t_sum[2 * i + 1] = r["tc"], r["tu"]
        s_sum[2 * i], s_sum[2 * i + 1] = r["sc"], r["su"]
    cond = np.arange(n) * 2
    unc = cond + 1
    want = []
    path = os.path.join(os.path.dirname(__file__), "golden", "filter_variants_table.txt")
    for line in open(path):
        if line.strip() and not line.startswith("#"):
            want.append([int(x) for x in line.split("|")[1].split()])
    want = np.asarray(want)
    inf = float("inf")
    variants = [dict(score="ifd_teacher", lo=0.0, hi=1.0), dict(score="ifd_student", lo=0.0, hi=1.0),
                dict(score="delta", lo=0.0, hi=inf, lo_inclusive=False),
                dict(score="delta", lo=-inf, hi=1.0, hi_inclusive=False),
                dict(score="delta", lo=0.0, hi=1.0)]
    for col, v in enumerate(variants):
        for dtype in (np.float64, np.float32):
            keep = orc.delta_ifd_select(cond, unc, s_sum, t_sum, count, dtype=dtype, **v)[3]
            assert keep.tolist() == want[:, col].tolist(), v


def test_reverse_kl_is_the_forward_kl_with_the_roles_swapped():
    # D(learner || generator) computed by the monitor = Eq. 2's divergence with the learner's
    # logits in the teacher's seat and the generator's logits produced by an identity head
    rng = np.random.default_rng(9)
    T, d, V = 7, 5, 6
    H, W = rng.standard_normal((T, d)), rng.standard_normal((V, d))
    G = rng.standard_normal((T, V)) * 2
    m = np.array([1, 0, 1, 1, 1, 0, 1], dtype=np.uint8)
    for tau in (1.0, 1.7):
        rkl = orc.reverse_kl_token(H, W, G, m, tau)
        swapped, _, _ = orc.kd_token_losses(G, np.eye(V), H @ W.T, np.full(T, -1), m, tau)
        assert np.allclose(rkl, swapped, atol=1e-13)
        assert np.all(rkl >= 0) and np.all(rkl[m == 0] == 0)
    assert np.abs(orc.reverse_kl_token(H, W, H @ W.T + 3.0, m)).max() < 1e-12   # same policy, shifted logits
    fwd, _, _ = orc.kd_token_losses(H, W, G, np.full(T, -1), m, 1.0)
    assert not np.allclose(fwd, orc.reverse_kl_token(H, W, G, m))              # the direction matters
    from scipy.special import rel_entr, softmax
    ref = rel_entr(softmax(H @ W.T, axis=1), softmax(G, axis=1)).sum(axis=1) * m
    assert np.allclose(orc.reverse_kl_token(H, W, G, m), ref, atol=1e-13)


# ----------------------------------------------------------------------------------------------
# Pack(D_select, Length = L): first-fit decreasing
# ----------------------------------------------------------------------------------------------
def _min_rows_brute_force(sizes, cap):
    """Smallest number of rows of capacity cap that hold all sizes (tiny inputs only)."""
    best = [len(sizes)]
    def place(k, room):
        if len(room) >= best[0]:
            return
        if k == len(sizes):
            best[0] = len(room)
            return
        for r in range(len(room)):
            if room[r] >= sizes[k]:
                room[r] -= sizes[k]
                place(k + 1, room)
                room[r] += sizes[k]
        room.append(cap - sizes[k])
        place(k + 1, room)
        room.pop()
    place(0, [])
    return best[0]


def test_packing_worked_example():
    # lengths 5 4 3 3 2 into rows of 8, all kept: 5 opens row 0, 4 opens row 1, the first 3 joins
    # row 0 (5+3), the second 3 joins row 1 (4+3), 2 fits nowhere (rooms 0 and 1) -> row 2
    order, row_of, cu, ptr = orc.pack_first_fit_decreasing([3, 5, 2, 4, 3], None, 8)
    assert order.tolist() == [1, 0, 3, 4, 2] and row_of.tolist() == [0, 0, 1, 1, 2]
    assert cu.tolist() == [0, 5, 8, 12, 15, 17] and ptr.tolist() == [0, 2, 4, 5]


def test_packing_invariants_and_quality():
    rng = np.random.default_rng(3)
    for trial in range(30):
        n = int(rng.integers(1, 9))
        cap = int(rng.integers(4, 12))
        lengths = rng.integers(0, cap + 3, size=n)
        keep = rng.random(n) < 0.8
        order, row_of, cu, ptr = orc.pack_first_fit_decreasing(lengths, keep, cap)
        want = sorted(i for i in range(n) if keep[i] and lengths[i] > 0)
        assert sorted(order.tolist()) == want                       # every kept sample exactly once
        sizes = np.minimum(lengths[order], cap)
        assert np.array_equal(np.diff(cu), sizes)
        for r in range(len(ptr) - 1):
            assert sizes[ptr[r]:ptr[r + 1]].sum() <= cap             # no row overflows
            assert np.all(row_of[ptr[r]:ptr[r + 1]] == r)
        if want:
            opt = _min_rows_brute_force(sorted(np.minimum(lengths[want], cap).tolist(), reverse=True), cap)
            rows = len(ptr) - 1
            assert opt <= rows <= (11 * opt + 6) // 9 + 1            # the known first-fit-decreasing bound


# --------------------------------------------------------------------------- #
# Per-sample perplexity (filter ablation, row "Perplexity (PPL)")
# --------------------------------------------------------------------------- #

def _ppl_table():
    rows = []
    with open(os.path.join(os.path.dirname(GOLDEN), "perplexity_table.txt")) as f:
        for ln in f:
            if ln.startswith("#") or not ln.strip():
                continue
            left, right = ln.split("|")
            seg, cnt, s = left.split()
            rows.append((int(seg), int(cnt), float(s), float(right.split()[0])))
    return rows


def test_perplexity_matches_the_hand_worked_table():
    rows = _ppl_table()
    cnt = np.asarray([r[1] for r in rows])
    sums = np.asarray([r[2] for r in rows])
    want = np.asarray([r[3] for r in rows])
    got = orc.perplexity_scores(np.arange(len(rows)), sums, cnt)
    assert np.array_equal(np.isnan(got), np.isnan(want))
    ok = ~np.isnan(want)
    assert np.allclose(got[ok], want[ok], rtol=1e-14, atol=0)
    # the segment index really selects: a permuted request gives the permuted scores
    perm = np.asarray([5, 0, 3])
    assert np.allclose(orc.perplexity_scores(perm, sums, cnt), want[perm], rtol=1e-14)
    # float32 mode: the same two operations in float32
    g32 = orc.perplexity_scores(np.arange(len(rows)), sums, cnt, dtype=np.float32)
    assert g32.dtype == np.float32 and np.allclose(g32[ok], want[ok], rtol=1e-6)


def test_perplexity_is_the_inverse_geometric_mean_of_the_label_probabilities():
    # independent restatement: PPL = (prod_t p(y_t))^(-1/n), with the probabilities taken from a
    # softmax written out here, through the whole chain losses -> segment sums -> score
    rng = np.random.default_rng(5)
    T, d, V = 14, 5, 9
    H, W = rng.standard_normal((T, d)), rng.standard_normal((V, d))
    Z = rng.standard_normal((T, V))
    y = rng.integers(0, V, size=T)
    m = np.ones(T, dtype=np.uint8)
    cu = np.asarray([0, 5, 6, 14])
    y[4] = y[5] = y[13] = -100
    m[[4, 5, 13]] = 0
    m[7] = 0                                   # a masked token inside a segment
    kl, ns, nt = orc.kd_token_losses(H, W, Z, y, m, 1.0)
    _, s_sum, t_sum, cnt = orc.segment_stats(cu, m, y, kl, ns, nt)
    ppl_s = orc.perplexity_scores([0, 1, 2], s_sum, cnt)
    ppl_t = orc.perplexity_scores([0, 1, 2], t_sum, cnt)
    O_S = H @ W.T
    pS = np.exp(O_S) / np.exp(O_S).sum(1, keepdims=True)
    pT = np.exp(Z) / np.exp(Z).sum(1, keepdims=True)
    for s, (a, b) in enumerate(zip(cu[:-1], cu[1:])):
        tok = [t for t in range(a, b) if m[t] and y[t] >= 0]
        if not tok:
            assert np.isnan(ppl_s[s]) and np.isnan(ppl_t[s])
            continue
        gs = np.prod([pS[t, y[t]] for t in tok]) ** (-1.0 / len(tok))
        gt = np.prod([pT[t, y[t]] for t in tok]) ** (-1.0 / len(tok))
        assert np.isclose(ppl_s[s], gs, rtol=1e-12) and np.isclose(ppl_t[s], gt, rtol=1e-12)


def test_perplexity_of_a_uniform_model_is_the_vocabulary_size():
    T, d, V = 6, 3, 37
    H, W = np.zeros((T, d)), np.zeros((V, d))          # uniform student
    Z = np.full((T, V), 0.25)                          # uniform teacher
    y = np.arange(T) % V
    m = np.ones(T, dtype=np.uint8)
    kl, ns, nt = orc.kd_token_losses(H, W, Z, y, m, 1.0)
    _, s_sum, t_sum, cnt = orc.segment_stats([0, 2, 6], m, y, kl, ns, nt)
    assert np.allclose(orc.perplexity_scores([0, 1], s_sum, cnt), V, rtol=1e-12)
    assert np.allclose(orc.perplexity_scores([0, 1], t_sum, cnt), V, rtol=1e-12)


# --------------------------------------------------------------------------- #
# Input validation (what the debug mode of the step checks)
# --------------------------------------------------------------------------- #

def test_validate_step_inputs_literal_cases():
    V = 6
    H = np.ones((4, 3))
    Z = np.zeros((4, V))
    y = np.asarray([0, 5, -100, 2])
    m = np.asarray([1, 1, 0, 1], dtype=np.uint8)
    ok = lambda **kw: orc.validate_step_inputs(kw.get("H", H), kw.get("Z", Z), kw.get("y", y), kw.get("m", m), V,
                                               kw.get("idx"))
    assert ok()
    assert not ok(y=np.asarray([0, 6, -100, 2]))                 # a label that names no class
    assert ok(y=np.asarray([0, 5, -7, 2]))                       # any negative label means "none"
    Zi = Z.copy(); Zi[1, :] = -np.inf
    assert not ok(Z=Zi)                                          # a loss token without any support
    Zi = Z.copy(); Zi[1, :5] = -np.inf
    assert ok(Z=Zi)                                              # one class left: fine
    Zi = Z.copy(); Zi[2, :] = -np.inf
    assert ok(Z=Zi)                                              # the masked token's row is never read
    Zi = Z.copy(); Zi[0, 3] = np.nan
    assert not ok(Z=Zi)
    Zi = Z.copy(); Zi[3, 0] = np.inf
    assert not ok(Z=Zi)
    Hi = H.copy(); Hi[3, 1] = np.inf
    assert not ok(H=Hi)
    Hi = H.copy(); Hi[2, 1] = np.nan
    assert ok(H=Hi)                                              # masked token again
    idx = np.asarray([[0, 5], [1, 2], [9, 9], [3, 4]])
    assert ok(idx=idx)                                           # row 2 is masked
    assert not ok(idx=np.asarray([[0, 6], [1, 2], [0, 0], [3, 4]]))
    assert not ok(idx=np.asarray([[0, 5], [-1, 2], [0, 0], [3, 4]]))

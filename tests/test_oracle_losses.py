"""Pins for the oracle's per-token losses (Eq. 2 and the cross-entropy of Eq. 3):
closed forms, invariances, library routines and brute force.  CPU only."""

import math

import numpy as np
import pytest
import scipy.special as sps
import torch

from oracle import npd_oracle as orc


def _rand_problem(seed, T=7, d=5, V=11, zt_std=2.0):
    rng = np.random.default_rng(seed)
    H = rng.standard_normal((T, d))
    W = rng.standard_normal((V, d)) * 0.5
    Zt = rng.standard_normal((T, V)) * zt_std
    labels = rng.integers(0, V, size=T)
    mask = np.ones(T, dtype=np.uint8)
    return H, W, Zt, labels, mask


def test_kl_nonnegative_and_zero_when_teacher_equals_student():
    H, W, Zt, y, m = _rand_problem(1, T=40, d=8, V=33)
    for tau in (1.0, 0.7, 2.5):
        kl, _, _ = orc.kd_token_losses(H, W, Zt, y, m, tau)
        assert np.all(kl > 0)
        kl0, nll_s, nll_t = orc.kd_token_losses(H, W, H @ W.T, y, m, tau)
        assert np.max(np.abs(kl0)) < 1e-12
        assert np.allclose(nll_s, nll_t, rtol=0, atol=1e-12)


def test_kl_invariant_to_row_shift_of_either_logit_row():
    H, W, Zt, y, m = _rand_problem(2)
    kl, _, nll_t = orc.kd_token_losses(H, W, Zt, y, m, 1.3)
    shift = np.linspace(-30, 30, Zt.shape[0])[:, None]
    kl2, _, nll_t2 = orc.kd_token_losses(H, W, Zt + shift, y, m, 1.3)
    assert np.allclose(kl, kl2, rtol=1e-10, atol=1e-12)
    assert np.allclose(nll_t, nll_t2, rtol=1e-10, atol=1e-12)
    # student shift: append a constant feature to H and a constant column to W
    Hs = np.concatenate([H, np.ones((H.shape[0], 1))], axis=1)
    Ws = np.concatenate([W, np.full((W.shape[0], 1), 4.25)], axis=1)
    kl3, _, _ = orc.kd_token_losses(Hs, Ws, Zt, y, m, 1.3)
    assert np.allclose(kl, kl3, rtol=1e-10, atol=1e-12)


def test_temperature_is_a_rescaling_of_both_logit_sets():
    H, W, Zt, y, m = _rand_problem(3)
    tau = 2.0
    kl_tau, _, _ = orc.kd_token_losses(H, W, Zt, y, m, tau)
    kl_one, _, _ = orc.kd_token_losses(H / tau, W, Zt / tau, y, m, 1.0)
    assert np.allclose(kl_tau, kl_one, rtol=1e-12, atol=1e-14)
    # and it matters: tau=1 differs
    kl_1, _, _ = orc.kd_token_losses(H, W, Zt, y, m, 1.0)
    assert not np.allclose(kl_tau, kl_1, rtol=1e-3)


def test_nll_is_not_tempered():
    H, W, Zt, y, m = _rand_problem(4)
    _, s1, t1 = orc.kd_token_losses(H, W, Zt, y, m, 1.0)
    _, s2, t2 = orc.kd_token_losses(H, W, Zt, y, m, 3.0)
    assert np.array_equal(s1, s2) and np.array_equal(t1, t2)


def test_uniform_student_closed_form():
    # H = 0 gives a uniform p_S: KL = log V - entropy(p_T).
    _, W, Zt, y, m = _rand_problem(5, T=9, V=13)
    H = np.zeros((9, 5))
    kl, nll_s, _ = orc.kd_token_losses(H, W, Zt, y, m, 1.0)
    p = sps.softmax(Zt, axis=1)
    ent = -(p * np.log(p)).sum(1)
    assert np.allclose(kl, math.log(13) - ent, rtol=1e-12)
    assert np.allclose(nll_s, math.log(13), rtol=1e-12)


def test_two_class_case_is_binary_kl_of_sigmoids():
    rng = np.random.default_rng(6)
    T = 12
    H = rng.standard_normal((T, 3))
    W = rng.standard_normal((2, 3))
    Zt = rng.standard_normal((T, 2)) * 3
    kl, nll_s, nll_t = orc.kd_token_losses(H, W, Zt, np.zeros(T, int), np.ones(T), 1.0)
    zs = H @ W.T
    p = 1 / (1 + np.exp(-(Zt[:, 0] - Zt[:, 1])))
    q = 1 / (1 + np.exp(-(zs[:, 0] - zs[:, 1])))
    ref = p * np.log(p / q) + (1 - p) * np.log((1 - p) / (1 - q))
    assert np.allclose(kl, ref, rtol=1e-11)
    assert np.allclose(nll_s, -np.log(q), rtol=1e-11)
    assert np.allclose(nll_t, -np.log(p), rtol=1e-11)


def test_against_scipy_rel_entr_and_torch_kl_div():
    H, W, Zt, y, m = _rand_problem(7, T=16, d=6, V=50)
    tau = 1.7
    kl, nll_s, nll_t = orc.kd_token_losses(H, W, Zt, y, m, tau)
    zs = H @ W.T
    ref = sps.rel_entr(sps.softmax(Zt / tau, axis=1), sps.softmax(zs / tau, axis=1)).sum(1)
    assert np.allclose(kl, ref, rtol=1e-11)
    lt = torch.log_softmax(torch.from_numpy(Zt) / tau, dim=1)
    ls = torch.log_softmax(torch.from_numpy(zs) / tau, dim=1)
    ref_t = torch.nn.functional.kl_div(ls, lt, reduction="none", log_target=True).sum(1)
    assert np.allclose(kl, ref_t.numpy(), rtol=1e-11)
    ce_s = torch.nn.functional.cross_entropy(torch.from_numpy(zs), torch.from_numpy(y),
                                             reduction="none")
    ce_t = torch.nn.functional.cross_entropy(torch.from_numpy(Zt), torch.from_numpy(y),
                                             reduction="none")
    assert np.allclose(nll_s, ce_s.numpy(), rtol=1e-11)
    assert np.allclose(nll_t, ce_t.numpy(), rtol=1e-11)


def test_brute_force_python_loops():
    H, W, Zt, y, m = _rand_problem(8, T=3, d=2, V=5)
    tau = 0.9
    kl, nll_s, nll_t = orc.kd_token_losses(H, W, Zt, y, m, tau)
    for t in range(3):
        zs = [sum(H[t, k] * W[c, k] for k in range(2)) for c in range(5)]
        es = [math.exp(v / tau) for v in zs]
        et = [math.exp(v / tau) for v in Zt[t]]
        ps = [e / sum(es) for e in es]
        pt = [e / sum(et) for e in et]
        ref = sum(a * math.log(a / b) for a, b in zip(pt, ps))
        assert abs(kl[t] - ref) < 1e-12
        e1 = [math.exp(v) for v in zs]
        assert abs(nll_s[t] + math.log(e1[y[t]] / sum(e1))) < 1e-12
        e2 = [math.exp(v) for v in Zt[t]]
        assert abs(nll_t[t] + math.log(e2[y[t]] / sum(e2))) < 1e-12


def test_kl_direction_is_teacher_to_student():
    # forward KL(teacher || student) is asymmetric: swapping roles changes it.
    H, W, Zt, y, m = _rand_problem(9, T=5, d=4, V=9)
    zs = H @ W.T
    kl, _, _ = orc.kd_token_losses(H, W, Zt, y, m, 1.0)
    pt, ps = sps.softmax(Zt, axis=1), sps.softmax(zs, axis=1)
    fwd = (pt * np.log(pt / ps)).sum(1)
    rev = (ps * np.log(ps / pt)).sum(1)
    assert np.allclose(kl, fwd, rtol=1e-11)
    assert not np.allclose(kl, rev, rtol=1e-2)


def test_minus_inf_teacher_entries_reproduce_the_top_k_support_form():
    # Eq. 2 over the teacher's top-k support, teacher renormalised on the k
    # stored logits, student softmax over the full vocabulary.
    H, W, Zt, y, m = _rand_problem(10, T=6, d=4, V=20)
    k = 4
    zs = H @ W.T
    ps = sps.softmax(zs, axis=1)
    dense = np.full_like(Zt, -np.inf)
    ref = np.zeros(6)
    for t in range(6):
        idx = np.argsort(-Zt[t])[:k]
        dense[t, idx] = Zt[t, idx]
        pt = sps.softmax(Zt[t, idx])
        ref[t] = np.sum(pt * np.log(pt / ps[t, idx]))
    kl, _, _ = orc.kd_token_losses(H, W, dense, y, m, 1.0)
    assert np.all(np.isfinite(kl))
    assert np.allclose(kl, ref, rtol=1e-11)
    # lower bound of that form: KL >= -log(sum of student mass on the support)
    assert np.all(kl >= -np.log([ps[t, np.isfinite(dense[t])].sum() for t in range(6)]) - 1e-12)


def test_masks_and_ignored_labels_zero_the_outputs():
    H, W, Zt, y, m = _rand_problem(11, T=10)
    m = np.array([1, 0, 1, 1, 0, 1, 1, 1, 0, 1], dtype=np.uint8)
    y = y.copy()
    y[2] = -100
    kl, nll_s, nll_t = orc.kd_token_losses(H, W, Zt, y, m, 1.0)
    assert np.all(kl[m == 0] == 0) and np.all(kl[m == 1] > 0)
    assert nll_s[2] == 0 and nll_t[2] == 0 and kl[2] > 0
    assert np.all(nll_s[m == 0] == 0) and np.all(nll_t[m == 0] == 0)
    on = (m == 1) & (y >= 0)
    assert np.all(nll_s[on] > 0) and np.all(nll_t[on] > 0)


def test_teacher_columns_beyond_vocab_are_ignored():
    H, W, Zt, y, m = _rand_problem(12)
    pad = np.concatenate([Zt, np.full((Zt.shape[0], 5), 99.0)], axis=1)
    a = orc.kd_token_losses(H, W, Zt, y, m, 1.0)
    b = orc.kd_token_losses(H, W, pad, y, m, 1.0)
    for x, z in zip(a, b):
        assert np.array_equal(x, z)


def test_log_softmax_normalises():
    x = np.random.default_rng(0).standard_normal((4, 9)) * 50
    assert np.allclose(np.exp(orc.log_softmax(x)).sum(1), 1.0, rtol=1e-12)
    assert np.allclose(orc.log_softmax(x), sps.log_softmax(x, axis=1), rtol=1e-12, atol=1e-12)

"""Pins for the oracle's gradients: finite differences of the loss the oracle
itself defines, torch autograd of an independently written loss, and the
structural identities the gradient of a softmax/KL must satisfy.  CPU only."""

import numpy as np
import pytest
import torch

from oracle import npd_oracle as orc


def _problem(seed, T=6, d=5, V=7):
    rng = np.random.default_rng(seed)
    H = rng.standard_normal((T, d))
    W = rng.standard_normal((V, d)) * 0.7
    Zt = rng.standard_normal((T, V)) * 2
    mask = (rng.random(T) < 0.7).astype(np.uint8)
    mask[0] = 1
    mask[1] = 0
    y = rng.integers(0, V, size=T)
    return H, W, Zt, mask, y


def _loss(H, W, Zt, mask, y, tau, g):
    kl, _, _ = orc.kd_token_losses(H, W, Zt, y, mask, tau)
    return g * kl.sum()


@pytest.mark.parametrize("tau,g", [(1.0, 1.0), (2.5, 0.37), (0.6, 1 / 3)])
def test_central_finite_differences(tau, g):
    H, W, Zt, mask, y = _problem(0)
    dH, dW = orc.kd_backward(H, W, Zt, mask, tau, g)
    h = 1e-5
    fdH = np.zeros_like(H)
    for i in range(H.shape[0]):
        for j in range(H.shape[1]):
            Hp, Hm = H.copy(), H.copy()
            Hp[i, j] += h
            Hm[i, j] -= h
            fdH[i, j] = (_loss(Hp, W, Zt, mask, y, tau, g) - _loss(Hm, W, Zt, mask, y, tau, g)) / (2 * h)
    fdW = np.zeros_like(W)
    for i in range(W.shape[0]):
        for j in range(W.shape[1]):
            Wp, Wm = W.copy(), W.copy()
            Wp[i, j] += h
            Wm[i, j] -= h
            fdW[i, j] = (_loss(H, Wp, Zt, mask, y, tau, g) - _loss(H, Wm, Zt, mask, y, tau, g)) / (2 * h)
    assert np.linalg.norm(fdH - dH) / np.linalg.norm(dH) < 1e-6
    assert np.linalg.norm(fdW - dW) / np.linalg.norm(dW) < 1e-6


def test_logit_gradient_by_finite_differences_on_the_logits():
    # d kl_t / d O_S[t,c] with the LM head taken out: use d = V and W = I.
    rng = np.random.default_rng(1)
    V = 6
    O = rng.standard_normal((3, V))
    Zt = rng.standard_normal((3, V)) * 2
    W = np.eye(V)
    tau, g = 1.9, 0.5
    dO = orc.kd_logit_gradient(O, W, Zt, np.ones(3), tau, g)
    h = 1e-6
    for t in range(3):
        for c in range(V):
            Op, Om = O.copy(), O.copy()
            Op[t, c] += h
            Om[t, c] -= h
            fd = g * (orc.kd_token_losses(Op, W, Zt, np.zeros(3, int), np.ones(3), tau)[0].sum()
                      - orc.kd_token_losses(Om, W, Zt, np.zeros(3, int), np.ones(3), tau)[0].sum()) / (2 * h)
            assert abs(fd - dO[t, c]) < 1e-8


def test_torch_autograd_of_an_independent_loss():
    H, W, Zt, mask, y = _problem(2, T=9, d=6, V=12)
    tau, g = 1.4, 0.25
    Ht = torch.tensor(H, requires_grad=True)
    Wt = torch.tensor(W, requires_grad=True)
    ls = torch.log_softmax(Ht @ Wt.T / tau, dim=1)
    lt = torch.log_softmax(torch.tensor(Zt) / tau, dim=1)
    kl = torch.nn.functional.kl_div(ls, lt, reduction="none", log_target=True).sum(1)
    (g * (kl * torch.tensor(mask, dtype=torch.float64)).sum()).backward()
    dH, dW = orc.kd_backward(H, W, Zt, mask, tau, g)
    assert np.allclose(dH, Ht.grad.numpy(), rtol=1e-10, atol=1e-13)
    assert np.allclose(dW, Wt.grad.numpy(), rtol=1e-10, atol=1e-13)


def test_gradient_rows_sum_to_zero_and_masked_rows_vanish():
    H, W, Zt, mask, y = _problem(3, T=20, d=4, V=31)
    dO = orc.kd_logit_gradient(H, W, Zt, mask, 1.3, 0.8)
    assert np.max(np.abs(dO.sum(1))) < 1e-15
    assert np.all(dO[mask == 0] == 0)
    assert np.all(np.abs(dO[mask == 1]).sum(1) > 0)
    dH, dW = orc.kd_backward(H, W, Zt, mask, 1.3, 0.8)
    assert np.all(dH[mask == 0] == 0)
    # columns of dW summed over the vocabulary vanish as well
    assert np.max(np.abs(dW.sum(0))) < 1e-13


def test_sign_and_scale_of_the_logit_gradient():
    # where the student puts more mass than the teacher the gradient is positive,
    # it is linear in grad_scale and carries exactly one factor 1/tau.
    H, W, Zt, mask, y = _problem(4, T=5, d=4, V=8)
    mask[:] = 1
    tau = 2.0
    dO = orc.kd_logit_gradient(H, W, Zt, mask, tau, 1.0)
    ps = np.exp(orc.log_softmax(H @ W.T / tau))
    pt = np.exp(orc.log_softmax(Zt / tau))
    assert np.array_equal(np.sign(dO), np.sign(ps - pt))
    assert np.allclose(dO * tau, ps - pt, rtol=1e-13)
    assert np.allclose(orc.kd_logit_gradient(H, W, Zt, mask, tau, 3.0), 3 * dO, rtol=1e-13)


def test_identical_weight_rows_give_zero_hidden_gradient():
    H, W, Zt, mask, y = _problem(5)
    W[:] = W[0]
    dH, dW = orc.kd_backward(H, W, Zt, mask, 1.0, 1.0)
    assert np.max(np.abs(dH)) < 1e-14
    assert np.max(np.abs(dW)) > 1e-3


def test_dweight_of_packed_batch_is_sum_over_segments():
    H, W, Zt, mask, y = _problem(6, T=12, d=4, V=9)
    cu = [0, 3, 8, 12]
    _, dW = orc.kd_backward(H, W, Zt, mask, 1.2, 0.5)
    acc = np.zeros_like(dW)
    for s in range(3):
        sl = slice(cu[s], cu[s + 1])
        dHs, dWs = orc.kd_backward(H[sl], W, Zt[sl], mask[sl], 1.2, 0.5)
        acc += dWs
    assert np.allclose(acc, dW, rtol=1e-12, atol=1e-15)


def test_row_restricted_gradients_match_the_full_ones():
    H, W, Zt, mask, y = _problem(7, T=14, d=5, V=17)
    dH, dW = orc.kd_backward(H, W, Zt, mask, 0.8, 0.1)
    rows = [0, 1, 5, 13]
    assert np.allclose(orc.kd_dhidden_rows(H, W, Zt, mask, 0.8, 0.1, rows), dH[rows],
                       rtol=1e-13, atol=1e-16)
    vr = [16, 0, 3]
    for grp in (0, 4, 5):
        got = orc.kd_dweight_rows(H, W, Zt, mask, 0.8, 0.1, vr, token_group=grp)
        assert np.allclose(got, dW[vr], rtol=1e-12, atol=1e-16)


# ----------------------------------------------------------------------------------------------
# Eq. 1: composite objective
# ----------------------------------------------------------------------------------------------
def _composite_loss(H, W, Zt, mask, y, tau, g, lam):
    kl, ns, _ = orc.kd_token_losses(H, W, Zt, y, mask, tau)
    return g * orc.composite_token_loss(kl, ns, lam).sum()


@pytest.mark.parametrize("tau,g,lam", [(1.0, 1.0, 0.9), (2.5, 0.37, 0.5), (0.6, 1 / 3, 0.0), (1.7, 2.0, 1.0)])
def test_composite_gradient_by_central_finite_differences(tau, g, lam):
    H, W, Zt, mask, y = _problem(3)
    y[2] = -100                                   # a loss token without a label: KD only
    mask[2] = 1
    dH, dW = orc.composite_backward(H, W, Zt, y, mask, tau, g, lam)
    h = 1e-5
    fdH = np.zeros_like(H)
    for i in range(H.shape[0]):
        for j in range(H.shape[1]):
            Hp, Hm = H.copy(), H.copy()
            Hp[i, j] += h
            Hm[i, j] -= h
            fdH[i, j] = (_composite_loss(Hp, W, Zt, mask, y, tau, g, lam) -
                         _composite_loss(Hm, W, Zt, mask, y, tau, g, lam)) / (2 * h)
    fdW = np.zeros_like(W)
    for i in range(W.shape[0]):
        for j in range(W.shape[1]):
            Wp, Wm = W.copy(), W.copy()
            Wp[i, j] += h
            Wm[i, j] -= h
            fdW[i, j] = (_composite_loss(H, Wp, Zt, mask, y, tau, g, lam) -
                         _composite_loss(H, Wm, Zt, mask, y, tau, g, lam)) / (2 * h)
    assert np.linalg.norm(fdH - dH) / np.linalg.norm(dH) < 1e-6
    assert np.linalg.norm(fdW - dW) / np.linalg.norm(dW) < 1e-6


def test_composite_reduces_to_its_two_terms():
    H, W, Zt, mask, y = _problem(4)
    tau, g = 1.3, 0.7
    # lambda = 1: the distillation gradient alone
    a = orc.composite_logit_gradient(H, W, Zt, y, mask, tau, g, 1.0)
    assert np.allclose(a, orc.kd_logit_gradient(H, W, Zt, mask, tau, g), atol=1e-15)
    # lambda = 0: torch's cross-entropy gradient on the masked tokens
    Ht = torch.tensor(H, dtype=torch.float64, requires_grad=True)
    Wt = torch.tensor(W, dtype=torch.float64, requires_grad=True)
    logits = Ht @ Wt.T
    ce = torch.nn.functional.cross_entropy(logits, torch.tensor(y), reduction="none")
    (g * (ce * torch.tensor(mask, dtype=torch.float64)).sum()).backward()
    dH, dW = orc.composite_backward(H, W, Zt, y, mask, tau, g, 0.0)
    assert np.allclose(dH, Ht.grad.numpy(), atol=1e-12) and np.allclose(dW, Wt.grad.numpy(), atol=1e-12)
    # linear in lambda, rows sum to zero, masked rows are zero
    mid = orc.composite_logit_gradient(H, W, Zt, y, mask, tau, g, 0.25)
    b = orc.composite_logit_gradient(H, W, Zt, y, mask, tau, g, 0.0)
    assert np.allclose(mid, 0.25 * a + 0.75 * b, atol=1e-15)
    assert np.abs(mid.sum(axis=1)).max() < 1e-12 and np.all(mid[mask == 0] == 0)


# ----------------------------------------------------------------------------------------------
# Eq. 2 as printed: top-k teacher support
# ----------------------------------------------------------------------------------------------
def _topk_problem(seed, T=6, d=5, V=11, k=4):
    H, W, Zt, mask, y = _problem(seed, T=T, d=d, V=V)
    idx = np.argsort(-Zt, axis=1)[:, :k]
    vals = np.take_along_axis(Zt, idx, axis=1)
    return H, W, Zt, mask, y, vals, idx


@pytest.mark.parametrize("tau", [1.0, 2.0])
def test_topk_form_equals_dense_form_with_minus_inf_outside_the_support(tau):
    H, W, Zt, mask, y, vals, idx = _topk_problem(5)
    dense = np.full_like(Zt, -np.inf)
    np.put_along_axis(dense, idx, vals, axis=1)
    kl_d, ns_d, _ = orc.kd_token_losses(H, W, dense, y, mask, tau)
    kl_k, ns_k = orc.topk_kd_token_losses(H, W, vals, idx, y, mask, tau)
    assert np.allclose(kl_k, kl_d, atol=1e-13) and np.allclose(ns_k, ns_d, atol=1e-15)
    g_d = orc.kd_logit_gradient(H, W, dense, mask, tau, 0.4)
    g_k = orc.topk_kd_logit_gradient(H, W, vals, idx, mask, tau, 0.4)
    assert np.allclose(g_k, g_d, atol=1e-14)


def test_topk_loss_brute_force_and_lower_bound():
    H, W, Zt, mask, y, vals, idx = _topk_problem(6)
    tau = 1.4
    kl, _ = orc.topk_kd_token_losses(H, W, vals, idx, y, mask, tau)
    O = H @ W.T
    for t in range(H.shape[0]):
        e = [np.exp(v / tau) for v in vals[t]]
        pT = [x / sum(e) for x in e]
        zs = [np.exp(o / tau) for o in O[t]]
        pS = [z / sum(zs) for z in zs]
        ref = sum(pT[j] * (np.log(pT[j]) - np.log(pS[idx[t, j]])) for j in range(len(pT)))
        assert abs(kl[t] - (ref if mask[t] else 0.0)) < 1e-12
        # the student's mass on the support is at most one: KL >= -log(that mass) >= 0
        mass = sum(pS[c] for c in idx[t])
        if mask[t]:
            assert kl[t] >= -np.log(mass) - 1e-12 >= -1e-12


def test_topk_gradient_by_central_finite_differences():
    H, W, Zt, mask, y, vals, idx = _topk_problem(7)
    tau, g = 1.8, 0.6
    dH, dW = orc.topk_kd_backward(H, W, vals, idx, mask, tau, g)
    loss = lambda H_, W_: g * orc.topk_kd_token_losses(H_, W_, vals, idx, y, mask, tau)[0].sum()
    h = 1e-5
    fdH = np.zeros_like(H)
    for i in range(H.shape[0]):
        for j in range(H.shape[1]):
            Hp, Hm = H.copy(), H.copy()
            Hp[i, j] += h
            Hm[i, j] -= h
            fdH[i, j] = (loss(Hp, W) - loss(Hm, W)) / (2 * h)
    fdW = np.zeros_like(W)
    for i in range(W.shape[0]):
        for j in range(W.shape[1]):
            Wp, Wm = W.copy(), W.copy()
            Wp[i, j] += h
            Wm[i, j] -= h
            fdW[i, j] = (loss(H, Wp) - loss(H, Wm)) / (2 * h)
    assert np.linalg.norm(fdH - dH) / np.linalg.norm(dH) < 1e-6
    assert np.linalg.norm(fdW - dW) / np.linalg.norm(dW) < 1e-6

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

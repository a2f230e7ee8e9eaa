"""Shared helpers of the GPU parity tests: run the CUDA library through the C ABI,
run the oracle on the same inputs, compare with the stated tolerances.

Tolerances (bf16 operands, fp32 accumulation and softmax; bf16 gradient tiles):
  per-token losses   |gpu - ref| <= 2e-3 * |ref| + 1e-6
  gradients          ||gpu - ref||_F / ||ref||_F <= 1e-2   (bf16 gradient tiles)
  counts, segment ids, cu boundaries   bit-exact
  keep mask          bit-exact except samples whose Delta lies within 1e-4 of lo or hi
"""

import numpy as np
import torch

from oracle import npd_oracle as orc
from paper_2605_05940_b200 import binding as B

LOSS_RTOL, LOSS_ATOL = 2e-3, 1e-6
GRAD_FROB = 1e-2
BAND = 1e-4


def host(t):
    return t.detach().float().cpu().numpy().astype(np.float64)


def frob(a, r):
    return float(np.linalg.norm(np.asarray(a, np.float64) - r) / max(np.linalg.norm(r), 1e-300))


def assert_losses_close(got, ref, what):
    got, ref = np.asarray(got, np.float64), np.asarray(ref, np.float64)
    same = (got == ref) | (np.isnan(got) & np.isnan(ref))        # equal infinities / NaN scores
    with np.errstate(invalid="ignore"):
        bad = ~same & ~(np.abs(got - ref) <= LOSS_RTOL * np.abs(ref) + LOSS_ATOL)
    assert not bad.any(), f"{what}: {bad.sum()} of {bad.size} outside tolerance; worst " \
                          f"{np.max(np.abs(got - ref) / (np.abs(ref) + 1e-12)):.3e}"


def oracle_inputs(b):
    return (host(b.hidden), host(b.weight), host(b.teacher), b.labels.cpu().numpy(),
            b.loss_mask.cpu().numpy())


def run_step(b, **kw):
    step = B.KDStep(b, **kw)
    step.run()
    torch.cuda.synchronize()
    assert step.status() == B.NPD_OK
    return step


def check_full_parity(b, step, check_grads=True):
    """Element-by-element comparison of every output against the oracle."""
    H, W, Z, y, m = oracle_inputs(b)
    kl, ns, nt = orc.kd_token_losses(H, W, Z, y, m, b.tau)
    assert_losses_close(host(step.kl), kl, "kl")
    assert_losses_close(host(step.nll_student), ns, "nll_student")
    assert_losses_close(host(step.nll_teacher), nt, "nll_teacher")
    assert np.all(host(step.kl)[m == 0] == 0)
    if check_grads:
        dH, dW = orc.kd_backward(H, W, Z, m, b.tau, step.grad_scale)
        assert frob(host(step.d_hidden), dH) <= GRAD_FROB
        assert frob(host(step.d_weight), dW) <= GRAD_FROB
        assert np.all(host(step.d_hidden)[m == 0] == 0)
    return kl, ns, nt


def check_stats_and_select(b, step, kl, ns, nt, lo=0.0, hi=None, q=0.8):
    """Segment statistics on the library's own per-token outputs against the oracle's
    on its own, then Delta-IFD selection."""
    cu = b.cu_seqlens.cpu().numpy()
    y, m = b.labels.cpu().numpy(), b.loss_mask.cpu().numpy()
    ref = orc.segment_stats(cu, m, y, kl, ns, nt)
    got = B.npd_segment_stats(b.cu_seqlens, b.loss_mask, b.labels, step.kl, step.nll_student,
                              step.nll_teacher)
    torch.cuda.synchronize()
    assert np.array_equal(got[3].cpu().numpy(), ref[3])                       # counts
    assert np.array_equal(got[4].cpu().numpy(), orc.segment_ids(cu, b.T))     # seg ids
    for g, r, name in zip(got[:3], ref[:3], ("kl_sum", "nll_s_sum", "nll_t_sum")):
        assert_losses_close(host(g), r, name)
    if b.cond_seg is None:
        return
    cond, unc = b.cond_seg.cpu().numpy(), b.uncond_seg.cpu().numpy()
    if hi is None:
        d0 = orc.delta_ifd_select(cond, unc, ref[1], ref[2], ref[3], 0.0, 1.0)[2]
        hi = orc.nearest_rank_percentile(d0, q)
    o_it, o_is, o_dl, o_keep, o_n = orc.delta_ifd_select(cond, unc, ref[1], ref[2], ref[3], lo, hi)
    it, is_, dl, keep, n_keep = B.npd_select(b.cond_seg, b.uncond_seg, got[1], got[2], got[3], lo, hi)
    torch.cuda.synchronize()
    assert_losses_close(host(it), o_it, "ifd_teacher")
    assert_losses_close(host(is_), o_is, "ifd_student")
    near = (np.abs(o_dl - lo) <= BAND) | (np.abs(o_dl - hi) <= BAND)
    k = keep.cpu().numpy()
    assert np.array_equal(k[~near], o_keep[~near])
    assert int(n_keep.item()) == int(k.sum())
    return float(k.mean())

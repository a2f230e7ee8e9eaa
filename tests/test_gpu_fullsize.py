"""GPU parity at the benchmark's full sizes, in the launch configuration bench.py
times (library defaults), on sampled outputs the oracle computes one by one, plus
properties that hold at any size."""

import numpy as np
import pytest
import torch

from oracle import npd_oracle as orc
from paper_2605_05940_b200 import binding as B
from paper_2605_05940_b200 import synth_inputs as syn

from _parity import (GRAD_FROB, GRAD_FROB_BLOCK, assert_losses_close, edge_vocab_rows, frob, host,
                     oracle_dweight_rows_all_tokens, run_step)

pytestmark = pytest.mark.gpu
DEV = "cuda"


def _sample_rows(b, n, seed):
    rng = np.random.default_rng(seed)
    cu = b.cu_seqlens.cpu().numpy()
    fixed = {0, b.T - 1, int(cu[1]) - 1, int(cu[1]), 127, 128, b.T - 129}
    rows = sorted(fixed | set(rng.integers(0, b.T, size=n).tolist()))
    return np.asarray([r for r in rows if 0 <= r < b.T])


def _check_sampled_rows(b, step, rows):
    W = host(b.weight)
    r = torch.from_numpy(rows).to(DEV)
    H, Z = host(b.hidden[r]), host(b.teacher[r])
    y, m = b.labels[r].cpu().numpy(), b.loss_mask[r].cpu().numpy()
    kl, ns, nt = orc.kd_token_losses(H, W, Z, y, m, b.tau)
    assert_losses_close(host(step.kl[r]), kl, "kl rows")
    assert_losses_close(host(step.nll_student[r]), ns, "nll_student rows")
    assert_losses_close(host(step.nll_teacher[r]), nt, "nll_teacher rows")
    dH = orc.kd_dhidden_rows(H, W, Z, m, b.tau, step.grad_scale, np.arange(len(rows)))
    assert frob(host(step.d_hidden[r]), dH) <= GRAD_FROB
    on = m == 1
    assert on.any() and (~on).any()
    assert np.all(host(step.d_hidden[r])[~on] == 0)
    return W


def _check_dweight_rows(b, step, n=64, seed=11):
    """dW against the oracle on `n` vocabulary rows (tile edges, chunk edges, the last rows,
    random ones); each row needs every loss token's softmax, so the oracle sweeps them all."""
    _, chunks = B.npd_phase_count(step.args)
    vtiles = -(-b.V // 256)
    chunk_cols = -(-vtiles // chunks) * 256
    vr = edge_vocab_rows(b.V, chunk_cols, n, seed)
    got = host(step.d_weight[torch.from_numpy(vr).to(DEV)])
    ref = oracle_dweight_rows_all_tokens(b, step.grad_scale, vr)
    assert frob(got, ref) <= GRAD_FROB
    # and row by row, so that a single wrong row cannot hide among the others
    err = np.linalg.norm(got - ref, axis=1)
    nrm = np.linalg.norm(ref, axis=1)
    assert np.all(err <= GRAD_FROB_BLOCK * np.maximum(nrm, 1e-3 * nrm.mean())), \
        f"dW rows {vr[err > GRAD_FROB_BLOCK * np.maximum(nrm, 1e-3 * nrm.mean())]}"


def _check_properties(b, step):
    m = b.loss_mask.bool()
    assert float(step.kl[~m].abs().max()) == 0.0
    assert bool((step.kl[m] > 0).all()) and bool(torch.isfinite(step.kl).all())
    assert float(step.d_hidden[~m].float().abs().max()) == 0.0
    dW = step.d_weight.float()
    colsum = dW.sum(dim=0)
    # rows of dO_S sum to zero over the vocabulary, hence so do the columns of dW
    assert float(colsum.norm() / dW.norm()) < 5e-2
    # segment statistics: counts bit-exact against the definition, at any size
    got = B.npd_segment_stats(b.cu_seqlens, b.loss_mask, b.labels, step.kl, step.nll_student,
                              step.nll_teacher)
    cu = b.cu_seqlens.cpu().numpy()
    y, mm = b.labels.cpu().numpy(), b.loss_mask.cpu().numpy()
    z = np.zeros(b.T)
    ref_cnt = orc.segment_stats(cu, mm, y, z, z, z)[3]
    assert np.array_equal(got[3].cpu().numpy(), ref_cnt)
    assert np.array_equal(got[4].cpu().numpy(), orc.segment_ids(cu, b.T))
    ref_kl = orc.segment_stats(cu, mm, y, host(step.kl), z, z)[0]      # the reduction itself
    assert_losses_close(host(got[0]), ref_kl, "kl_sum")


def test_config2_full_size_sampled_rows_and_dweight_rows():
    b = syn.config2_1b(device=DEV)
    step = run_step(b)                       # library defaults, as bench.py runs it
    rows = _sample_rows(b, 40, 0)
    W = _check_sampled_rows(b, step, rows)
    _check_properties(b, step)
    _check_dweight_rows(b, step)


def test_config2_full_size_top_k_teacher_sampled_rows():
    # the paper's storage form: k = 10 teacher logits per token, composite objective with lambda = 0.9
    b = syn.config2_1b(device=DEV)
    vals, idx = b.teacher.float().topk(10, dim=1)
    idx = idx.to(torch.int32).contiguous()
    vals = vals.contiguous()
    step = run_step(b, topk_values=vals, topk_indices=idx, kd_lambda=0.9)
    rows = _sample_rows(b, 40, 5)
    r = torch.from_numpy(rows).to(DEV)
    W = host(b.weight)
    H, v, i = host(b.hidden[r]), host(vals[r]), idx[r].cpu().numpy()
    y, m = b.labels[r].cpu().numpy(), b.loss_mask[r].cpu().numpy()
    kl, ns = orc.topk_kd_token_losses(H, W, v, i, y, m, b.tau)
    assert_losses_close(host(step.kl[r]), kl, "kl rows")
    assert_losses_close(host(step.nll_student[r]), ns, "nll_student rows")
    dense = np.full((len(rows), b.V), -np.inf)
    np.put_along_axis(dense, i.astype(np.int64), v, axis=1)
    dO = orc.composite_logit_gradient(H, W, dense, y, m, b.tau, step.grad_scale, 0.9)
    assert frob(host(step.d_hidden[r]), dO @ W) <= GRAD_FROB
    mm = b.loss_mask.bool()
    assert float(step.kl[~mm].abs().max()) == 0.0 and float(step.d_hidden[~mm].float().abs().max()) == 0.0
    assert bool(torch.isfinite(step.d_weight.float()).all())


def test_config2_full_size_fp32_teacher_sampled_rows():
    b = syn.config2_1b(device=DEV)
    g = torch.Generator(device=DEV).manual_seed(23)
    for r0 in range(0, b.T, 1024):       # fp32 logits that bf16 cannot represent, built in row slabs
        if r0 == 0:
            t32 = torch.empty(b.teacher.shape, dtype=torch.float32, device=DEV)
        sl = slice(r0, min(b.T, r0 + 1024))
        t32[sl] = b.teacher[sl].float() + 2e-3 * torch.randn((sl.stop - sl.start, b.V), device=DEV, generator=g)
    b.teacher = t32
    step = run_step(b)
    assert step.args.teacher_dtype == B.NPD_DTYPE_F32
    _check_sampled_rows(b, step, _sample_rows(b, 24, 7))
    _check_properties(b, step)


def test_config3_full_size_sampled_rows_temperature_two():
    b = syn.config3_rows(device=DEV)
    assert (b.T, b.d, b.tau) == (32768, 2048, 2.0)
    step = run_step(b)
    _check_sampled_rows(b, step, _sample_rows(b, 24, 1))
    _check_properties(b, step)
    _check_dweight_rows(b, step, seed=12)


def test_config4_full_size_segments_and_selection_sampled():
    b = syn.config4_short(device=DEV)
    assert b.S > 350
    step = run_step(b)
    _check_sampled_rows(b, step, _sample_rows(b, 24, 2))
    _check_properties(b, step)
    _check_dweight_rows(b, step, seed=13)
    # selection on whole samples the oracle can afford: the first 12 pairs (24 segments)
    cu = b.cu_seqlens.cpu().numpy()
    n_pairs, t_end = 12, int(cu[24])
    W = host(b.weight)
    kl, ns, nt = orc.kd_token_losses(host(b.hidden[:t_end]), W, host(b.teacher[:t_end]),
                                     b.labels[:t_end].cpu().numpy(), b.loss_mask[:t_end].cpu().numpy(), b.tau)
    ref = orc.segment_stats(cu[:25], b.loss_mask[:t_end].cpu().numpy(), b.labels[:t_end].cpu().numpy(), kl, ns, nt)
    got = B.npd_segment_stats(b.cu_seqlens, b.loss_mask, b.labels, step.kl, step.nll_student, step.nll_teacher)
    for g, r in zip(got[:3], ref[:3]):
        assert_losses_close(host(g[:24]), r, "segment sums")
    cond, unc = np.arange(n_pairs) * 2, np.arange(n_pairs) * 2 + 1
    d0 = orc.delta_ifd_select(cond, unc, ref[1], ref[2], ref[3], 0.0, 1.0)[2]
    hi = orc.nearest_rank_percentile(d0, 0.8)
    o = orc.delta_ifd_select(cond, unc, ref[1], ref[2], ref[3], 0.0, hi)
    sel = B.npd_select(b.cond_seg[:n_pairs], b.uncond_seg[:n_pairs], got[1], got[2], got[3], 0.0, hi)
    near = (np.abs(o[2]) <= 1e-4) | (np.abs(o[2] - hi) <= 1e-4)
    assert np.array_equal(sel[3].cpu().numpy()[~near], o[3][~near])
    assert_losses_close(host(sel[2]), o[2], "delta")


def test_config5_full_size_sampled_rows():
    free, _ = torch.cuda.mem_get_info()
    if free < 40 * 2**30:
        pytest.skip("needs about 30 GB of free device memory")
    b = syn.config5_large(device=DEV)
    assert (b.T, b.d) == (65536, 4096)
    step = run_step(b)
    _check_sampled_rows(b, step, _sample_rows(b, 16, 3))
    _check_properties(b, step)
    _check_dweight_rows(b, step, seed=14)

"""Shared helpers of the GPU parity tests: run the CUDA library through the C ABI,
run the oracle on the same inputs, compare with the stated tolerances.

Tolerances (bf16 operands, fp32 accumulation and softmax; bf16 gradient tiles):
  per-token losses   |gpu - ref| <= 2e-3 * |ref| + 1e-6
  gradients          ||gpu - ref||_F / ||ref||_F <= 1e-2   (bf16 gradient tiles), over the whole
                     matrix AND, at 2e-2, over every block of 128 rows of dH and of 256 rows of dW
                     (the row extents of the kernels' tiles), so that one wrong tile, stripe or
                     chunk offset cannot hide in the norm of a large matrix.  Why 2e-2: an element
                     of a gradient is a sum of products whose logit-gradient factor was rounded to
                     bf16 (relative error <= 2^-9, about 1.1e-3 rms) and the result is rounded to
                     bf16 once more; both errors are independent per element, so the relative
                     Frobenius error of any block is about 2e-3 whatever its size.  The block bound
                     keeps the same factor of ~5-10 of slack over that as the matrix bound does.
                     Blocks whose reference norm is below 1e-3 of the mean block norm are skipped
                     (their entries are rounding noise of the larger rows' scale).
  counts, segment ids, cu boundaries   bit-exact
  keep mask          bit-exact except samples whose Delta lies within 1e-4 of lo or hi
"""

import numpy as np
import torch

from oracle import npd_oracle as orc
from paper_2605_05940_b200 import binding as B

LOSS_RTOL, LOSS_ATOL = 2e-3, 1e-6
GRAD_FROB = 1e-2
GRAD_FROB_BLOCK = 2e-2
BAND = 1e-4


def host(t):
    return t.detach().float().cpu().numpy().astype(np.float64)


def frob(a, r):
    return float(np.linalg.norm(np.asarray(a, np.float64) - r) / max(np.linalg.norm(r), 1e-300))


def assert_blocks_close(got, ref, block_rows, what):
    """Relative Frobenius error of every block of `block_rows` consecutive rows."""
    got, ref = np.asarray(got, np.float64), np.asarray(ref, np.float64)
    n = -(-ref.shape[0] // block_rows)
    pad = n * block_rows - ref.shape[0]
    sq = lambda a: np.add.reduceat((a * a).sum(axis=1), np.arange(0, a.shape[0], block_rows))
    err, nrm = np.sqrt(sq(got - ref)), np.sqrt(sq(ref))
    floor = 1e-3 * np.sqrt(np.mean(nrm ** 2))
    live = nrm > floor
    bad = live & (err > GRAD_FROB_BLOCK * nrm)
    # a block that should be (almost) zero must be (almost) zero
    bad |= ~live & (err > GRAD_FROB_BLOCK * max(floor, 1e-300))
    assert not bad.any(), f"{what}: blocks {np.flatnonzero(bad)[:8]} of {n} ({block_rows} rows each, " \
                          f"last one {block_rows - pad}) outside {GRAD_FROB_BLOCK}; worst " \
                          f"{np.max(err[live] / nrm[live]) if live.any() else float('nan'):.3e}"


def assert_grads_close(got_dH, ref_dH, got_dW, ref_dW):
    assert frob(got_dH, ref_dH) <= GRAD_FROB
    assert frob(got_dW, ref_dW) <= GRAD_FROB
    assert_blocks_close(got_dH, ref_dH, 128, "dH")
    assert_blocks_close(got_dW, ref_dW, 256, "dW")


def oracle_dweight_rows_all_tokens(b, grad_scale, vocab_rows, token_group=128, workers=None):
    """Rows `vocab_rows` of dW from the oracle, swept over every token that carries loss.

    dW is a sum over tokens.  The sum is taken group by group (the oracle's own `token_group`
    form of the same sum); here the groups are evaluated by a pool of threads, each calling
    the oracle on its slice (NumPy releases the interpreter lock inside its loops), and the
    partial sums are added in token order.  Tokens without loss are left out of the sweep:
    their logit gradient is exactly zero by definition (pinned in the oracle's own tests)."""
    import os
    from concurrent.futures import ThreadPoolExecutor
    from threadpoolctl import threadpool_limits
    rows = np.asarray(vocab_rows, dtype=np.int64)
    W = host(b.weight)
    idx = torch.nonzero(b.loss_mask != 0).flatten()
    workers = workers or max(1, (os.cpu_count() or 2) - 1)
    ones = np.ones(token_group, dtype=np.uint8)

    def part(sl):
        H, Z = sl
        return orc.kd_dweight_rows(H, W, Z, ones[: len(H)], b.tau, grad_scale, rows)

    def slices():
        for i in range(0, idx.numel(), token_group):
            r = idx[i: i + token_group]
            yield host(b.hidden[r]), b.teacher[r].float().cpu().numpy()

    out = np.zeros((rows.size, b.d))
    with threadpool_limits(limits=1), ThreadPoolExecutor(workers) as ex:
        pending = []
        for sl in slices():
            pending.append(ex.submit(part, sl))
            if len(pending) >= 2 * workers:          # bounded host memory
                out += pending.pop(0).result()
        for f in pending:
            out += f.result()
    return out


def edge_vocab_rows(V, chunk_cols, n, seed):
    """`n` vocabulary rows: the ends of the 256-wide tiles and of the backward's vocabulary
    chunks (each boundary and its neighbours), the last rows, and random ones."""
    rng = np.random.default_rng(seed)
    fixed = {0, 1, 127, 128, 255, 256, 511, 512, V - 129, V - 128, V - 1}
    for c in range(chunk_cols, V, chunk_cols):
        fixed |= {c - 1, c, c + 1}
    fixed = sorted(r for r in fixed if 0 <= r < V)
    if len(fixed) > n // 2:                          # many chunks: keep a spread of their edges
        keep = np.linspace(0, len(fixed) - 1, n // 2).round().astype(int)
        fixed = sorted({fixed[i] for i in keep} | {0, V - 1})
    extra = rng.choice(V, size=n, replace=False)
    rows = list(fixed)
    for r in extra:
        if len(rows) >= n:
            break
        if int(r) not in rows:
            rows.append(int(r))
    return np.asarray(sorted(rows))


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
        assert_grads_close(host(step.d_hidden), dH, host(step.d_weight), dW)
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

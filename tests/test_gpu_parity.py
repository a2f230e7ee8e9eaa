"""GPU parity: the CUDA library, called through the C ABI, against the CPU oracle
on the same seeded inputs, element by element, at sizes the oracle finishes in
seconds that still span several tiles and ragged tails; plus the edge cases."""

import ctypes as C

import numpy as np
import pytest
import torch

from oracle import npd_oracle as orc
from paper_2605_05940_b200 import binding as B
from paper_2605_05940_b200 import synth_inputs as syn

from _parity import (GRAD_FROB, assert_grads_close, assert_losses_close, check_full_parity, check_stats_and_select, frob,
                     host, oracle_inputs, run_step)

pytestmark = pytest.mark.gpu
DEV = "cuda"


# ----------------------------------------------------------------------------------------------
# the tensor-core contraction building block (dH = dO W, dW = dO^T H)
# ----------------------------------------------------------------------------------------------
@pytest.mark.parametrize("a_mn,b_mn", [(False, False), (True, False), (False, True), (True, True)])
@pytest.mark.parametrize("M,N,K", [(128, 256, 64), (296, 520, 200), (8, 8, 8), (1000, 264, 4200)])
def test_gemm_operand_layouts(a_mn, b_mn, M, N, K):
    g = torch.Generator(device=DEV).manual_seed(M * 7 + N * 3 + K)
    A = torch.randn((K, M) if a_mn else (M, K), device=DEV, generator=g).to(torch.bfloat16)
    Bm = torch.randn((K, N) if b_mn else (N, K), device=DEV, generator=g).to(torch.bfloat16)
    out = torch.full((M, N), float("nan"), device=DEV)
    B.npd_gemm_bf16(A, Bm, out, a_mn_major=a_mn, b_mn_major=b_mn)
    torch.cuda.synchronize()
    Ah, Bh = host(A), host(Bm)
    ref = orc.student_logits(Ah.T if a_mn else Ah, Bh.T if b_mn else Bh)   # A B^T in fp64
    assert frob(host(out), ref) < 2e-5      # fp32 accumulation over K


def test_gemm_output_modes_and_split_k():
    g = torch.Generator(device=DEV).manual_seed(5)
    M, N, K = 520, 776, 1800
    A = torch.randn((M, K), device=DEV, generator=g).to(torch.bfloat16)
    Bm = torch.randn((K, N), device=DEV, generator=g).to(torch.bfloat16)
    ref = orc.student_logits(host(A), host(Bm).T)
    base = torch.randn((M, N), device=DEV, generator=g)
    out = base.clone()
    B.npd_gemm_bf16(A, Bm, out, b_mn_major=True, out_mode=B.NPD_GEMM_ADD_F32)
    assert frob(host(out), ref + host(base)) < 2e-5
    out = base.clone()
    B.npd_gemm_bf16(A, Bm, out, b_mn_major=True, out_mode=B.NPD_GEMM_ATOMIC_F32, k_splits=5)
    assert frob(host(out), ref + host(base)) < 2e-5
    outb = torch.empty((M, N), device=DEV, dtype=torch.bfloat16)
    B.npd_gemm_bf16(A, Bm, outb, b_mn_major=True, out_mode=B.NPD_GEMM_STORE_BF16)
    assert frob(host(outb), ref) < 4e-3
    # strided output and operands
    big = torch.zeros((M, N + 24), device=DEV)
    Apad = torch.zeros((M, K + 8), device=DEV, dtype=torch.bfloat16)
    Apad[:, :K] = A
    B.npd_gemm_bf16(Apad[:, :K], Bm, big[:, :N], b_mn_major=True)
    torch.cuda.synchronize()
    assert frob(host(big[:, :N]), ref) < 2e-5 and float(big[:, N:].abs().max()) == 0.0


# ----------------------------------------------------------------------------------------------
# the fused step
# ----------------------------------------------------------------------------------------------
def test_config1_tiny_all_outputs():
    b = syn.config1_tiny(device=DEV, teacher_dtype=torch.bfloat16)
    step = run_step(b, dw_dtype=torch.float32)
    kl, ns, nt = check_full_parity(b, step)
    check_stats_and_select(b, step, kl, ns, nt)
    assert np.array_equal(b.cu_seqlens.cpu().numpy(), [0, 32, 96, 192, 256])


def test_config1_tiny_with_its_fp32_teacher():
    # the tiny configuration as stated: dense fp32 teacher logits (H and W rounded to bf16)
    b = syn.config1_tiny(device=DEV, teacher_dtype=torch.float32)
    assert b.teacher.dtype == torch.float32
    step = run_step(b, dw_dtype=torch.float32)
    assert step.args.teacher_dtype == B.NPD_DTYPE_F32
    kl, ns, nt = check_full_parity(b, step)
    check_stats_and_select(b, step, kl, ns, nt)


@pytest.mark.parametrize("tau,lam,chunk", [(1.0, None, 0), (2.0, None, 512), (1.0, 0.9, 1024), (0.7, 0.5, 256)])
def test_fp32_teacher_ragged_shapes(tau, lam, chunk):
    b = syn.scaled("c2", device=DEV, T=700, d=128, V=3000, min_len=20, max_len=300)
    b.tau = tau
    g = torch.Generator(device=DEV).manual_seed(17)
    b.teacher = b.teacher.float() + 1e-3 * torch.randn(b.teacher.shape, device=DEV, generator=g)  # not bf16-representable
    step = run_step(b, kd_lambda=lam, grad_chunk_cols=chunk, dw_dtype=torch.float32)
    H, W, Z, y, m = oracle_inputs(b)
    kl, ns, nt = orc.kd_token_losses(H, W, Z, y, m, tau)
    assert_losses_close(host(step.kl), kl, "kl")
    assert_losses_close(host(step.nll_student), ns, "nll_student")
    assert_losses_close(host(step.nll_teacher), nt, "nll_teacher")
    dH, dW = (orc.kd_backward(H, W, Z, m, tau, step.grad_scale) if lam is None else
              orc.composite_backward(H, W, Z, y, m, tau, step.grad_scale, lam))
    assert_grads_close(host(step.d_hidden), dH, host(step.d_weight), dW)
    assert np.all(host(step.d_hidden)[m == 0] == 0)


@pytest.mark.parametrize("chunk", [0, 256, 1024])
def test_scaled_config2_multi_tile_ragged(chunk):
    # 6 row blocks with a ragged last one, 12 vocabulary tiles with a ragged tail, 2 k-steps
    b = syn.scaled("c2", device=DEV, T=700, d=128, V=3000, min_len=20, max_len=300)
    step = run_step(b, grad_chunk_cols=chunk)
    kl, ns, nt = check_full_parity(b, step)
    check_stats_and_select(b, step, kl, ns, nt)


def test_scaled_config3_temperature_two_and_row_boundaries():
    b = syn.scaled("c3", device=DEV, rows=2, row_len=512, d=192, V=5000)
    assert b.tau == 2.0
    step = run_step(b, grad_chunk_cols=2048, dw_dtype=torch.float32)
    kl, ns, nt = check_full_parity(b, step)
    check_stats_and_select(b, step, kl, ns, nt)


def test_scaled_config5_wide_hidden():
    b = syn.scaled("c5", device=DEV, T=1100, d=1024, V=2304)
    step = run_step(b, grad_chunk_cols=768)
    check_full_parity(b, step)


def test_config4_short_segments_full_segment_count_and_selection():
    # all ~400 paired segments of the workload, vocabulary and width reduced for the oracle
    b = syn.scaled("c4", device=DEV, T=16384, d=128, V=2048)
    assert b.S > 350
    step = run_step(b, grads=False)
    kl, ns, nt = check_full_parity(b, step, check_grads=False)
    frac = check_stats_and_select(b, step, kl, ns, nt, q=0.8)
    assert 0.2 < frac < 0.9       # the 80th-percentile threshold keeps a real subset


@pytest.mark.parametrize("tau,lam", [(1.0, 0.9), (2.0, 0.5), (1.0, 0.0), (1.5, 1.0)])
def test_composite_objective_gradients(tau, lam):
    # Eq. 1: (1 - lambda) CE + lambda KD; the per-token outputs do not change
    b = syn.scaled("c2", device=DEV, T=700, d=128, V=3000, min_len=20, max_len=300)
    b.tau = tau
    step = run_step(b, kd_lambda=lam, dw_dtype=torch.float32, grad_chunk_cols=1024)
    H, W, Z, y, m = oracle_inputs(b)
    kl, ns, nt = orc.kd_token_losses(H, W, Z, y, m, tau)
    assert_losses_close(host(step.kl), kl, "kl")
    assert_losses_close(host(step.nll_student), ns, "nll_student")
    dH, dW = orc.composite_backward(H, W, Z, y, m, tau, step.grad_scale, lam)
    assert_grads_close(host(step.d_hidden), dH, host(step.d_weight), dW)
    assert np.all(host(step.d_hidden)[m == 0] == 0)
    if lam == 1.0:      # the flag with lambda = 1 is the plain distillation gradient
        plain = run_step(b, dw_dtype=torch.float32, grad_chunk_cols=1024)
        assert torch.equal(plain.d_weight, step.d_weight)


def _topk_of(b, k):
    """The k largest teacher logits per token and their indices, as the annotation phase stores them."""
    vals, idx = b.teacher.float().topk(k, dim=1)
    return vals.contiguous(), idx.to(torch.int32).contiguous()


@pytest.mark.parametrize("tau,k,lam", [(1.0, 10, None), (2.0, 4, None), (1.0, 16, 0.9), (1.3, 1, 0.5)])
def test_topk_teacher_matches_the_oracle(tau, k, lam):
    # Eq. 2 as printed: the teacher is its k largest logits per token
    b = syn.scaled("c2", device=DEV, T=700, d=128, V=3000, min_len=20, max_len=300)
    b.tau = tau
    vals, idx = _topk_of(b, k)
    step = run_step(b, topk_values=vals, topk_indices=idx, kd_lambda=lam, dw_dtype=torch.float32,
                    grad_chunk_cols=1024)
    H, W, Z, y, m = oracle_inputs(b)
    v, i = host(vals), idx.cpu().numpy()
    kl, ns = orc.topk_kd_token_losses(H, W, v, i, y, m, tau)
    assert_losses_close(host(step.kl), kl, "kl")
    assert_losses_close(host(step.nll_student), ns, "nll_student")
    if lam is None:
        dH, dW = orc.topk_kd_backward(H, W, v, i, m, tau, step.grad_scale)
    else:   # composite objective with the top-k distillation term: same Eq. 1, dense form with -inf fill
        dense = np.full_like(Z, -np.inf)
        np.put_along_axis(dense, i.astype(np.int64), v, axis=1)
        dH, dW = orc.composite_backward(H, W, dense, y, m, tau, step.grad_scale, lam)
    assert_grads_close(host(step.d_hidden), dH, host(step.d_weight), dW)
    assert np.all(host(step.d_hidden)[m == 0] == 0) and np.all(host(step.kl)[m == 0] == 0)


def test_topk_teacher_equals_dense_teacher_with_minus_inf_fill():
    # the two entry forms of the same teacher agree on the GPU as well
    b = syn.scaled("c2", device=DEV, T=300, d=64, V=1000, min_len=20, max_len=90)
    vals, idx = _topk_of(b, 10)
    sparse = run_step(b, topk_values=vals, topk_indices=idx, dw_dtype=torch.float32)
    dense = torch.full_like(b.teacher, float("-inf"))
    dense.scatter_(1, idx.long(), vals.to(torch.bfloat16))
    b.teacher = dense
    full = run_step(b, dw_dtype=torch.float32)
    assert_losses_close(host(sparse.kl), host(full.kl), "kl")
    assert frob(host(sparse.d_weight), host(full.d_weight)) < 5e-3
    assert frob(host(sparse.d_hidden), host(full.d_hidden)) < 1e-2


def test_topk_teacher_argument_errors():
    b = _mini()
    vals, idx = _topk_of(b, 4)
    step = B.KDStep(b, topk_values=vals, topk_indices=idx)
    a = B.npd_kd_args.from_buffer_copy(step.args)
    a.topk = 17
    assert B.lib().npd_kd_fwd_bwd(C.byref(a), None) == B.NPD_EUNSUPPORTED
    a = B.npd_kd_args.from_buffer_copy(step.args)
    a.topk_indices = None
    assert B.lib().npd_kd_fwd_bwd(C.byref(a), None) == B.NPD_EINVAL
    a = B.npd_kd_args.from_buffer_copy(step.args)
    a.nll_teacher = step.kl.data_ptr()
    assert B.lib().npd_kd_fwd_bwd(C.byref(a), None) == B.NPD_EINVAL


def test_runs_are_reproducible():
    # per-token outputs and dW bit for bit; dH is summed with fp32 atomic adds in no fixed order,
    # so two runs may round a few elements differently when they are stored as bf16
    b = syn.scaled("c2", device=DEV, T=700, d=128, V=3000, min_len=20, max_len=300)
    s1 = run_step(b, grad_chunk_cols=1024)
    outs1 = [t.clone() for t in (s1.kl, s1.nll_student, s1.nll_teacher, s1.d_weight)]
    dh1 = s1.d_hidden.clone()
    s1.run()
    torch.cuda.synchronize()
    for a, c in zip(outs1, (s1.kl, s1.nll_student, s1.nll_teacher, s1.d_weight)):
        assert torch.equal(a, c)
    assert frob(host(s1.d_hidden), host(dh1)) < 1e-3


# ----------------------------------------------------------------------------------------------
# edge cases
# ----------------------------------------------------------------------------------------------
def _mini(T=40, d=64, V=96, seed=3, **kw):
    return syn.scaled("c2", device=DEV, T=T, d=d, V=V, seed_base=seed, min_len=kw.pop("min_len", 5),
                      max_len=kw.pop("max_len", 17))


def test_single_token_single_segment_and_tiny_vocab():
    b = _mini(T=1, V=8, min_len=1, max_len=1)
    b.loss_mask[:] = 1
    b.labels[:] = 3
    step = run_step(b)
    check_full_parity(b, step)
    got = B.npd_segment_stats(b.cu_seqlens, b.loss_mask, b.labels, step.kl, step.nll_student, step.nll_teacher)
    assert got[3].tolist() == [1] and got[4].tolist() == [0]


def test_all_tokens_masked_gives_zero_loss_and_zero_gradients():
    b = _mini()
    b.loss_mask[:] = 0
    step = run_step(b, dw_dtype=torch.float32)
    assert float(step.kl.abs().max()) == 0 and float(step.nll_student.abs().max()) == 0
    assert float(step.d_hidden.float().abs().max()) == 0 and float(step.d_weight.abs().max()) == 0


@pytest.mark.parametrize("ranges", [
    [(37, 90), (400, 401), (530, 790), (995, 1000)],     # six blocks, the last one runs past T
    [(37, 90), (530, 790), (995, 1000)],                 # five: one CTA of the last pair has no block
    [(0, 1)],                                            # a single loss token
    [(999, 1000)],                                       # ... which is the very last row
])
def test_loss_tokens_in_scattered_stretches(ranges):
    # the kernels only compute the (compacted) loss tokens; everything else must still come out
    # as exact zeros, and nothing may leak between neighbouring rows of a block
    b = syn.scaled("c2", device=DEV, T=1000, d=128, V=1304, seed_base=11, min_len=50, max_len=400)
    b.loss_mask[:] = 0
    for lo, hi in ranges:
        b.loss_mask[lo:hi] = 1
    for dw in (torch.bfloat16, torch.float32):
        step = run_step(b, dw_dtype=dw, grad_chunk_cols=512)
        check_full_parity(b, step)
    step = run_step(b)      # one chunk: dH stored directly
    check_full_parity(b, step)


def test_many_blocks_long_batch_small_vocabulary():
    # 70,000 packed tokens: hundreds of row blocks (an odd number of them), several tokens per
    # planning thread, one ragged vocabulary tile; small d and V keep the oracle quick
    b = syn.scaled("c2", device=DEV, T=70000, d=64, V=520, seed_base=21, min_len=30, max_len=3000)
    step = run_step(b, dw_dtype=torch.float32)
    kl, ns, nt = check_full_parity(b, step)
    check_stats_and_select(b, step, kl, ns, nt)
    # and with every token carrying loss (no mask at all)
    b.loss_mask[:] = 1
    step = run_step(b, dw_dtype=torch.float32)
    check_full_parity(b, step)


@pytest.mark.parametrize("seed", range(14))
def test_random_shapes_masks_and_modes(seed):
    # seeded random problems: odd sizes, masks from all-but-one-zero to all-one, every mode
    rng = np.random.default_rng(100 + seed)
    T = int(rng.integers(1, 700))
    d = int(rng.choice([64, 128, 192]))
    V = int(rng.integers(1, 260)) * 8
    tau = float(rng.choice([1.0, 1.0, 0.7, 2.5]))
    b = syn.scaled("c2", device=DEV, T=T, d=d, V=V, seed_base=300 + seed, min_len=1, max_len=max(2, T // 2))
    b.tau = tau
    density = float(rng.choice([0.02, 0.3, 0.7, 1.0]))
    mask = (rng.random(T) < density).astype(np.uint8)
    mask[int(rng.integers(0, T))] = 1
    b.loss_mask = torch.from_numpy(mask).to(DEV)
    mode = seed % 4
    kw = dict(dw_dtype=torch.float32 if seed % 2 else torch.bfloat16,
              grad_chunk_cols=int(rng.choice([0, 256, 512, 1024])))
    H, W, Z, y, m = oracle_inputs(b)
    if mode in (0, 1):          # dense teacher, Eq. 2 alone or the composite objective
        lam = None if mode == 0 else float(rng.choice([0.0, 0.5, 0.9]))
        step = run_step(b, kd_lambda=lam, **kw)
        kl, ns, nt = orc.kd_token_losses(H, W, Z, y, m, tau)
        assert_losses_close(host(step.nll_teacher), nt, "nll_teacher")
        dH, dW = (orc.kd_backward(H, W, Z, m, tau, step.grad_scale) if lam is None else
                  orc.composite_backward(H, W, Z, y, m, tau, step.grad_scale, lam))
    else:                       # top-k teacher, with or without the cross-entropy term
        k = int(min(V, rng.integers(1, 17)))
        vals, idx = _topk_of(b, k)
        lam = None if mode == 2 else 0.9
        step = run_step(b, topk_values=vals, topk_indices=idx, kd_lambda=lam, **kw)
        v, i = host(vals), idx.cpu().numpy()
        kl, ns = orc.topk_kd_token_losses(H, W, v, i, y, m, tau)
        dense = np.full_like(Z, -np.inf)
        np.put_along_axis(dense, i.astype(np.int64), v, axis=1)
        dH, dW = (orc.topk_kd_backward(H, W, v, i, m, tau, step.grad_scale) if lam is None else
                  orc.composite_backward(H, W, dense, y, m, tau, step.grad_scale, lam))
    assert_losses_close(host(step.kl), kl, "kl")
    assert_losses_close(host(step.nll_student), ns, "nll_student")
    if np.linalg.norm(dH) > 0:
        assert_grads_close(host(step.d_hidden), dH, host(step.d_weight), dW)
    assert np.all(host(step.d_hidden)[m == 0] == 0) and np.all(host(step.kl)[m == 0] == 0)


def test_step_can_be_captured_in_a_cuda_graph_and_replayed():
    # the whole step only enqueues work on the given stream, so a stream capture records it
    b = syn.scaled("c2", device=DEV, T=700, d=128, V=3000, min_len=20, max_len=300)
    step = run_step(b, dw_dtype=torch.float32, grad_chunk_cols=1024)     # eager, also warms everything up
    want = [t.clone() for t in (step.kl, step.nll_student, step.nll_teacher, step.d_weight)]
    dh = step.d_hidden.clone()
    s = torch.cuda.Stream()
    g = torch.cuda.CUDAGraph()
    s.wait_stream(torch.cuda.current_stream())
    with torch.cuda.graph(g, stream=s):
        step.run(torch.cuda.current_stream())
    for t in (step.kl, step.nll_student, step.nll_teacher, step.d_weight, step.d_hidden):
        t.fill_(float("nan"))
    g.replay()
    torch.cuda.synchronize()
    assert step.status() == B.NPD_OK
    for w, t in zip(want, (step.kl, step.nll_student, step.nll_teacher, step.d_weight)):
        assert torch.equal(w, t)
    assert frob(host(step.d_hidden), host(dh)) < 1e-3


def test_optional_inputs_may_be_null():
    b = _mini()
    H, W, Z, y, m = oracle_inputs(b)
    T = b.T
    kl = torch.empty(T, device=DEV)
    a = B.make_kd_args(b.hidden, b.weight, b.teacher, kl=kl, temperature=1.0, grad_scale=1.0)
    ws = torch.empty(B.npd_workspace_bytes(a) + 1024, dtype=torch.uint8, device=DEV)
    off = (-ws.data_ptr()) % 1024
    a = B.make_kd_args(b.hidden, b.weight, b.teacher, kl=kl, temperature=1.0, grad_scale=1.0,
                       workspace=ws[off:])
    B.npd_kd_fwd_bwd(a)
    torch.cuda.synchronize()
    ref, _, _ = orc.kd_token_losses(H, W, Z, np.full(T, -1), np.ones(T), 1.0)
    assert_losses_close(host(kl), ref, "kl without mask/labels/cu_seqlens")


def test_padded_strides_and_teacher_columns_beyond_vocab():
    b = _mini(T=150, d=64, V=1001 - 1)          # V = 1000
    V, T, d = b.V, b.T, b.d
    zpad = torch.full((T, V + 24), 77.0, device=DEV, dtype=torch.bfloat16)   # junk beyond V
    zpad[:, :V] = b.teacher
    hpad = torch.zeros((T, d + 8), device=DEV, dtype=torch.bfloat16)
    hpad[:, :d] = b.hidden
    b2 = syn.KDBatch(b.name, T, d, V, b.S, hpad[:, :d], b.weight, zpad[:, :V], b.cu_seqlens,
                     b.loss_mask, b.labels, b.tau)
    step = B.KDStep(b2)
    assert step.args.ldh == d + 8 and step.args.ldt == V + 24 and step.d_hidden.stride(0) == d + 8
    step.run()
    torch.cuda.synchronize()
    check_full_parity(b, step)


def test_minus_inf_teacher_entries_dense_top_k():
    # a top-k teacher densified with -inf outside its support (Eq. 2 on the top-k support)
    b = _mini(T=70, V=600)
    z = b.teacher.float()
    kth = z.topk(10, dim=1).values[:, -1:]
    b.teacher = torch.where(z >= kth, z, torch.full_like(z, float("-inf"))).to(torch.bfloat16)
    step = run_step(b, dw_dtype=torch.float32)
    assert torch.isfinite(step.kl).all() and torch.isfinite(step.d_weight).all()
    check_full_parity(b, step)


def test_forward_only_and_f32_accumulating_dweight():
    b = _mini(T=200, V=520)
    f = run_step(b, grads=False)
    g = run_step(b, dw_dtype=torch.float32)
    assert torch.equal(f.kl, g.kl) and f.d_hidden is None
    first = g.d_weight.clone()
    g.args.flags = B.NPD_KD_ACCUMULATE_DW
    g.run()
    torch.cuda.synchronize()
    assert frob(host(g.d_weight), 2 * host(first)) < 1e-6


def test_malformed_cu_seqlens_is_reported_not_faulted():
    b = _mini(T=60)
    good = b.cu_seqlens.clone()
    for bad in ([0, 70, 60], [1] + good.tolist()[1:], good.tolist()[:-1] + [59],
                [0, 30, 30, 60], [0, 40, 20, 60], [0, -5, 60]):
        b.cu_seqlens = torch.tensor(bad, dtype=torch.int32, device=DEV)
        b.S = len(bad) - 1
        step = B.KDStep(b, grads=False)
        step.run()
        assert step.status() == B.NPD_ESEQ, bad
        st = torch.zeros(1, dtype=torch.int32, device=DEV)
        B.npd_segment_stats(b.cu_seqlens, b.loss_mask, b.labels, step.kl, step.nll_student,
                            step.nll_teacher, status=st)
        assert int(st.item()) == B.NPD_ESEQ
    b.cu_seqlens, b.S = good, good.numel() - 1
    step = B.KDStep(b, grads=False)
    step.run()
    assert step.status() == B.NPD_OK


def test_workspace_and_option_errors():
    b = _mini()
    step = B.KDStep(b)
    a = B.npd_kd_args.from_buffer_copy(step.args)
    a.workspace_bytes = step.args.workspace_bytes - 1
    assert B.lib().npd_kd_fwd_bwd(C.byref(a), None) == B.NPD_EWORKSPACE
    a = B.npd_kd_args.from_buffer_copy(step.args)
    a.workspace = step.args.workspace + 16
    assert B.lib().npd_kd_fwd_bwd(C.byref(a), None) == B.NPD_EWORKSPACE
    a = B.npd_kd_args.from_buffer_copy(step.args)
    a.teacher_dtype = 7
    assert B.lib().npd_kd_fwd_bwd(C.byref(a), None) == B.NPD_EINVAL


def test_select_matches_float32_oracle_bit_for_bit():
    rng = np.random.default_rng(0)
    S = 4001
    N = 2000
    count = rng.integers(0, 40, size=S).astype(np.int32)
    s_sum = (rng.random(S) * 30).astype(np.float32)
    t_sum = (rng.random(S) * 30).astype(np.float32)
    s_sum[5] = 0.0
    cond = rng.integers(0, S, size=N).astype(np.int32)
    unc = rng.integers(0, S, size=N).astype(np.int32)
    to = lambda x: torch.from_numpy(x).to(DEV)
    for flags in (0, B.NPD_SELECT_TEACHER_IFD_LE_1):
        it, is_, dl, keep, n = B.npd_select(to(cond), to(unc), to(s_sum), to(t_sum), to(count), 0.0, 0.8, flags)
        o = orc.delta_ifd_select(cond, unc, s_sum, t_sum, count, 0.0, 0.8,
                                 require_teacher_ifd_le_1=bool(flags), dtype=np.float32)
        assert np.array_equal(it.cpu().numpy(), o[0], equal_nan=True)
        assert np.array_equal(is_.cpu().numpy(), o[1], equal_nan=True)
        assert np.array_equal(dl.cpu().numpy(), o[2], equal_nan=True)
        assert np.array_equal(keep.cpu().numpy(), o[3]) and int(n.item()) == o[4]


def test_filter_ablation_scopes_match_float32_oracle_bit_for_bit():
    rng = np.random.default_rng(1)
    S, N = 1001, 700
    count = rng.integers(0, 30, size=S).astype(np.int32)
    s_sum = (rng.random(S) * 20).astype(np.float32)
    t_sum = (rng.random(S) * 20).astype(np.float32)
    cond = rng.integers(0, S, size=N).astype(np.int32)
    unc = rng.integers(0, S, size=N).astype(np.int32)
    # make some scores land exactly on the ends 0 and 1
    s_sum[cond[:40]] = 0.0
    t_sum[cond[40:80]] = t_sum[unc[40:80]] * count[cond[40:80]] / np.maximum(count[unc[40:80]], 1)
    to = lambda x: torch.from_numpy(x).to(DEV)
    inf = float("inf")
    cases = [(B.NPD_SELECT_SCORE_IFD_TEACHER, 0.0, 1.0, dict(score="ifd_teacher")),
             (B.NPD_SELECT_SCORE_IFD_STUDENT, 0.0, 1.0, dict(score="ifd_student")),
             (B.NPD_SELECT_LO_EXCLUSIVE, 0.0, inf, dict(lo_inclusive=False)),
             (B.NPD_SELECT_HI_EXCLUSIVE, -inf, 1.0, dict(hi_inclusive=False)),
             (B.NPD_SELECT_SCORE_IFD_STUDENT | B.NPD_SELECT_LO_EXCLUSIVE | B.NPD_SELECT_HI_EXCLUSIVE, 0.0, 1.0,
              dict(score="ifd_student", lo_inclusive=False, hi_inclusive=False))]
    for flags, lo, hi, kw in cases:
        keep, n = B.npd_select(to(cond), to(unc), to(s_sum), to(t_sum), to(count), lo, hi, flags)[3:]
        o = orc.delta_ifd_select(cond, unc, s_sum, t_sum, count, lo, hi, dtype=np.float32, **kw)
        assert np.array_equal(keep.cpu().numpy(), o[3]) and int(n.item()) == o[4], kw
    assert B.lib().npd_select(N, 1, 1, 1, 1, 1, S, C.c_float(0), C.c_float(1), 6, 0, 0, 0, 1, 1, None) == B.NPD_EINVAL


@pytest.mark.parametrize("tau", [1.0, 2.0])
def test_policy_lag_monitor_reverse_kl(tau):
    b = syn.scaled("c2", device=DEV, T=700, d=128, V=3000, min_len=20, max_len=300)
    b.tau = tau
    step = run_step(b, grads=False, flags=B.NPD_KD_REVERSE_KL)
    H, W, Z, y, m = oracle_inputs(b)
    assert_losses_close(host(step.kl), orc.reverse_kl_token(H, W, Z, m, tau), "reverse kl")
    _, ns, nt = orc.kd_token_losses(H, W, Z, y, m, tau)
    assert_losses_close(host(step.nll_student), ns, "nll_student")
    assert_losses_close(host(step.nll_teacher), nt, "nll_teacher")
    a = B.npd_kd_args.from_buffer_copy(run_step(b).args)
    a.flags = B.NPD_KD_REVERSE_KL            # with gradients requested: refused
    assert B.lib().npd_kd_fwd_bwd(C.byref(a), None) == B.NPD_EINVAL


def test_host_buffer_entry_point_matches_device_entry_point():
    b = syn.scaled("c2", device=DEV, T=300, d=64, V=520, min_len=20, max_len=90)
    ref = run_step(b)
    pin = lambda t: t.cpu().pin_memory()
    hh, hz, hcu, hm, hy = map(pin, (b.hidden, b.teacher, b.cu_seqlens, b.loss_mask, b.labels))
    hkl, hns, hnt = (torch.empty(b.T).pin_memory() for _ in range(3))
    # fresh device staging buffers (zeroed), resident weight
    stage = syn.KDBatch(b.name, b.T, b.d, b.V, b.S, torch.zeros_like(b.hidden), b.weight,
                        torch.zeros_like(b.teacher), torch.zeros_like(b.cu_seqlens),
                        torch.zeros_like(b.loss_mask), torch.zeros_like(b.labels), b.tau)
    step = B.KDStep(stage, grad_scale=ref.grad_scale)
    hargs = B.make_kd_args(hh, b.weight, hz, cu_seqlens=hcu, loss_mask=hm, labels=hy, kl=hkl,
                           nll_student=hns, nll_teacher=hnt, temperature=b.tau)
    B.npd_kd_fwd_bwd_host(hargs, step.args)
    torch.cuda.synchronize()
    assert step.status() == B.NPD_OK
    assert torch.equal(hkl, ref.kl.cpu()) and torch.equal(hns, ref.nll_student.cpu())
    assert torch.equal(hnt, ref.nll_teacher.cpu())
    assert frob(host(step.d_hidden), host(ref.d_hidden)) < 1e-3 and torch.equal(step.d_weight, ref.d_weight)
    h2d, d2h = B.npd_last_copy_bytes()
    n_loss = int(b.loss_mask.sum().item())
    assert h2d == n_loss * (b.d + b.V) * 2 + 4 * (b.S + 1) + b.T + 4 * b.T and d2h == 12 * b.T
    # the same with the copies on a stream of their own, twice in a row on the same staging buffers
    copy_stream, compute = torch.cuda.Stream(), torch.cuda.Stream()
    for _ in range(2):
        hkl.zero_()
        step.kl.zero_()
        B.npd_kd_fwd_bwd_host_streams(hargs, step.args, copy_stream, compute)
    torch.cuda.synchronize()
    assert torch.equal(hkl, ref.kl.cpu()) and torch.equal(step.d_weight, ref.d_weight)


def test_perplexity_scores_match_the_oracle():
    b = syn.config4_short(device=DEV, T=2048, d=128, V=3000)
    step = run_step(b, grads=False)
    kl, ns, nt = check_full_parity(b, step, check_grads=False)
    cu, y, m = b.cu_seqlens.cpu().numpy(), b.labels.cpu().numpy(), b.loss_mask.cpu().numpy()
    ref = orc.segment_stats(cu, m, y, kl, ns, nt)
    got = B.npd_segment_stats(b.cu_seqlens, b.loss_mask, b.labels, step.kl, step.nll_student, step.nll_teacher)
    seg = torch.arange(b.S, dtype=torch.int32, device=DEV)
    ps, pt = B.npd_perplexity(seg, got[1], got[2], got[3])
    torch.cuda.synchronize()
    assert_losses_close(host(ps), orc.perplexity_scores(np.arange(b.S), ref[1], ref[3]), "ppl_student")
    assert_losses_close(host(pt), orc.perplexity_scores(np.arange(b.S), ref[2], ref[3]), "ppl_teacher")
    # the same two operations in float32 on the same sums: bit for bit up to the exponential's last place
    o32 = orc.perplexity_scores(np.arange(b.S), host(got[1]), got[3].cpu().numpy(), dtype=np.float32)
    assert np.allclose(host(ps), o32, rtol=3e-7, atol=0, equal_nan=True)
    # empty sample and a segment index out of range: NaN; one output alone is allowed
    cnt = got[3].clone()
    cnt[1] = 0
    bad = torch.tensor([1, -1, b.S, 0], dtype=torch.int32, device=DEV)
    ps2, none = B.npd_perplexity(bad, got[1], None, cnt)
    assert none is None
    p = host(ps2)
    assert np.isnan(p[:3]).all() and np.isfinite(p[3])
    with pytest.raises(B.NpdError):
        B.npd_perplexity(bad, None, None, cnt)


def test_bounded_wait_runs_out_and_reports_timeout():
    # a wait on a barrier nothing arrives on, with a limit of 2e5 cycles (about 0.1 ms): the status
    # word must read NPD_ETIMEOUT, every thread must have given up, and the device must be fine
    import time
    torch.cuda.synchronize()
    t0 = time.perf_counter()
    out = B.npd_selftest_wait_timeout(200_000, device=DEV)
    torch.cuda.synchronize()
    dt = time.perf_counter() - t0
    status, all_gave_up, cycles = out.cpu().tolist()
    assert status == B.NPD_ETIMEOUT and all_gave_up == 1
    assert 200_000 <= cycles < 1_000_000
    assert dt < 0.5
    with pytest.raises(B.NpdError):
        B.npd_selftest_wait_timeout(10**9, device=DEV)          # refused on the host: too long
    # the context is still usable
    b = syn.config1_tiny(device=DEV, teacher_dtype=torch.bfloat16)
    check_full_parity(b, run_step(b))


def test_serialized_launches_give_the_same_results():
    b = syn.config2_1b(device=DEV, T=1024, d=256, V=5000, min_len=32, max_len=256)
    s1 = run_step(b, grad_chunk_cols=1024)
    s2 = run_step(b, grad_chunk_cols=1024, flags=B.NPD_KD_SERIALIZE_LAUNCHES)
    assert torch.equal(s1.kl, s2.kl) and torch.equal(s1.d_weight, s2.d_weight)
    assert frob(host(s1.d_hidden), host(s2.d_hidden)) < 1e-3


def test_debug_checks_flag_inputs_the_step_may_not_be_given():
    def fresh():
        return syn.config2_1b(device=DEV, T=600, d=128, V=2000, min_len=20, max_len=200)

    def status_of(b, **kw):
        step = B.KDStep(b, flags=B.NPD_KD_DEBUG_CHECKS, **kw)
        step.run()
        torch.cuda.synchronize()
        H, _, Z, y, m = oracle_inputs(b)
        idx = kw["topk_indices"].cpu().numpy() if "topk_indices" in kw else None
        want_ok = orc.validate_step_inputs(H, Z, y, m, b.V, idx)
        assert (step.status() == B.NPD_OK) == want_ok
        return step

    b = fresh()
    clean = status_of(b)
    assert clean.status() == B.NPD_OK
    plain = run_step(b)                               # same results with and without the checks
    assert torch.equal(clean.kl, plain.kl) and torch.equal(clean.d_weight, plain.d_weight)
    on = torch.nonzero(b.loss_mask).flatten()
    off = torch.nonzero(b.loss_mask == 0).flatten()

    b = fresh(); b.labels[int(on[3])] = b.V           # a label that names no class
    assert status_of(b).status() == B.NPD_EDATA
    b = fresh(); b.teacher[int(on[5]), :] = float("-inf")
    assert status_of(b).status() == B.NPD_EDATA       # a loss token without any support
    b = fresh(); b.teacher[int(on[5]), 1:] = float("-inf")
    assert status_of(b).status() == B.NPD_OK          # one class left
    b = fresh(); b.teacher[int(off[0]), :] = float("nan"); b.hidden[int(off[0]), :] = float("inf")
    assert status_of(b).status() == B.NPD_OK          # rows of tokens without loss are not read
    b = fresh(); b.teacher[int(on[-1]), b.V - 1] = float("nan")
    assert status_of(b).status() == B.NPD_EDATA
    b = fresh(); b.hidden[int(on[0]), 7] = float("inf")
    assert status_of(b).status() == B.NPD_EDATA
    # top-k teacher: stored indices must lie inside the vocabulary
    b = fresh()
    vals, idx = b.teacher.float().topk(4, dim=1)
    idx = idx.to(torch.int32).contiguous()
    assert status_of(b, topk_values=vals.contiguous(), topk_indices=idx).status() == B.NPD_OK
    idx2 = idx.clone(); idx2[int(on[2]), 1] = b.V
    assert status_of(b, topk_values=vals.contiguous(), topk_indices=idx2).status() == B.NPD_EDATA

"""The forward entry point for callers that cannot allocate device memory
(`npd_kd_forward_noalloc`): its scratch is a fixed array inside the library, so the
caller passes inputs and outputs only.  Checked against the ordinary entry point, which
runs the same kernels on a caller-provided workspace, and against the CPU oracle, on two calls
in a row (the array is shared between calls and keeps the previous call's contents).  That the
call takes no device memory is read from the driver (free bytes before and after), which also
sees an allocation made inside the library.  Collected last on purpose:
a run that stops at the first failure has then already run every other test."""

import ctypes as C

import pytest
import torch

from paper_2605_05940_b200 import binding as B
from paper_2605_05940_b200 import synth_inputs as syn

from oracle import npd_oracle as orc

from _parity import LOSS_ATOL, LOSS_RTOL, assert_losses_close, host, oracle_inputs

pytestmark = pytest.mark.gpu
DEV = "cuda"


def _close(a, b):
    return bool(torch.all((a - b).abs() <= LOSS_RTOL * b.abs() + LOSS_ATOL))


def _forward_args(b, kl, ns, nt):
    return B.make_kd_args(b.hidden, b.weight, b.teacher, cu_seqlens=b.cu_seqlens, loss_mask=b.loss_mask,
                          labels=b.labels, temperature=b.tau, kl=kl, nll_student=ns, nll_teacher=nt)


def test_noalloc_forward_matches_workspace_forward_twice_in_a_row():
    first = syn.scaled("c2", device=DEV, T=700, d=128, V=3000, min_len=20, max_len=300)
    second = syn.scaled("c3", device=DEV, rows=2, row_len=512, d=192, V=5000)      # tau = 2, other shape
    for b in (first, second):
        ref = B.KDStep(b, grads=False)
        ref.run()
        torch.cuda.synchronize()
        assert ref.status() == B.NPD_OK
        kl, ns, nt = (torch.full((b.T,), float("nan"), device=DEV) for _ in range(3))
        args = _forward_args(b, kl, ns, nt)
        # one call first, so that the library's module (and with it the static array) is resident
        # and the array's address is looked up; from then on a call may take nothing
        assert B.npd_kd_forward_noalloc(args, want_status=True) == B.NPD_OK
        kl.fill_(float("nan"))
        torch.cuda.synchronize()
        before_torch, before_free = torch.cuda.memory_allocated(), torch.cuda.mem_get_info()[0]
        status = B.npd_kd_forward_noalloc(args, want_status=True)
        assert status == B.NPD_OK
        assert torch.cuda.memory_allocated() == before_torch
        assert torch.cuda.mem_get_info()[0] == before_free        # the driver saw no allocation either
        for got, want in ((kl, ref.kl), (ns, ref.nll_student), (nt, ref.nll_teacher)):
            assert _close(got, want)
        # and against the oracle directly
        H, W, Z, y, m = oracle_inputs(b)
        o_kl, o_ns, o_nt = orc.kd_token_losses(H, W, Z, y, m, b.tau)
        assert_losses_close(host(kl), o_kl, "kl")
        assert_losses_close(host(ns), o_ns, "nll_student")
        assert_losses_close(host(nt), o_nt, "nll_teacher")
        # same problem again, enqueue-only form: the stale contents of the array must not matter
        kl2, ns2, nt2 = (torch.full((b.T,), float("nan"), device=DEV) for _ in range(3))
        B.npd_kd_forward_noalloc(_forward_args(b, kl2, ns2, nt2))
        torch.cuda.synchronize()
        assert torch.equal(kl2, kl) and torch.equal(ns2, ns) and torch.equal(nt2, nt)


def test_noalloc_refuses_gradients_and_oversized_problems():
    b = syn.scaled("c2", device=DEV, T=300, d=64, V=520, min_len=20, max_len=90)
    kl = torch.empty(b.T, device=DEV)
    a = _forward_args(b, kl, None, None)
    a.d_hidden, a.d_weight = b.hidden.data_ptr(), b.weight.data_ptr()
    assert B.lib().npd_kd_forward_noalloc(C.byref(a), None, None) == B.NPD_EINVAL
    # a token count whose partials cannot fit the fixed array (pointers are never touched)
    a = _forward_args(b, kl, None, None)
    a.T = 4_000_000
    need = B.npd_workspace_bytes(a)
    assert need > B.NPD_STATIC_SCRATCH_BYTES
    assert B.lib().npd_kd_forward_noalloc(C.byref(a), None, None) == B.NPD_EWORKSPACE

"""ctypes binding of the C-ABI library (include/npd.h).

Argument marshalling only: every step of the computation runs in the library's
CUDA kernels.  PyTorch supplies device memory and streams.  There is no CPU or
PyTorch fallback: if the library is not built the first call raises.
"""

from __future__ import annotations

import ctypes as C
import os
from typing import Optional

import torch

_HERE = os.path.dirname(os.path.abspath(__file__))
LIB_PATH = os.path.join(_HERE, "libnpd.so")

NPD_OK = 0
NPD_EINVAL, NPD_ESHAPE, NPD_EALIGN, NPD_ESEQ, NPD_EARCH = -1, -2, -3, -4, -5
NPD_EWORKSPACE, NPD_ECUDA, NPD_ETIMEOUT, NPD_EUNSUPPORTED, NPD_EDATA = -6, -7, -8, -9, -10
NPD_DTYPE_BF16, NPD_DTYPE_F32 = 0, 1
NPD_KD_ACCUMULATE_DW = 1
NPD_KD_COMPOSITE_LOSS = 2
NPD_KD_REVERSE_KL = 4
NPD_KD_SERIALIZE_LAUNCHES = 8
NPD_KD_DEBUG_CHECKS = 16
NPD_SELECT_TEACHER_IFD_LE_1 = 1
NPD_SELECT_SCORE_IFD_TEACHER, NPD_SELECT_SCORE_IFD_STUDENT = 2, 4
NPD_SELECT_LO_EXCLUSIVE, NPD_SELECT_HI_EXCLUSIVE = 8, 16
NPD_GEMM_STORE_F32, NPD_GEMM_ADD_F32, NPD_GEMM_STORE_BF16, NPD_GEMM_ATOMIC_F32 = range(4)

EXPORTS = ("npd_workspace_bytes", "npd_phase_count", "npd_kd_fwd_bwd", "npd_kd_fwd_bwd_host", "npd_segment_stats",
           "npd_select", "npd_last_status", "npd_strerror", "npd_last_launch_count", "npd_gemm_bf16",
           "npd_kd_forward_noalloc", "npd_pack_sequences", "npd_last_copy_bytes",
           "npd_kd_fwd_bwd_host_streams", "npd_perplexity", "npd_selftest_wait_timeout",
           "npd_debug_chunk_schedule")
NPD_STATIC_SCRATCH_BYTES = 48 * 1024 * 1024


class NpdError(RuntimeError):
    def __init__(self, code: int, where: str):
        self.code = code
        super().__init__(f"{where}: {strerror(code)} ({code})")


class npd_kd_args(C.Structure):
    _fields_ = [
        ("size", C.c_size_t),
        ("T", C.c_int32), ("d", C.c_int32), ("V", C.c_int32), ("S", C.c_int32),
        ("hidden", C.c_void_p), ("weight", C.c_void_p), ("teacher", C.c_void_p),
        ("ldh", C.c_int64), ("ldw", C.c_int64), ("ldt", C.c_int64),
        ("teacher_dtype", C.c_int32), ("reserved0", C.c_int32),
        ("cu_seqlens", C.c_void_p), ("loss_mask", C.c_void_p), ("labels", C.c_void_p),
        ("temperature", C.c_float), ("grad_scale", C.c_float),
        ("kl", C.c_void_p), ("nll_student", C.c_void_p), ("nll_teacher", C.c_void_p),
        ("d_hidden", C.c_void_p), ("d_weight", C.c_void_p),
        ("d_weight_dtype", C.c_int32), ("flags", C.c_int32),
        ("grad_chunk_cols", C.c_int32), ("kd_lambda", C.c_float),
        ("workspace", C.c_void_p), ("workspace_bytes", C.c_size_t),
        ("phase_events", C.POINTER(C.c_void_p)), ("n_phase_events", C.c_int32), ("reserved2", C.c_int32),
        ("topk_values", C.c_void_p), ("topk_indices", C.c_void_p), ("topk", C.c_int32), ("reserved3", C.c_int32),
    ]


_lib = None


def lib() -> C.CDLL:
    """The loaded library.  Raises if it has not been built (no fallback)."""
    global _lib
    if _lib is None:
        from . import build as _build
        if _build.is_stale():          # missing, or built from other sources than the ones present
            _build.build()             # raises if it cannot: never run kernels of other sources
        if not os.path.exists(LIB_PATH):
            raise RuntimeError(
                f"{LIB_PATH} is missing: build it with `python -m paper_2605_05940_b200.build` "
                "(there is no CPU or PyTorch fallback)")
        l = C.CDLL(LIB_PATH)
        l.npd_strerror.restype = C.c_char_p
        l.npd_strerror.argtypes = [C.c_int]
        l.npd_workspace_bytes.argtypes = [C.POINTER(npd_kd_args), C.POINTER(C.c_size_t)]
        l.npd_kd_fwd_bwd.argtypes = [C.POINTER(npd_kd_args), C.c_void_p]
        l.npd_phase_count.argtypes = [C.POINTER(npd_kd_args), C.POINTER(C.c_int32), C.POINTER(C.c_int32)]
        l.npd_kd_fwd_bwd_host.argtypes = [C.POINTER(npd_kd_args), C.POINTER(npd_kd_args), C.c_void_p]
        l.npd_kd_fwd_bwd_host_streams.argtypes = [C.POINTER(npd_kd_args), C.POINTER(npd_kd_args), C.c_void_p,
                                                  C.c_void_p]
        l.npd_segment_stats.argtypes = [C.c_int32, C.c_int32] + [C.c_void_p] * 13
        l.npd_select.argtypes = ([C.c_int32] + [C.c_void_p] * 5 + [C.c_int32, C.c_float, C.c_float, C.c_int32]
                                 + [C.c_void_p] * 6)
        l.npd_last_status.argtypes = [C.c_void_p, C.c_void_p, C.POINTER(C.c_int32)]
        l.npd_last_launch_count.argtypes = []
        l.npd_last_copy_bytes.argtypes = [C.POINTER(C.c_int64), C.POINTER(C.c_int64)]
        l.npd_kd_forward_noalloc.argtypes = [C.POINTER(npd_kd_args), C.c_void_p, C.POINTER(C.c_int32)]
        l.npd_pack_sequences.argtypes = [C.c_int32, C.c_void_p, C.c_void_p, C.c_int32] + [C.c_void_p] * 6
        l.npd_perplexity.argtypes = [C.c_int32] + [C.c_void_p] * 4 + [C.c_int32] + [C.c_void_p] * 3
        l.npd_selftest_wait_timeout.argtypes = [C.c_int64, C.c_void_p, C.c_void_p]
        l.npd_debug_chunk_schedule.argtypes = [C.c_int32] * 6 + [C.c_void_p, C.POINTER(C.c_int32)]
        l.npd_gemm_bf16.argtypes = [C.c_int32, C.c_int32, C.c_int32, C.c_void_p, C.c_int64, C.c_int32,
                                    C.c_void_p, C.c_int64, C.c_int32, C.c_void_p, C.c_int64,
                                    C.c_int32, C.c_int32, C.c_void_p]
        _lib = l
    return _lib


def strerror(code: int) -> str:
    return lib().npd_strerror(int(code)).decode()


def _ptr(t: Optional[torch.Tensor]) -> Optional[int]:
    return None if t is None else t.data_ptr()


def _stream(stream) -> int:
    if stream is None:
        stream = torch.cuda.current_stream()
    return stream.cuda_stream if hasattr(stream, "cuda_stream") else int(stream)


def _check(rc: int, where: str):
    if rc != NPD_OK:
        raise NpdError(rc, where)


def make_kd_args(hidden, weight, teacher, *, cu_seqlens=None, loss_mask=None, labels=None,
                 temperature=1.0, grad_scale=1.0, kl=None, nll_student=None, nll_teacher=None,
                 d_hidden=None, d_weight=None, flags=0, grad_chunk_cols=0, kd_lambda=None,
                 topk_values=None, topk_indices=None, workspace=None) -> npd_kd_args:
    """Fill an npd_kd_args from tensors (device tensors, or host tensors for the
    `host` argument of npd_kd_fwd_bwd_host)."""
    a = npd_kd_args()
    a.size = C.sizeof(npd_kd_args)
    a.T, a.d = hidden.shape
    a.V = weight.shape[0]
    a.S = 0 if cu_seqlens is None else cu_seqlens.numel() - 1
    a.hidden, a.weight, a.teacher = _ptr(hidden), _ptr(weight), _ptr(teacher)
    a.ldh, a.ldw = hidden.stride(0), weight.stride(0)
    if teacher is not None:
        a.ldt = teacher.stride(0)
        a.teacher_dtype = NPD_DTYPE_F32 if teacher.dtype == torch.float32 else NPD_DTYPE_BF16
    else:                           # top-k teacher: f32 [T,k] logits and int32 [T,k] indices
        a.ldt = (a.V + 7) // 8 * 8
        a.teacher_dtype = NPD_DTYPE_BF16
    if topk_values is not None:
        a.topk_values, a.topk_indices, a.topk = _ptr(topk_values), _ptr(topk_indices), topk_values.shape[1]
    a.cu_seqlens, a.loss_mask, a.labels = _ptr(cu_seqlens), _ptr(loss_mask), _ptr(labels)
    a.temperature, a.grad_scale = float(temperature), float(grad_scale)
    a.kl, a.nll_student, a.nll_teacher = _ptr(kl), _ptr(nll_student), _ptr(nll_teacher)
    a.d_hidden, a.d_weight = _ptr(d_hidden), _ptr(d_weight)
    a.d_weight_dtype = (NPD_DTYPE_F32 if d_weight is not None and d_weight.dtype == torch.float32
                        else NPD_DTYPE_BF16)
    a.flags, a.grad_chunk_cols = int(flags), int(grad_chunk_cols)
    if kd_lambda is not None:       # composite objective of Eq. 1
        a.flags |= NPD_KD_COMPOSITE_LOSS
        a.kd_lambda = float(kd_lambda)
    if workspace is not None:
        a.workspace, a.workspace_bytes = workspace.data_ptr(), workspace.numel() * workspace.element_size()
    return a


def npd_workspace_bytes(args: npd_kd_args) -> int:
    out = C.c_size_t(0)
    _check(lib().npd_workspace_bytes(C.byref(args), C.byref(out)), "npd_workspace_bytes")
    return out.value


def npd_phase_count(args: npd_kd_args):
    """(launch groups, vocabulary chunks) of a call with these arguments."""
    g, c = C.c_int32(0), C.c_int32(0)
    _check(lib().npd_phase_count(C.byref(args), C.byref(g), C.byref(c)), "npd_phase_count")
    return g.value, c.value


def npd_kd_fwd_bwd(args: npd_kd_args, stream=None) -> None:
    _check(lib().npd_kd_fwd_bwd(C.byref(args), _stream(stream)), "npd_kd_fwd_bwd")


def npd_kd_fwd_bwd_host(host: npd_kd_args, dev: npd_kd_args, stream=None) -> None:
    _check(lib().npd_kd_fwd_bwd_host(C.byref(host), C.byref(dev), _stream(stream)), "npd_kd_fwd_bwd_host")


def npd_kd_fwd_bwd_host_streams(host: npd_kd_args, dev: npd_kd_args, copy_stream, stream=None) -> None:
    _check(lib().npd_kd_fwd_bwd_host_streams(C.byref(host), C.byref(dev), _stream(copy_stream), _stream(stream)),
           "npd_kd_fwd_bwd_host_streams")


def npd_kd_forward_noalloc(args: npd_kd_args, stream=None, want_status: bool = False):
    """Forward pass on the library's built-in scratch array (no workspace, no allocation).
    For callers that cannot allocate device memory; see include/npd.h for the limits.
    With want_status the call synchronises the stream and returns the device status."""
    st = C.c_int32(0)
    _check(lib().npd_kd_forward_noalloc(C.byref(args), _stream(stream), C.byref(st) if want_status else None),
           "npd_kd_forward_noalloc")
    return st.value if want_status else None


def npd_last_status(workspace: torch.Tensor, stream=None) -> int:
    out = C.c_int32(0)
    _check(lib().npd_last_status(workspace.data_ptr(), _stream(stream), C.byref(out)), "npd_last_status")
    return out.value


def npd_last_launch_count() -> int:
    return lib().npd_last_launch_count()


def npd_last_copy_bytes():
    """(host-to-device, device-to-host) bytes of the last npd_kd_fwd_bwd_host call on this thread."""
    a, b = C.c_int64(0), C.c_int64(0)
    _check(lib().npd_last_copy_bytes(C.byref(a), C.byref(b)), "npd_last_copy_bytes")
    return a.value, b.value


def npd_segment_stats(cu_seqlens, loss_mask, labels, kl, nll_student, nll_teacher, *,
                      kl_sum=None, nll_s_sum=None, nll_t_sum=None, count=None, seg_id=None,
                      status=None, stream=None):
    """Per-segment sums and counts.  Allocates the outputs that are not given and
    returns (kl_sum, nll_s_sum, nll_t_sum, count, seg_id)."""
    S = cu_seqlens.numel() - 1
    ref = next(t for t in (kl, nll_student, nll_teacher, loss_mask, labels, cu_seqlens) if t is not None)
    T = ref.numel() if ref is not cu_seqlens else int(cu_seqlens[-1].item())
    dev = cu_seqlens.device
    f = lambda src, out: (torch.empty(S, dtype=torch.float32, device=dev) if out is None and src is not None else out)
    kl_sum, nll_s_sum, nll_t_sum = f(kl, kl_sum), f(nll_student, nll_s_sum), f(nll_teacher, nll_t_sum)
    if count is None:
        count = torch.empty(S, dtype=torch.int32, device=dev)
    if seg_id is None:
        seg_id = torch.empty(T, dtype=torch.int32, device=dev)
    _check(lib().npd_segment_stats(T, S, _ptr(cu_seqlens), _ptr(loss_mask), _ptr(labels), _ptr(kl),
                                   _ptr(nll_student), _ptr(nll_teacher), _ptr(kl_sum), _ptr(nll_s_sum),
                                   _ptr(nll_t_sum), _ptr(count), _ptr(seg_id), _ptr(status),
                                   _stream(stream)), "npd_segment_stats")
    return kl_sum, nll_s_sum, nll_t_sum, count, seg_id


def npd_select(cond_seg, uncond_seg, nll_s_sum, nll_t_sum, count, lo: float, hi: float, flags: int = 0,
               stream=None):
    """Delta-IFD scores and keep mask.  Returns (ifd_teacher, ifd_student, delta, keep, n_keep)."""
    N, S, dev = cond_seg.numel(), count.numel(), cond_seg.device
    ifd_t = torch.empty(N, dtype=torch.float32, device=dev)
    ifd_s = torch.empty(N, dtype=torch.float32, device=dev)
    delta = torch.empty(N, dtype=torch.float32, device=dev)
    keep = torch.empty(N, dtype=torch.uint8, device=dev)
    n_keep = torch.empty(1, dtype=torch.int32, device=dev)
    _check(lib().npd_select(N, _ptr(cond_seg), _ptr(uncond_seg), _ptr(nll_s_sum), _ptr(nll_t_sum),
                            _ptr(count), S, float(lo), float(hi), int(flags), _ptr(ifd_t), _ptr(ifd_s),
                            _ptr(delta), _ptr(keep), _ptr(n_keep), _stream(stream)), "npd_select")
    return ifd_t, ifd_s, delta, keep, n_keep


def npd_perplexity(seg, nll_s_sum, nll_t_sum, count, stream=None):
    """Per-sample perplexities exp(nll_sum / count) of the segments `seg`.  Returns
    (ppl_student, ppl_teacher); an output is None when its sums are None."""
    N, S, dev = seg.numel(), count.numel(), seg.device
    ps = torch.empty(N, dtype=torch.float32, device=dev) if nll_s_sum is not None else None
    pt = torch.empty(N, dtype=torch.float32, device=dev) if nll_t_sum is not None else None
    _check(lib().npd_perplexity(N, _ptr(seg), _ptr(nll_s_sum), _ptr(nll_t_sum), _ptr(count), S, _ptr(ps),
                                _ptr(pt), _stream(stream)), "npd_perplexity")
    return ps, pt


def npd_selftest_wait_timeout(limit_cycles: int, device="cuda", stream=None):
    """Runs the time-out path of the bounded device waits on purpose (see include/npd.h).
    Returns the int32[3] device tensor {status, every wait gave up, cycles waited}."""
    out = torch.empty(3, dtype=torch.int32, device=device)
    _check(lib().npd_selftest_wait_timeout(int(limit_cycles), _ptr(out), _stream(stream)),
           "npd_selftest_wait_timeout")
    return out


def npd_debug_chunk_schedule(row_blocks: int, d: int, chunk_cols: int, pairs: int, pair: int):
    """Host only: the (problem, row, column, k-step begin, k-step end) units of one CTA pair in the
    launch of a chunk's two backward contractions, as an int32 array [n, 5]."""
    import numpy as np
    n = C.c_int32(0)
    cap = 64
    while True:
        units = np.empty((cap, 5), np.int32)
        _check(lib().npd_debug_chunk_schedule(row_blocks, d, chunk_cols, pairs, pair, cap, units.ctypes.data,
                                              C.byref(n)), "npd_debug_chunk_schedule")
        if n.value <= cap:
            return units[: n.value].copy()
        cap = n.value


def npd_pack_sequences(lengths, keep, capacity: int):
    """First-fit-decreasing packing of the kept samples into rows of `capacity` tokens (host only).
    lengths: int32 array-like, keep: uint8 array-like or None.  Returns numpy arrays
    (order, row_of, cu_seqlens, row_ptr)."""
    import numpy as np
    lengths = np.ascontiguousarray(lengths, dtype=np.int32)
    N = lengths.size
    k = None if keep is None else np.ascontiguousarray(keep, dtype=np.uint8)
    order, row_of = np.empty(N, np.int32), np.empty(N, np.int32)
    cu, ptr = np.empty(N + 1, np.int32), np.empty(N + 1, np.int32)
    placed, rows = C.c_int32(0), C.c_int32(0)
    _check(lib().npd_pack_sequences(N, lengths.ctypes.data, None if k is None else k.ctypes.data, int(capacity),
                                    order.ctypes.data, row_of.ctypes.data, cu.ctypes.data, ptr.ctypes.data,
                                    C.addressof(placed), C.addressof(rows)), "npd_pack_sequences")
    return order[:placed.value], row_of[:placed.value], cu[:placed.value + 1], ptr[:rows.value + 1]


def npd_gemm_bf16(A, B, out, *, a_mn_major=False, b_mn_major=False, out_mode=NPD_GEMM_STORE_F32,
                  k_splits=1, stream=None):
    """out[M,N] (+)= sum_k A[m,k] B[n,k].  A is [M,K] (K-major) or [K,M] (MN-major); same for B."""
    M, N = out.shape
    K = A.shape[0] if a_mn_major else A.shape[1]
    _check(lib().npd_gemm_bf16(M, N, K, _ptr(A), A.stride(0), int(a_mn_major), _ptr(B), B.stride(0),
                               int(b_mn_major), _ptr(out), out.stride(0), int(out_mode), int(k_splits),
                               _stream(stream)), "npd_gemm_bf16")
    return out


class KDStep:
    """Holds the output and workspace tensors of one problem shape and runs the
    fused step on them; a convenience over the raw calls."""

    def __init__(self, batch, *, grads=True, dw_dtype=torch.bfloat16, grad_chunk_cols=0, grad_scale=None,
                 kd_lambda=None, topk_values=None, topk_indices=None, flags=0):
        dev = batch.hidden.device
        T, d, V = batch.T, batch.d, batch.V
        f32 = dict(dtype=torch.float32, device=dev)
        self.batch = batch
        self.kl = torch.empty(T, **f32)
        self.nll_student = torch.empty(T, **f32)
        self.nll_teacher = torch.empty(T, **f32) if topk_values is None else None
        self.topk_values, self.topk_indices = topk_values, topk_indices
        # the gradients use the row strides of the tensors they belong to (ldh, ldw)
        self.d_hidden = (torch.empty_strided((T, d), (batch.hidden.stride(0), 1), dtype=torch.bfloat16,
                                             device=dev) if grads else None)
        self.d_weight = (torch.empty_strided((V, d), (batch.weight.stride(0), 1), dtype=dw_dtype,
                                             device=dev) if grads else None)
        self.grad_scale = (1.0 / max(batch.n_loss, 1)) if grad_scale is None else grad_scale
        self._kw = dict(cu_seqlens=batch.cu_seqlens, loss_mask=batch.loss_mask, labels=batch.labels,
                        temperature=batch.tau, grad_scale=self.grad_scale, kl=self.kl,
                        nll_student=self.nll_student, nll_teacher=self.nll_teacher,
                        d_hidden=self.d_hidden, d_weight=self.d_weight, grad_chunk_cols=grad_chunk_cols,
                        kd_lambda=kd_lambda, topk_values=topk_values, topk_indices=topk_indices,
                        flags=flags)
        teacher = batch.teacher if topk_values is None else None
        probe = make_kd_args(batch.hidden, batch.weight, teacher, **self._kw)
        nbytes = npd_workspace_bytes(probe)
        self.workspace = torch.empty(nbytes + 1024, dtype=torch.uint8, device=dev)
        off = (-self.workspace.data_ptr()) % 1024
        self._ws_view = self.workspace[off: off + nbytes]
        self.args = make_kd_args(batch.hidden, batch.weight, teacher, workspace=self._ws_view,
                                 **self._kw)

    def run(self, stream=None):
        npd_kd_fwd_bwd(self.args, stream)

    def phase_names(self):
        """Names of the launch groups of a call, in the order their phase events are recorded."""
        groups, chunks = npd_phase_count(self.args)
        names = ["forward_tiles", "merge"]
        for _ in range(chunks):
            names += ["gradient_tiles", "backward_gemms"]
        names += ["dhidden_convert"] * (groups - len(names))
        return names

    def new_phase_events(self, stream=None):
        """groups + 1 timing events, each recorded once so that it owns a CUDA handle."""
        evs = [torch.cuda.Event(enable_timing=True) for _ in range(len(self.phase_names()) + 1)]
        s = torch.cuda.current_stream() if stream is None else stream
        for e in evs:
            e.record(s)
        return evs

    def run_recording(self, evs, stream=None):
        """One step with the library's phase events attached; only enqueues."""
        arr = (C.c_void_p * len(evs))(*[e.cuda_event for e in evs])
        a = npd_kd_args.from_buffer_copy(self.args)
        a.phase_events = C.cast(arr, C.POINTER(C.c_void_p))
        a.n_phase_events = len(evs)
        npd_kd_fwd_bwd(a, stream)

    def run_with_phase_times(self, stream=None):
        """One step with the library's phase events attached.  Returns a list of
        (group name, milliseconds); synchronises."""
        names = self.phase_names()
        evs = self.new_phase_events(stream)
        self.run_recording(evs, stream)
        torch.cuda.synchronize()
        return [(names[i], evs[i].elapsed_time(evs[i + 1])) for i in range(len(names))]

    def status(self, stream=None) -> int:
        return npd_last_status(self._ws_view, stream)

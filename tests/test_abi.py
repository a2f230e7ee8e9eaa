"""The C-ABI library: it loads, exports every symbol include/npd.h declares, its
struct layout matches the binding, and argument errors are reported on the host
before any CUDA call.  No GPU needed."""

import ctypes as C
import os
import re

import pytest
import torch

from paper_2605_05940_b200 import binding as B
from paper_2605_05940_b200 import build as npd_build

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))


@pytest.fixture(scope="module", autouse=True)
def _built():
    npd_build.build()


def _declared_functions():
    text = open(os.path.join(ROOT, "include", "npd.h")).read()
    text = re.sub(r"/\*.*?\*/", "", text, flags=re.S)
    return sorted(set(re.findall(r"\b(npd_[a-z0-9_]+)\s*\(", text)))


def test_library_exports_every_declared_symbol():
    names = _declared_functions()
    assert {"npd_kd_fwd_bwd", "npd_segment_stats", "npd_select"} <= set(names)
    lib = B.lib()
    for n in names:
        assert hasattr(lib, n), n
    assert set(names) == set(B.EXPORTS)


def test_struct_layout_matches_the_header():
    # compile a tiny C program against the header and compare sizeof/offsets
    import subprocess
    import tempfile
    src = r'''
#include <stdio.h>
#include <stddef.h>
#include "npd.h"
int main(void){ printf("%zu %zu %zu %zu %zu %zu\n", sizeof(npd_kd_args), offsetof(npd_kd_args, ldh),
  offsetof(npd_kd_args, temperature), offsetof(npd_kd_args, d_weight_dtype),
  offsetof(npd_kd_args, workspace), offsetof(npd_kd_args, cu_seqlens)); return 0; }
'''
    with tempfile.TemporaryDirectory() as td:
        c = os.path.join(td, "t.c")
        open(c, "w").write(src)
        exe = os.path.join(td, "t")
        subprocess.run(["gcc", "-std=c99", "-I", os.path.join(ROOT, "include"), c, "-o", exe], check=True)
        got = [int(x) for x in subprocess.run([exe], capture_output=True, text=True, check=True).stdout.split()]
    A = B.npd_kd_args
    want = [C.sizeof(A), A.ldh.offset, A.temperature.offset, A.d_weight_dtype.offset,
            A.workspace.offset, A.cu_seqlens.offset]
    assert got == want


def test_strerror_is_total():
    for code in range(-10, 1):
        assert isinstance(B.strerror(code), str) and B.strerror(code)
    assert B.strerror(0) == "ok" and "cu_seqlens" in B.strerror(B.NPD_ESEQ)


def _args(T=16, d=64, V=40, **kw):
    h = torch.zeros((T, d), dtype=torch.bfloat16)
    w = torch.zeros((V, d), dtype=torch.bfloat16)
    z = torch.zeros((T, V), dtype=kw.pop("tdtype", torch.bfloat16))
    kl = torch.zeros(T)
    return B.make_kd_args(h, w, z, kl=kl, **kw), (h, w, z, kl)


def _ws_rc(a):
    out = C.c_size_t(0)
    return B.lib().npd_workspace_bytes(C.byref(a), C.byref(out))


def test_argument_errors_are_found_on_the_host():
    lib = B.lib()
    a, keep = _args()
    assert lib.npd_workspace_bytes(None, C.byref(C.c_size_t())) == B.NPD_EINVAL
    assert lib.npd_workspace_bytes(C.byref(a), None) == B.NPD_EINVAL
    bad = B.npd_kd_args.from_buffer_copy(a); bad.size = 8
    assert _ws_rc(bad) == B.NPD_EINVAL
    bad = B.npd_kd_args.from_buffer_copy(a); bad.temperature = 0.0
    assert _ws_rc(bad) == B.NPD_EINVAL
    bad = B.npd_kd_args.from_buffer_copy(a); bad.temperature = float("nan")
    assert _ws_rc(bad) == B.NPD_EINVAL
    bad = B.npd_kd_args.from_buffer_copy(a); bad.T = 0
    assert _ws_rc(bad) == B.NPD_EINVAL
    bad = B.npd_kd_args.from_buffer_copy(a); bad.d = 96
    assert _ws_rc(bad) == B.NPD_ESHAPE
    bad = B.npd_kd_args.from_buffer_copy(a); bad.ldt = 32
    assert _ws_rc(bad) == B.NPD_ESHAPE
    bad = B.npd_kd_args.from_buffer_copy(a); bad.ldt = 42
    assert _ws_rc(bad) == B.NPD_EALIGN
    bad = B.npd_kd_args.from_buffer_copy(a); bad.teacher_dtype = 5
    assert _ws_rc(bad) == B.NPD_EINVAL
    bad = B.npd_kd_args.from_buffer_copy(a); bad.topk = 17                  # more than the kernels keep per token
    assert _ws_rc(bad) == B.NPD_EUNSUPPORTED
    bad = B.npd_kd_args.from_buffer_copy(a); bad.d_hidden = 4096            # dH without dW
    assert _ws_rc(bad) == B.NPD_EINVAL
    bad = B.npd_kd_args.from_buffer_copy(a); bad.flags = B.NPD_KD_ACCUMULATE_DW
    assert _ws_rc(bad) == B.NPD_EINVAL                                     # needs f32 dW
    # the compute entry point refuses the same things before touching the device
    bad = B.npd_kd_args.from_buffer_copy(a); bad.kl = None
    assert lib.npd_kd_fwd_bwd(C.byref(bad), None) == B.NPD_EINVAL
    bad = B.npd_kd_args.from_buffer_copy(a); bad.hidden = a.hidden + 2
    assert lib.npd_kd_fwd_bwd(C.byref(bad), None) == B.NPD_EALIGN
    assert lib.npd_segment_stats(0, 1, *([None] * 13)) == B.NPD_EINVAL
    assert lib.npd_select(0, None, None, None, None, None, 1, 0.0, 1.0, 0, *([None] * 6)) == B.NPD_EINVAL
    assert lib.npd_gemm_bf16(0, 8, 8, None, 8, 0, None, 8, 0, None, 8, 0, 1, None) == B.NPD_EINVAL
    assert lib.npd_last_status(None, None, None) == B.NPD_EINVAL


@pytest.mark.skipif(torch.cuda.is_available(), reason="checks the behaviour on a box without a GPU")
def test_no_silent_fallback_without_a_gpu():
    a, keep = _args()
    out = C.c_size_t(0)
    assert B.lib().npd_workspace_bytes(C.byref(a), C.byref(out)) == B.NPD_ECUDA
    with pytest.raises(B.NpdError):
        B.npd_kd_fwd_bwd(a, stream=0)


def test_missing_library_fails_loudly(monkeypatch):
    monkeypatch.setattr(B, "_lib", None)
    monkeypatch.setattr(B, "LIB_PATH", "/nonexistent/libnpd.so")
    with pytest.raises(RuntimeError, match="no CPU or PyTorch fallback"):
        B.lib()


def test_sequence_packer_matches_the_oracle():
    # host-only entry point: runs without a GPU
    import numpy as np
    from oracle import npd_oracle as orc
    rng = np.random.default_rng(0)
    for n, cap in [(0, 8), (1, 8), (5, 8), (200, 512), (3000, 32768)]:
        lengths = rng.integers(0, cap + cap // 4 + 2, size=n).astype(np.int32)
        for keep in (None, (rng.random(n) < 0.7).astype(np.uint8)):
            got = B.npd_pack_sequences(lengths, keep, cap)
            want = orc.pack_first_fit_decreasing(lengths, keep, cap)
            for g, w in zip(got, want):
                assert np.array_equal(g, w)
    assert B.lib().npd_pack_sequences(3, None, None, 8, None, None, None, None, None, None) == B.NPD_EINVAL

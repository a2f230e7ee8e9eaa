"""Seeded synthetic workloads for the packed distillation loss step.

This module only *draws inputs*: random hidden states, LM-head weights, teacher
logits, packed-segment boundaries, loss masks and labels, in the shapes and
distributions of the five benchmark configurations.  It contains none of the
method's loss, gradient, reduction or selection arithmetic and is the single
piece of code that both the CPU oracle's tests and the CUDA library's tests and
benchmark consume.  (The "student-like" teacher of two configurations needs the
product H W^T as part of the *recipe*; it is taken with a plain torch.matmul.)

The inputs stand in for the paper's training data (student roll-outs packed to
fixed-length rows with teacher logits attached), none of which is available.
``N(0, x)`` in a recipe means standard deviation x.
"""

from __future__ import annotations

import dataclasses
import math
from typing import Optional

import numpy as np
import torch

V_QWEN = 151_936
IGNORE = -100


@dataclasses.dataclass
class KDBatch:
    """One packed batch.  Tensors live on ``device``; dtypes as the C-ABI expects."""
    name: str
    T: int
    d: int
    V: int
    S: int
    hidden: torch.Tensor          # bf16 [T, d]
    weight: torch.Tensor          # bf16 [V, d]
    teacher: torch.Tensor         # bf16 or fp32 [T, V]
    cu_seqlens: torch.Tensor      # int32 [S+1]
    loss_mask: torch.Tensor       # uint8 [T]
    labels: torch.Tensor          # int32 [T]
    tau: float
    cond_seg: Optional[torch.Tensor] = None     # int32 [N]  (paired-sample workloads)
    uncond_seg: Optional[torch.Tensor] = None   # int32 [N]

    @property
    def n_loss(self) -> int:
        return int(self.loss_mask.sum().item())


# ----------------------------------------------------------------------------- #
# segment layouts
# ----------------------------------------------------------------------------- #

def _fill_segments(rng: np.random.Generator, T: int, draw) -> np.ndarray:
    """Draw lengths until they reach T; the last one is truncated to fill."""
    cu = [0]
    while cu[-1] < T:
        cu.append(min(T, cu[-1] + int(draw(rng))))
    return np.asarray(cu, dtype=np.int32)


def _mask_and_labels(rng: np.random.Generator, cu: np.ndarray, V: int, prompt_frac,
                     T: int):
    """Prompt = leading floor(frac*len) tokens of a segment (mask 0).  The last
    token of every segment predicts nothing: label IGNORE, mask 0, so that no
    loss term crosses a packed boundary."""
    mask = np.ones(T, dtype=np.uint8)
    labels = rng.integers(0, V, size=T, dtype=np.int64).astype(np.int32)
    for s in range(len(cu) - 1):
        lo, hi = int(cu[s]), int(cu[s + 1])
        frac = prompt_frac(s) if callable(prompt_frac) else prompt_frac
        mask[lo: lo + int(math.floor(frac * (hi - lo)))] = 0
        mask[hi - 1] = 0
        labels[hi - 1] = IGNORE
    return mask, labels


def _randn(shape, std, seed, device, dtype, chunk_rows=4096):
    """Seeded N(0, std) tensor, drawn in row chunks in fp32 and cast."""
    g = torch.Generator(device=device)
    g.manual_seed(seed)
    out = torch.empty(shape, dtype=dtype, device=device)
    for r0 in range(0, shape[0], chunk_rows):
        r1 = min(shape[0], r0 + chunk_rows)
        out[r0:r1] = (torch.randn((r1 - r0,) + tuple(shape[1:]), generator=g,
                                  device=device, dtype=torch.float32) * std).to(dtype)
    return out


def _student_like_teacher(hidden, weight, noise_std, seed, chunk_rows=1024):
    """bf16( fp32(H W^T) + N(0, noise_std) ), built in row chunks."""
    dev = hidden.device
    g = torch.Generator(device=dev)
    g.manual_seed(seed)
    T, V = hidden.shape[0], weight.shape[0]
    out = torch.empty((T, V), dtype=torch.bfloat16, device=dev)
    wt = weight.float().t().contiguous() if dev.type == "cpu" else weight.t()
    for r0 in range(0, T, chunk_rows):
        r1 = min(T, r0 + chunk_rows)
        z = torch.matmul(hidden[r0:r1].float() if dev.type == "cpu" else hidden[r0:r1],
                         wt).float()
        z += torch.randn(z.shape, generator=g, device=dev, dtype=torch.float32) * noise_std
        out[r0:r1] = z.to(torch.bfloat16)
    return out


def _to(dev, *arrs):
    return [torch.from_numpy(np.ascontiguousarray(a)).to(dev) for a in arrs]


# ----------------------------------------------------------------------------- #
# the five configurations
# ----------------------------------------------------------------------------- #

def config1_tiny(device="cpu", teacher_dtype=torch.float32) -> KDBatch:
    """T=256 in 4 segments (32,64,96,64), d=64, V=1000, drawn in fp32 with seed 0:
    H~N(0,1), W~N(0,0.02), teacher~N(0,2) dense, prompt = first 25 % of each
    segment, tau=1.  H and W are rounded to bf16 (what the tensor cores read);
    the teacher keeps fp32 unless ``teacher_dtype`` says bf16."""
    rng = np.random.default_rng(0)
    T, d, V = 256, 64, 1000
    cu = np.asarray([0, 32, 96, 192, 256], dtype=np.int32)
    H = rng.standard_normal((T, d)).astype(np.float32)
    W = (rng.standard_normal((V, d)) * 0.02).astype(np.float32)
    Z = (rng.standard_normal((T, V)) * 2.0).astype(np.float32)
    mask, labels = _mask_and_labels(rng, cu, V, 0.25, T)
    h, w, z, cu_t, m_t, y_t = _to(device, H, W, Z, cu, mask, labels)
    return KDBatch("c1_tiny", T, d, V, 4, h.to(torch.bfloat16), w.to(torch.bfloat16),
                   z.to(teacher_dtype), cu_t, m_t, y_t, 1.0)


def config2_1b(device="cuda", T=8192, d=1536, V=V_QWEN, seed_base=2000,
               min_len=128, max_len=2048) -> KDBatch:
    """~1B-student shape: segments uniform in [128,2048] (last truncated), bf16
    H~N(0,1), W~N(0,0.02), teacher = student-like logits + N(0,1), 30 % of each
    segment prompt-masked, tau=1."""
    rng = np.random.default_rng(seed_base)
    cu = _fill_segments(rng, T, lambda r: r.integers(min_len, max_len + 1))
    mask, labels = _mask_and_labels(rng, cu, V, 0.30, T)
    h = _randn((T, d), 1.0, seed_base + 1, device, torch.bfloat16)
    w = _randn((V, d), 0.02, seed_base + 2, device, torch.bfloat16)
    z = _student_like_teacher(h, w, 1.0, seed_base + 3)
    cu_t, m_t, y_t = _to(device, cu, mask, labels)
    return KDBatch("c2_1b", T, d, V, len(cu) - 1, h, w, z, cu_t, m_t, y_t, 1.0)


def config3_rows(device="cuda", rows=4, row_len=8192, d=2048, V=V_QWEN,
                 seed_base=3000) -> KDBatch:
    """Batch of packed rows: 4 x 8192 tokens, lengths lognormal(6.5, 0.8) clipped
    to [32,8192], no segment spans a row, teacher ~N(0,3) independent of the
    student, 30 % prompt mask, tau=2."""
    rng = np.random.default_rng(seed_base)
    cu = [0]
    for r in range(rows):
        end = (r + 1) * row_len
        while cu[-1] < end:
            ln = int(np.clip(round(math.exp(rng.normal(6.5, 0.8))), 32, 8192))
            cu.append(min(end, cu[-1] + ln))
    cu = np.asarray(cu, dtype=np.int32)
    T = rows * row_len
    mask, labels = _mask_and_labels(rng, cu, V, 0.30, T)
    h = _randn((T, d), 1.0, seed_base + 1, device, torch.bfloat16)
    w = _randn((V, d), 0.02, seed_base + 2, device, torch.bfloat16)
    z = _randn((T, V), 3.0, seed_base + 3, device, torch.bfloat16, chunk_rows=1024)
    cu_t, m_t, y_t = _to(device, cu, mask, labels)
    return KDBatch("c3_rows", T, d, V, len(cu) - 1, h, w, z, cu_t, m_t, y_t, 2.0)


def config4_short(device="cuda", T=16384, d=1536, V=V_QWEN, seed_base=4000,
                  min_len=16, max_len=64) -> KDBatch:
    """Many short samples, generated in pairs for the Delta-IFD filter: segment
    2i is "prompt + answer" (25 % prompt prefix masked), segment 2i+1 is the
    answer alone (only its last token masked).  Labels follow the teacher's
    arg-max with a per-segment probability in [0.2, 0.9], else uniform, which
    spreads the IFD ratios.  Student-like teacher, tau=1."""
    rng = np.random.default_rng(seed_base)
    cu = _fill_segments(rng, T, lambda r: r.integers(min_len, max_len + 1))
    S = len(cu) - 1
    mask, labels = _mask_and_labels(
        rng, cu, V, (lambda s: 0.25 if s % 2 == 0 else 0.0), T)
    h = _randn((T, d), 1.0, seed_base + 1, device, torch.bfloat16)
    w = _randn((V, d), 0.02, seed_base + 2, device, torch.bfloat16)
    z = _student_like_teacher(h, w, 1.0, seed_base + 3)
    amax = torch.empty(T, dtype=torch.int64, device=z.device)
    for r0 in range(0, T, 2048):
        amax[r0:r0 + 2048] = z[r0:r0 + 2048].float().argmax(dim=1)
    amax = amax.cpu().numpy()
    q = rng.uniform(0.2, 0.9, size=S)
    follow = rng.random(T)
    for s in range(S):
        lo, hi = int(cu[s]), int(cu[s + 1]) - 1          # last token stays IGNORE
        sel = follow[lo:hi] < q[s]
        labels[lo:hi][sel] = amax[lo:hi][sel].astype(np.int32)
    n_pairs = S // 2
    cond = np.arange(n_pairs, dtype=np.int32) * 2
    uncond = cond + 1
    cu_t, m_t, y_t, c_t, u_t = _to(device, cu, mask, labels, cond, uncond)
    return KDBatch("c4_short", T, d, V, S, h, w, z, cu_t, m_t, y_t, 1.0, c_t, u_t)


def config5_large(device="cuda", T=65536, d=4096, V=V_QWEN, seed_base=5000) -> KDBatch:
    """Large step: segments uniform in [256,4096], teacher ~N(0,2), 30 % prompt
    mask, tau=1."""
    rng = np.random.default_rng(seed_base)
    cu = _fill_segments(rng, T, lambda r: r.integers(256, 4097))
    mask, labels = _mask_and_labels(rng, cu, V, 0.30, T)
    h = _randn((T, d), 1.0, seed_base + 1, device, torch.bfloat16)
    w = _randn((V, d), 0.02, seed_base + 2, device, torch.bfloat16)
    z = _randn((T, V), 2.0, seed_base + 3, device, torch.bfloat16, chunk_rows=1024)
    cu_t, m_t, y_t = _to(device, cu, mask, labels)
    return KDBatch("c5_large", T, d, V, len(cu) - 1, h, w, z, cu_t, m_t, y_t, 1.0)


def scaled(name: str, device="cpu", **kw) -> KDBatch:
    """A configuration by name with overridden sizes (for cases the CPU oracle
    finishes in seconds)."""
    return {"c2": config2_1b, "c3": config3_rows, "c4": config4_short,
            "c5": config5_large}[name](device=device, **kw)

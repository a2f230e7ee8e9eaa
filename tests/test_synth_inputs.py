"""The seeded input generator: shapes, dtypes, determinism and segment structure."""

import numpy as np
import torch

from oracle import npd_oracle as orc
from paper_2605_05940_b200 import synth_inputs as syn


def _check_structure(b):
    cu = b.cu_seqlens.cpu().numpy()
    assert orc.validate_cu_seqlens(cu, b.T) and len(cu) == b.S + 1
    m = b.loss_mask.cpu().numpy()
    y = b.labels.cpu().numpy()
    assert b.hidden.shape == (b.T, b.d) and b.weight.shape == (b.V, b.d)
    assert b.teacher.shape == (b.T, b.V)
    assert b.hidden.dtype == torch.bfloat16 and b.weight.dtype == torch.bfloat16
    assert b.cu_seqlens.dtype == torch.int32 and b.labels.dtype == torch.int32
    assert b.loss_mask.dtype == torch.uint8
    for s in range(b.S):
        assert y[cu[s + 1] - 1] == syn.IGNORE and m[cu[s + 1] - 1] == 0
    inner = np.ones(b.T, bool)
    inner[cu[1:] - 1] = False
    assert np.all((y[inner] >= 0) & (y[inner] < b.V))


def test_config1_is_the_stated_tiny_case_and_deterministic():
    a, b = syn.config1_tiny(), syn.config1_tiny()
    assert (a.T, a.d, a.V, a.S, a.tau) == (256, 64, 1000, 4, 1.0)
    assert a.cu_seqlens.tolist() == [0, 32, 96, 192, 256]
    assert a.teacher.dtype == torch.float32
    assert torch.equal(a.hidden, b.hidden) and torch.equal(a.teacher, b.teacher)
    _check_structure(a)
    m = a.loss_mask.numpy()
    assert m[:8].sum() == 0 and m[8] == 1          # first 25 % of the 32-token segment
    assert abs(a.teacher.std().item() - 2.0) < 0.05
    assert abs(a.weight.float().std().item() - 0.02) < 0.002


def test_scaled_configs_on_cpu():
    b2 = syn.scaled("c2", T=300, d=64, V=520, min_len=20, max_len=90)
    _check_structure(b2)
    assert abs(1 - b2.n_loss / b2.T - 0.3) < 0.08
    b3 = syn.scaled("c3", rows=2, row_len=256, d=64, V=264)
    _check_structure(b3)
    assert b3.tau == 2.0 and 256 in b3.cu_seqlens.tolist()
    b4 = syn.scaled("c4", T=400, d=64, V=300)
    _check_structure(b4)
    assert b4.cond_seg.tolist() == list(range(0, 2 * (b4.S // 2), 2))
    assert torch.equal(b4.uncond_seg, b4.cond_seg + 1)
    b5 = syn.scaled("c5", T=5000, d=32, V=128)
    _check_structure(b5)
    again = syn.scaled("c2", T=300, d=64, V=520, min_len=20, max_len=90)
    assert torch.equal(again.teacher, b2.teacher) and torch.equal(again.labels, b2.labels)

"""The unit schedule of the launch that holds a chunk's two backward contractions, checked on
the host: the library evaluates the kernel's own scheduling code for every CTA pair
(npd_debug_chunk_schedule) and the test checks that the units tile both products exactly once,
that the pairs carry (almost) the same number of k-steps, and that the members of a group
sweep the same rows at the same time (which is what lets them share the operand through L2)."""

import numpy as np
import pytest

from paper_2605_05940_b200 import binding as B

PM, BN, BK = 256, 512, 64


def _all_units(row_blocks, d, cols, pairs):
    return [B.npd_debug_chunk_schedule(row_blocks, d, cols, pairs, p) for p in range(pairs)]


CASES = [
    (45, 1536, 15360, 74),     # the benchmark's shape: 5760 compact rows, 10 chunks
    (45, 1536, 15104, 74),     # its ragged last chunk is narrower
    (180, 2048, 15360, 74),    # d = 2048: four column tiles, 18 groups + 2 lone pairs
    (359, 4096, 9728, 74),     # d = 4096: eight column tiles
    (12, 1536, 38144, 74),     # few rows, wide chunk
    (1, 64, 256, 74),          # tiny: one tile each
    (3, 192, 1000, 5),         # ragged everything, few pairs
    (7, 1536, 4096, 2),        # fewer pairs than column tiles: the ungrouped walk
    (0, 1536, 4096, 74),       # no token carries loss
    (45, 1536, 15360, 66),     # a device with fewer SMs
]


@pytest.mark.parametrize("row_blocks,d,cols,pairs", CASES)
def test_units_tile_both_products_exactly_once(row_blocks, d, cols, pairs):
    units = _all_units(row_blocks, d, cols, pairs)
    rows = 128 * row_blocks
    tn = -(-d // BN)
    k_dw, k_dh = -(-rows // BK), -(-cols // BK)
    mt_dw, mt_dh = -(-cols // PM), -(-rows // PM)
    cover_dw = np.zeros((mt_dw, tn, max(k_dw, 1)), np.int32)
    cover_dh = np.zeros((mt_dh, tn, max(k_dh, 1)), np.int32)
    zero_k_tiles = set()
    for u in units:
        for prob, m0, n0, k0, k1 in u:
            assert m0 % PM == 0 and n0 % BN == 0 and 0 <= k0 <= k1
            cov = cover_dw if prob == 0 else cover_dh
            assert m0 // PM < cov.shape[0] and n0 // BN < tn
            if k0 == k1:
                zero_k_tiles.add((prob, m0, n0))
            cov[m0 // PM, n0 // BN, k0:k1] += 1
    if k_dw > 0:
        assert np.all(cover_dw[:, :, :k_dw] == 1)
    else:   # no rows: every dW tile is still visited once (it is written with zeros)
        assert len([t for t in zero_k_tiles if t[0] == 0]) == mt_dw * tn
    if mt_dh > 0:
        assert np.all(cover_dh[:, :, :k_dh] == 1)


@pytest.mark.parametrize("row_blocks,d,cols,pairs", CASES[:5] + CASES[-1:])
def test_pairs_carry_about_the_same_number_of_k_steps(row_blocks, d, cols, pairs):
    units = _all_units(row_blocks, d, cols, pairs)
    load = np.asarray([sum(int(k1 - k0) for _, _, _, k0, k1 in u) for u in units], np.float64)
    total = load.sum()
    # nobody carries more than a few per cent above the even share (whole dW tiles cannot be cut)
    assert load.max() <= 1.04 * total / pairs + 1
    # the pairs outside the groups never exceed the even share
    tn = -(-d // BN)
    lone = pairs - (pairs // tn) * tn
    if lone:
        assert load[-lone:].max() <= total / pairs + 1


@pytest.mark.parametrize("row_blocks,d,cols,pairs", CASES[:5])
def test_group_members_sweep_the_same_rows_in_lockstep(row_blocks, d, cols, pairs):
    units = _all_units(row_blocks, d, cols, pairs)
    tn = -(-d // BN)
    groups = pairs // tn
    for g in range(groups):
        members = units[g * tn:(g + 1) * tn]
        ref = members[0]
        for j, u in enumerate(members):
            assert len(u) == len(ref)
            # same problem, same rows, same k range, unit by unit; only the column tile differs
            assert np.array_equal(u[:, [0, 1, 3, 4]], ref[:, [0, 1, 3, 4]])
            assert np.all(u[:, 2] == j * BN)

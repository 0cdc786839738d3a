"""How much of the input a layer could skip under the paper's adaptive setting (Sec. 3.1: a group as long as
the input-channel axis, N = (1 - sparsity) * M), counted on the CPU with the oracle's pruner on the
benchmark's synthetic ResNet-50 weights: 32-byte sectors (8 consecutive channels of one tap) and
32-column blocks (one shared-memory operand stage) in which NO tile of a 256-channel work item retains a column.

The counts decide whether a kernel that skips dead blocks, or a byte count that excludes dead sectors, is
worth having.  They are essentially zero: the retained columns of independent tiles cover every sector, so the
bytes a layer must read do not shrink and no operand stage can be skipped (for weights whose importance is
not correlated across tiles, as these are; trained networks may differ)."""
import numpy as np
import pytest

import oracle
from paper_2507_17301_b200 import inputs

LAYERS = ("s1b1_c2", "s1b2_c1", "s2b2_c2", "s3b2_c1", "s3b2_c2", "s4b2_c2")


def _dead_fractions(s, li, sparsity, tile_t):
    w = inputs.make_weights(s, li).numpy().reshape(s.c_out, -1)
    m = s.c_in
    n = max(1, round(m * (1.0 - sparsity)))
    _, idx = oracle.prune(w, n, m, tile_t)
    k, n_tiles = w.shape[1], idx.shape[0]
    keep = np.zeros((n_tiles, k), dtype=bool)
    for t in range(n_tiles):
        keep[t, idx[t]] = True
    g = max(1, min(n_tiles, 256 // tile_t))                      # tiles of one 256-channel work item
    item = keep.reshape(n_tiles // g, g, k).any(axis=1)
    sectors_tile = 1.0 - keep.reshape(n_tiles, k // 8, 8).any(axis=2).mean()
    sectors_item = 1.0 - item.reshape(-1, k // 8, 8).any(axis=2).mean()
    blocks_item = 1.0 - item.reshape(-1, k // 32, 32).any(axis=2).mean()
    return sectors_tile, sectors_item, blocks_item, g


@pytest.mark.parametrize("tile_t", [8, 64])
@pytest.mark.parametrize("sparsity", [0.5, 0.75])
def test_dead_sectors_and_blocks_under_adaptive_m(sparsity, tile_t):
    stack = {s.name: (li, s) for li, s in enumerate(inputs.resnet_conv_stack(50, 1, 2, 4, tile_t=tile_t))}
    for name in LAYERS:
        li, s = stack[name]
        sectors_tile, sectors_item, blocks_item, g = _dead_fractions(s, li, sparsity, tile_t)
        assert blocks_item == 0.0, f"{name}: a 32-column block without survivors"      # nothing for a kernel to skip
        if g > 1:
            assert sectors_item < 0.01, f"{name}: {sectors_item:.4f} of the sectors dead for a work item"
        # a single tile does lose sectors at 75 % sparsity (about a tenth), but never more than an eighth
        assert sectors_tile <= 0.13 if sparsity > 0.5 else sectors_tile < 0.02

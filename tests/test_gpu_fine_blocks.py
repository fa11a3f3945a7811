"""GPU parity for block masks whose blocks are finer than the kernels' 128 x 128 tiles (block edge 32 or 64;
the sparse setting of Section 4.1 with a finer pattern): the tensor-core kernels visit the tiles that keep at
least one block and mask the other blocks' entries inside them.  Every algorithm, with and without the causal
mask on top, ragged sizes, per-head masks, rows and columns that keep nothing."""
import numpy as np
import pytest

from paper_2410_09397_b200 import inputs
from tests import helpers as H

pytestmark = pytest.mark.gpu
BS, BC = inputs.MASK_BLOCK_SPARSE, inputs.MASK_BLOCK_SPARSE_CAUSAL


def cfgs():
    from paper_2410_09397_b200 import binding as B
    return {"fused128": B.Cfg(algo=B.ATTN_ALGO_FUSED), "fused64": B.Cfg(tile_q=64, algo=B.ATTN_ALGO_FUSED),
            "no_atomics": B.Cfg(algo=B.ATTN_ALGO_FUSED, deterministic=1)}


def _skip(which, d):
    if d == 256 and which != "fused64":
        pytest.skip("d = 256: the fused backward has 64-query tiles only")
    if d == 64 and which == "fused64":
        pytest.skip("64-query tiles: d = 128 and 256")


@pytest.mark.parametrize("which", ["fused128", "fused64", "no_atomics"])
@pytest.mark.parametrize("kind", [BS, BC])
@pytest.mark.parametrize("n,block,d", [(512, 64, 128), (640, 32, 64), (600, 32, 128), (520, 64, 256), (384, 32, 256)])
def test_fine_blocks_tensor_core_paths(which, kind, n, block, d):
    _skip(which, d)
    errs = H.run_case(1, 2, n, d, "bf16", kind, seed=81, block=block, keep_prob=0.35, cfg=cfgs()[which])
    H.assert_within(errs, "bf16")


@pytest.mark.parametrize("which", ["fused128", "fused64", "no_atomics"])
def test_fine_blocks_per_head_masks_empty_rows_and_columns(which):
    """Head 0: a sparse random pattern of 32-wide blocks; head 1: query rows 64..95 and key columns 160..191 keep
    nothing although their 128 x 128 tiles are visited; head 2: a whole 128-wide tile row and tile column empty."""
    n, block, b, h = 512, 32, 1, 3
    nb = n // block
    bm = np.zeros((b * h, nb, nb), dtype=np.uint8)
    bm[0] = inputs.block_mask(83, nb, 0.2)
    bm[1] = inputs.block_mask(84, nb, 0.5)
    bm[1, 2, :] = 0
    bm[1, :, 5] = 0
    bm[2] = inputs.block_mask(85, nb, 0.5)
    bm[2, 4:8, :] = 0
    bm[2, :, 8:12] = 0
    errs = H.run_case(b, h, n, 128, "bf16", BS, seed=82, block=block, bmask=bm, cfg=cfgs()[which])
    H.assert_within(errs, "bf16")


def test_fine_blocks_auto_picks_the_tensor_cores():
    """ATTN_ALGO_AUTO with a 64-wide block mask resolves to the fused kernels (workspace holds the tile lists)."""
    import torch
    import paper_2410_09397_b200 as attn
    from paper_2410_09397_b200 import binding as B
    n = 512
    bm = torch.ones(1, n // 64, n // 64, dtype=torch.uint8, device="cuda")
    mask = attn.Mask(kind=attn.ATTN_MASK_BLOCK_SPARSE, block=64, block_mask=bm)
    fused = attn.attn_bwd_workspace_bytes(n, 128, 1, 1, mask, attn.ATTN_BF16, B.Cfg(algo=B.ATTN_ALGO_FUSED))
    assert fused > 0 and attn.attn_bwd_workspace_bytes(n, 128, 1, 1, mask, attn.ATTN_BF16, None) == fused
    bad = attn.Mask(kind=attn.ATTN_MASK_BLOCK_SPARSE, block=16, block_mask=bm)
    assert attn.attn_bwd_workspace_bytes(n, 128, 1, 1, bad, attn.ATTN_BF16, B.Cfg(algo=B.ATTN_ALGO_FUSED)) == 0

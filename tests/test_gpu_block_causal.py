"""GPU parity for the mask "block mask AND causal" (a sparse score matrix in the sense of Section 4.1 whose
kept entries also satisfy j <= i) on every algorithm: the fused kernels with 128- and 64-query tiles, the path
without atomics, and the fp32 FMA kernels.  The oracle's version of this mask is pinned against an explicit
n x n element mask."""
import numpy as np
import pytest

from paper_2410_09397_b200 import inputs
from tests import helpers as H

pytestmark = pytest.mark.gpu
BC = inputs.MASK_BLOCK_SPARSE_CAUSAL


def cfgs():
    from paper_2410_09397_b200 import binding as B
    return {"fused128": B.Cfg(algo=B.ATTN_ALGO_FUSED), "fused64": B.Cfg(tile_q=64, algo=B.ATTN_ALGO_FUSED),
            "no_atomics": B.Cfg(algo=B.ATTN_ALGO_FUSED, deterministic=1)}


@pytest.mark.parametrize("which", ["fused128", "fused64", "no_atomics"])
@pytest.mark.parametrize("n,block,d", [(512, 128, 128), (1024, 256, 64), (600, 128, 128), (896, 128, 256)])
def test_block_causal_tensor_core_paths(which, n, block, d):
    if d == 256 and which != "fused64":
        pytest.skip("d = 256: the fused backward has 64-query tiles only")
    if d == 64 and which == "fused64":
        pytest.skip("64-query tiles: d = 128 and 256")
    errs = H.run_case(1, 3, n, d, "bf16", BC, seed=71, block=block, keep_prob=0.5, cfg=cfgs()[which])
    H.assert_within(errs, "bf16")


def test_block_causal_rows_and_columns_without_any_kept_entry():
    """Diagonal blocks dropped: query rows of those blocks may keep nothing (O = 0, LSE = -inf, no gradient),
    and key columns may be visited by no query tile at all."""
    n, block, b, h = 768, 128, 1, 2
    nb = n // block
    bm = np.zeros((b * h, nb, nb), dtype=np.uint8)
    bm[0] = np.tril(np.ones((nb, nb), np.uint8))
    bm[0, 3, 3] = 0                       # rows 384..511 lose their diagonal block but keep earlier ones
    bm[1] = np.eye(nb, dtype=np.uint8)
    bm[1, 2, 2] = 0                       # rows 256..383 keep nothing; key block 2 is visited by nobody
    bm[1, 0, 5] = 1                       # kept by the block mask, dropped by causality
    for which in ("fused128", "fused64", "no_atomics"):
        errs = H.run_case(b, h, n, 128, "bf16", BC, seed=72, block=block, bmask=bm, cfg=cfgs()[which])
        H.assert_within(errs, "bf16")


@pytest.mark.parametrize("n,block", [(96, 16), (200, 24)])
def test_block_causal_fp32_path(n, block):
    errs = H.run_case(1, 2, n, 64, "f32", BC, seed=73, block=block, keep_prob=0.5)
    H.assert_within(errs, "f32")


def test_block_causal_is_refused_by_the_materialised_algorithm():
    import torch
    import paper_2410_09397_b200 as attn
    bm = torch.ones(1, 2, 2, dtype=torch.uint8, device="cuda")
    mask = attn.Mask(kind=attn.ATTN_MASK_BLOCK_SPARSE_CAUSAL, block=128, block_mask=bm)
    cfg = attn.Cfg(algo=attn.ATTN_ALGO_MATERIALIZED)
    assert attn.attn_bwd_workspace_bytes(256, 256, 1, 1, mask, attn.ATTN_BF16, cfg) == 0

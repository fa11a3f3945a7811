"""GPU parity of the fused backward with 64-query tiles against the float64 oracle.

This is the second tile shape of the key-stationary (large-cache) backward: tile_q = 64 at d = 128, and the
only fused shape at d = 256, where two CTAs share a key tile and each owns 128 columns of dK, dV and dQ.
Tolerance for bf16 inputs with fp32 accumulation: max|err| <= 2e-2 * max|ref| per tensor.
"""
import pytest

from paper_2410_09397_b200 import inputs
from tests import helpers as H

pytestmark = pytest.mark.gpu


def fused64():
    from paper_2410_09397_b200 import binding as B
    return B.Cfg(tile_q=64, algo=B.ATTN_ALGO_FUSED)


@pytest.mark.parametrize("d", [128, 256])
@pytest.mark.parametrize("n", [64, 256, 1000])
@pytest.mark.parametrize("mask_kind", [inputs.MASK_NONE, inputs.MASK_CAUSAL])
def test_fused64_backward(n, d, mask_kind):
    """Several key tiles and query tiles, a ragged tail (n = 1000), a single half-filled key tile (n = 64)."""
    errs = H.run_case(1, 2, n, d, "bf16", mask_kind, seed=61, cfg=fused64())
    H.assert_within(errs, "bf16")


@pytest.mark.parametrize("d", [128, 256])
@pytest.mark.parametrize("n", [8, 136, 1672])
def test_fused64_ragged_and_many_tiles(n, d):
    """n = 1672: 27 query tiles per key tile, so every stage ring and barrier phase wraps many times."""
    errs = H.run_case(2, 1, n, d, "bf16", inputs.MASK_CAUSAL, seed=62, cfg=fused64())
    H.assert_within(errs, "bf16")


@pytest.mark.parametrize("d", [128, 256])
@pytest.mark.parametrize("n,block", [(512, 128), (1024, 256), (600, 128)])
def test_fused64_block_sparse(n, d, block):
    errs = H.run_case(1, 3, n, d, "bf16", inputs.MASK_BLOCK_SPARSE, seed=63, block=block, keep_prob=0.3, cfg=fused64())
    H.assert_within(errs, "bf16")


def test_fused64_block_sparse_empty_columns_and_per_head_masks():
    """A block column without any kept row: the CTA loads K_j, V_j, visits nothing and must write zeros."""
    import numpy as np
    n, block, b, h = 768, 128, 1, 2
    nb = n // block
    bm = np.zeros((b * h, nb, nb), dtype=np.uint8)
    for hh in range(b * h):
        for i in range(nb):
            bm[hh, i, (i + hh) % nb] = 1
        bm[hh, :, 2] = 0          # key block 2 is never visited
        bm[hh, 2, 0] = 1          # ... but its query rows still have a kept key
    for d in (128, 256):
        errs = H.run_case(b, h, n, d, "bf16", inputs.MASK_BLOCK_SPARSE, seed=64, block=block, bmask=bm, cfg=fused64())
        H.assert_within(errs, "bf16")


def test_fused64_is_what_auto_runs_for_the_backward_at_d256():
    from paper_2410_09397_b200 import binding as B
    import paper_2410_09397_b200 as attn
    cfgs = attn.attn_supported_cfgs(256, B.ATTN_BF16)
    assert any(c.algo == B.ATTN_ALGO_FUSED and c.tile_q == 64 and c.tile_k == 128 for c in cfgs)
    # both regimes of the paper can be run at the same head dimension
    assert any(c.algo == B.ATTN_ALGO_MATERIALIZED for c in cfgs)
    m_fused = attn.attn_cfg_onchip_elems(256, B.ATTN_BF16, B.Cfg(algo=B.ATTN_ALGO_FUSED), True)
    m_mat = attn.attn_cfg_onchip_elems(256, B.ATTN_BF16, B.Cfg(algo=B.ATTN_ALGO_MATERIALIZED), True)
    assert m_fused >= 256 * 256 > 0 and m_mat > 0     # the fused CTA holds at least d^2 elements (large-cache regime)
    attn.attn_timing_enable(True)
    attn.attn_timing_collect()
    errs = H.run_case(1, 1, 384, 256, "bf16", inputs.MASK_CAUSAL, seed=65, cfg=None, check_bwd_only=False)
    names = [k for k, _ in attn.attn_timing_collect()]
    attn.attn_timing_enable(False)
    H.assert_within(errs, "bf16")
    assert "tc_bwd_fused64" in names, names


def test_fused64_d256_without_atomics_is_refused():
    import torch
    import paper_2410_09397_b200 as attn
    from paper_2410_09397_b200 import binding as B
    assert attn.attn_bwd_workspace_bytes(256, 256, 1, 1, None, B.ATTN_BF16, B.Cfg(tile_q=64, algo=B.ATTN_ALGO_FUSED, deterministic=1)) == 0

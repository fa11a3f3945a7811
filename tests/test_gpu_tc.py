"""GPU parity of the tensor-core (tcgen05 / TMEM / TMA) kernels against the float64 oracle.

Tolerance for bf16 inputs with fp32 accumulation: max|err| <= 2e-2 * max|ref| per tensor.
"""
import numpy as np
import pytest

from paper_2410_09397_b200 import inputs
from tests import helpers as H

pytestmark = pytest.mark.gpu


def fused():
    from paper_2410_09397_b200 import binding as B
    return B.Cfg(algo=B.ATTN_ALGO_FUSED)


@pytest.mark.parametrize("d", [64, 128])
@pytest.mark.parametrize("n", [128, 256, 640])
@pytest.mark.parametrize("mask_kind", [inputs.MASK_NONE, inputs.MASK_CAUSAL])
def test_fused_small(n, d, mask_kind):
    errs = H.run_case(1, 2, n, d, "bf16", mask_kind, seed=31, cfg=fused())
    H.assert_within(errs, "bf16")


@pytest.mark.parametrize("d", [64, 128])
@pytest.mark.parametrize("n", [8, 136, 200, 1000])
@pytest.mark.parametrize("mask_kind", [inputs.MASK_NONE, inputs.MASK_CAUSAL])
def test_fused_ragged_tails(n, d, mask_kind):
    """n not a multiple of the 128-row tile: TMA zero fill + masked tail columns."""
    errs = H.run_case(2, 1, n, d, "bf16", mask_kind, seed=32, cfg=fused())
    H.assert_within(errs, "bf16")


@pytest.mark.parametrize("d", [64, 128])
@pytest.mark.parametrize("n,block", [(512, 128), (1024, 256), (896, 128), (600, 128)])
def test_fused_block_sparse(n, d, block):
    errs = H.run_case(1, 3, n, d, "bf16", inputs.MASK_BLOCK_SPARSE, seed=33, block=block, keep_prob=0.3, cfg=fused())
    H.assert_within(errs, "bf16")


def test_fused_block_sparse_per_head_masks_and_empty_columns():
    b, h, n, d, block = 1, 2, 512, 64, 128
    bm = inputs.block_mask(34, n // block, 0.4, heads=b * h)
    bm[1, :, 2] = 0          # no query attends to key block 2 of head 1: dK = dV = 0 there
    bm[1, 2, 2] = 0
    bm[1, 2, 0] = 1          # row 2 still has a kept block
    errs = H.run_case(b, h, n, d, "bf16", inputs.MASK_BLOCK_SPARSE, seed=34, block=block, bmask=bm, cfg=fused())
    H.assert_within(errs, "bf16")


@pytest.mark.parametrize("n", [128, 320, 1024])
@pytest.mark.parametrize("mask_kind", [inputs.MASK_NONE, inputs.MASK_CAUSAL])
def test_forward_d256(n, mask_kind):
    """d = 256 forward runs fused (64-key tiles); its backward is not the fused kernel."""
    import torch
    import paper_2410_09397_b200 as attn
    from oracle import oracle as orc
    x = H.make_inputs(35, 1, 2, n, 256, "bf16")
    O_ref, LSE_ref = orc.attn_fwd(x["Q"], x["K"], x["V"], mask_kind=mask_kind)
    dev = {k: H.to_dev(v, "bf16") for k, v in x.items()}
    mask = attn.Mask(kind=mask_kind) if mask_kind else None
    O, LSE = attn.attn_fwd(dev["Q"], dev["K"], dev["V"], mask=mask, cfg=fused())
    torch.cuda.synchronize()
    assert H.rel_err(H.to_np(O), O_ref) <= 2e-2
    assert H.rel_err(H.to_np(LSE), LSE_ref) <= 2e-2


def test_auto_selects_tensor_cores_for_bf16():
    errs = H.run_case(2, 2, 512, 128, "bf16", inputs.MASK_CAUSAL, seed=36)
    H.assert_within(errs, "bf16")
    import paper_2410_09397_b200 as attn
    attn.attn_timing_enable(True)
    attn.attn_timing_collect()
    H.run_case(1, 1, 256, 128, "bf16", inputs.MASK_NONE, seed=36, check_bwd_only=False)
    names = [k for k, _ in attn.attn_timing_collect()]
    attn.attn_timing_enable(False)
    assert "tc_fwd" in names and "tc_bwd_fused" in names, names


def test_large_scores_trigger_rescale():
    """Scores that grow along the key axis force the running maximum to move (O rescale path)."""
    import torch
    import paper_2410_09397_b200 as attn
    from oracle import oracle as orc
    n, d = 512, 64
    x = H.make_inputs(37, 1, 1, n, d, "bf16")
    ramp = np.linspace(0.0, 6.0, n, dtype=np.float32)[None, None, :, None]
    x["K"] = inputs.round_to_bf16((x["K"] * 0.2 + ramp * np.sign(x["Q"].mean())).astype(np.float32))
    x["Q"] = inputs.round_to_bf16(np.abs(x["Q"]).astype(np.float32))
    O_ref, LSE_ref = orc.attn_fwd(x["Q"], x["K"], x["V"])
    dev = {k: H.to_dev(v, "bf16") for k, v in x.items()}
    O, LSE = attn.attn_fwd(dev["Q"], dev["K"], dev["V"], cfg=fused())
    torch.cuda.synchronize()
    assert H.rel_err(H.to_np(O), O_ref) <= 2e-2
    assert H.rel_err(H.to_np(LSE), LSE_ref) <= 2e-2


@pytest.mark.parametrize("d", [64, 128])
@pytest.mark.parametrize("n", [384, 1152])
@pytest.mark.parametrize("mask_kind", [inputs.MASK_NONE, inputs.MASK_CAUSAL])
@pytest.mark.parametrize("big", ["odd", "even", "rising"])
def test_forward_merges_partial_softmaxes_with_unequal_maxima(n, d, mask_kind, big):
    """The two softmax warpgroups own alternate 128-key tiles and are merged at the end: make the scores of one
    family of tiles (or of the late tiles) far larger than the others', so that the merge weights differ by
    many orders of magnitude and the running maxima have to move."""
    import torch
    import paper_2410_09397_b200 as attn
    from oracle import oracle as orc
    x = H.make_inputs(41, 1, 2, n, d, "bf16")
    tile = np.arange(n) // 128
    if big == "rising":
        shift = np.linspace(0.0, 5.0, n, dtype=np.float32)
    else:
        shift = np.where(tile % 2 == (1 if big == "odd" else 0), 4.0, 0.0).astype(np.float32)
    x["Q"] = inputs.round_to_bf16(np.abs(x["Q"]).astype(np.float32))                       # positive queries:
    x["K"] = inputs.round_to_bf16((x["K"] * 0.2 + shift[None, None, :, None]).astype(np.float32))   # score ~ shift * |q|_1
    O_ref, LSE_ref = orc.attn_fwd(x["Q"], x["K"], x["V"], mask_kind=mask_kind)
    dev = {k: H.to_dev(v, "bf16") for k, v in x.items()}
    mask = attn.Mask(kind=mask_kind) if mask_kind else None
    O, LSE = attn.attn_fwd(dev["Q"], dev["K"], dev["V"], mask=mask, cfg=fused())
    torch.cuda.synchronize()
    # forward only: with a common offset of 4 on the keys dQ = scale * dS K is a difference of large terms, and
    # the bf16 rounding of dS (part of the method's storage format) then dominates a tolerance relative to max|dQ|
    H.assert_within({"O": H.rel_err(H.to_np(O), O_ref), "LSE": H.rel_err(H.to_np(LSE), LSE_ref)}, "bf16")


def materialized(tile_k=0, tile_q=0):
    from paper_2410_09397_b200 import binding as B
    return B.Cfg(tile_q=tile_q, tile_k=tile_k, algo=B.ATTN_ALGO_MATERIALIZED)


@pytest.mark.parametrize("tile_q", [128, 256])
@pytest.mark.parametrize("tile_k", [128, 64, 32])
@pytest.mark.parametrize("n,d", [(256, 256), (1000, 256), (384, 128), (200, 64)])
@pytest.mark.parametrize("mask_kind", [inputs.MASK_NONE, inputs.MASK_CAUSAL])
def test_materialized_backward(n, d, tile_k, tile_q, mask_kind):
    """Small-cache algorithm: P, dP, dS go through device memory; blocks of 128 or 256 rows by 128, 64 or 32 columns
    (sizes with a ragged last block in either direction, and more tiles than one CTA's two accumulator sets)."""
    errs = H.run_case(1, 2, n, d, "bf16", mask_kind, seed=38, cfg=materialized(tile_k, tile_q))
    H.assert_within(errs, "bf16")


def test_materialized_backward_many_tiles_per_cta():
    """More tiles than resident CTAs: every CTA of the persistent products walks several tiles, so that the operand
    ring, both accumulator sets and both staging tiles wrap (n = 2432: 19 x 19 blocks x 10 heads = 3610 tiles)."""
    errs = H.run_case(2, 5, 2432, 64, "bf16", inputs.MASK_CAUSAL, seed=40, cfg=materialized(128, 128), check_bwd_only=False)
    H.assert_within(errs, "bf16")


def test_materialized_rejects_block_sparse_and_runs_its_own_phases():
    import torch
    import paper_2410_09397_b200 as attn
    from paper_2410_09397_b200 import binding as B
    bm = torch.ones(1, 2, 2, dtype=torch.uint8, device="cuda")
    mask = attn.Mask(kind=attn.ATTN_MASK_BLOCK_SPARSE, block=128, block_mask=bm)
    assert attn.attn_bwd_workspace_bytes(256, 256, 1, 1, mask, attn.ATTN_BF16, materialized()) == 0
    attn.attn_timing_enable(True)
    attn.attn_timing_collect()
    errs = H.run_case(1, 1, 256, 256, "bf16", inputs.MASK_NONE, seed=39, check_bwd_only=False, cfg=materialized())
    names = [k for k, _ in attn.attn_timing_collect()]
    attn.attn_timing_enable(False)
    H.assert_within(errs, "bf16")
    assert "mat_phase1_P" in names and "mat_phase4_dQ" in names, names


def fused_det():
    from paper_2410_09397_b200 import binding as B
    return B.Cfg(algo=B.ATTN_ALGO_FUSED, deterministic=1)


@pytest.mark.parametrize("d", [64, 128])
@pytest.mark.parametrize("n", [128, 640, 1000])
@pytest.mark.parametrize("mask_kind", [inputs.MASK_NONE, inputs.MASK_CAUSAL, inputs.MASK_BLOCK_SPARSE])
def test_deterministic_backward_without_atomics(n, d, mask_kind):
    """deterministic = 1: dK, dV from the key-stationary kernel, dQ from the query-stationary one."""
    errs = H.run_case(1, 2, n, d, "bf16", mask_kind, seed=40, block=128, cfg=fused_det())
    H.assert_within(errs, "bf16")


def test_deterministic_backward_is_bitwise_repeatable():
    import torch
    import paper_2410_09397_b200 as attn
    x = H.make_inputs(41, 2, 2, 768, 128, "bf16")
    dev = {k: H.to_dev(v, "bf16") for k, v in x.items()}
    mask = attn.Mask(kind=attn.ATTN_MASK_CAUSAL)
    O, LSE = attn.attn_fwd(dev["Q"], dev["K"], dev["V"], mask=mask, cfg=fused_det())
    runs = []
    for _ in range(3):
        g = attn.attn_bwd(dev["Q"], dev["K"], dev["V"], O, dev["dO"], LSE, mask=mask, cfg=fused_det())
        torch.cuda.synchronize()
        runs.append([t.clone() for t in g])
    for other in runs[1:]:
        for a, b in zip(runs[0], other):
            assert torch.equal(a, b)


@pytest.mark.parametrize("b,h", [(1, 3), (3, 2), (3, 4), (1, 8), (5, 1)])
@pytest.mark.parametrize("deterministic", [0, 1])
def test_head_group_sizes_and_explicit_scale(b, h, deterministic):
    """batch * heads = 3, 6, 12, 8, 5: the launch groups heads by 1, 2, 4, 8, 1; the scale is not 1/sqrt(d)."""
    from paper_2410_09397_b200 import binding as B
    cfg = B.Cfg(algo=B.ATTN_ALGO_FUSED, deterministic=deterministic)
    errs = H.run_case(b, h, 392, 128, "bf16", inputs.MASK_CAUSAL, seed=41, cfg=cfg, scale=0.11, check_bwd_only=False)
    H.assert_within(errs, "bf16")


@pytest.mark.parametrize("d", [64, 128])
def test_deterministic_block_sparse_with_per_head_masks(d):
    from paper_2410_09397_b200 import binding as B
    b, h, n, block = 2, 2, 768, 128
    bm = inputs.block_mask(42, n // block, 0.35, heads=b * h)
    cfg = B.Cfg(algo=B.ATTN_ALGO_FUSED, deterministic=1)
    errs = H.run_case(b, h, n, d, "bf16", inputs.MASK_BLOCK_SPARSE, seed=42, block=block, bmask=bm, cfg=cfg)
    H.assert_within(errs, "bf16")

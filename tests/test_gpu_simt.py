"""GPU parity of the fp32 FMA path (and D pre-pass) against the float64 oracle, through the C ABI."""
import numpy as np
import pytest

from paper_2410_09397_b200 import inputs
from tests import helpers as H

pytestmark = pytest.mark.gpu


def simt_cfg():
    from paper_2410_09397_b200 import binding as B
    return B.Cfg(algo=B.ATTN_ALGO_SIMT)


def test_config1_fp32_exact_check():
    """batch=1, heads=1, n=128, d=64, fp32, seed 0, no mask: tolerance 1e-4."""
    w = inputs.WORKLOADS["C1"]
    errs = H.run_case(w.batch, w.heads, w.n, w.d, "f32", w.mask, seed=w.seed)
    H.assert_within(errs, "f32")


@pytest.mark.parametrize("n,d", [(1, 8), (7, 16), (65, 24), (200, 72), (333, 64), (130, 128), (129, 256)])
@pytest.mark.parametrize("mask_kind", [inputs.MASK_NONE, inputs.MASK_CAUSAL, inputs.MASK_BLOCK_SPARSE])
def test_fp32_odd_shapes_all_masks(n, d, mask_kind):
    errs = H.run_case(1, 2, n, d, "f32", mask_kind, seed=21, block=32, cfg=simt_cfg())
    H.assert_within(errs, "f32")


@pytest.mark.parametrize("d", [64, 128, 256])
@pytest.mark.parametrize("mask_kind", [inputs.MASK_NONE, inputs.MASK_CAUSAL, inputs.MASK_BLOCK_SPARSE])
def test_bf16_storage_on_the_fp32_path(d, mask_kind):
    errs = H.run_case(2, 2, 320, d, "bf16", mask_kind, seed=22, block=128, cfg=simt_cfg())
    H.assert_within(errs, "bf16")


def test_explicit_scale_and_batches():
    errs = H.run_case(3, 2, 96, 40, "f32", inputs.MASK_CAUSAL, seed=23, scale=0.2, cfg=simt_cfg())
    H.assert_within(errs, "f32")


def test_per_head_block_masks_and_empty_rows():
    """mask_heads = batch*heads; one block row keeps nothing: O = 0, LSE = -inf, finite gradients."""
    import torch
    import paper_2410_09397_b200 as attn
    from oracle import oracle as orc
    b, h, n, d, block = 1, 3, 96, 32, 32
    nb = n // block
    bm = inputs.block_mask(31, nb, 0.5, heads=b * h)
    bm[1, 2, :] = 0
    errs = H.run_case(b, h, n, d, "f32", inputs.MASK_BLOCK_SPARSE, seed=24, block=block, bmask=bm, cfg=simt_cfg())
    H.assert_within(errs, "f32")
    x = H.make_inputs(24, b, h, n, d, "f32")
    mask = attn.Mask(kind=attn.ATTN_MASK_BLOCK_SPARSE, block=block, block_mask=torch.from_numpy(bm).cuda())
    O, LSE = attn.attn_fwd(*(H.to_dev(x[k], "f32") for k in "QKV"), mask=mask, cfg=simt_cfg())
    assert torch.all(O[0, 1, 64:96] == 0) and torch.all(torch.isneginf(LSE[0, 1, 64:96]))


def test_preprocess_D_matches_definition():
    import torch
    import paper_2410_09397_b200 as attn
    for dtype, rows, d in (("bf16", 1000, 128), ("bf16", 77, 64), ("bf16", 5, 256), ("f32", 300, 64), ("f32", 9, 24),
                           ("bf16", 33, 72)):
        O = inputs.normal_tensor(40, 0, (rows, d), bf16=dtype == "bf16")
        G = inputs.normal_tensor(40, 1, (rows, d), bf16=dtype == "bf16")
        D = attn.attn_bwd_preprocess(H.to_dev(O, dtype), H.to_dev(G, dtype))
        torch.cuda.synchronize()
        ref = (O.astype(np.float64) * G.astype(np.float64)).sum(-1)
        assert H.rel_err(H.to_np(D), ref) <= 1e-5


def test_runs_are_bitwise_repeatable():
    import torch
    import paper_2410_09397_b200 as attn
    x = H.make_inputs(25, 1, 2, 200, 64, "f32")
    dev = {k: H.to_dev(v, "f32") for k, v in x.items()}
    outs = []
    for _ in range(2):
        O, LSE = attn.attn_fwd(dev["Q"], dev["K"], dev["V"], cfg=simt_cfg())
        g = attn.attn_bwd(dev["Q"], dev["K"], dev["V"], O, dev["dO"], LSE, cfg=simt_cfg())
        torch.cuda.synchronize()
        outs.append([t.clone() for t in (O, LSE) + tuple(g)])
    for a, b in zip(*outs):
        assert torch.equal(a, b)


def test_missing_arch_or_bad_args_raise():
    import torch
    import paper_2410_09397_b200 as attn
    q = torch.zeros(1, 1, 16, 12, device="cuda")
    with pytest.raises(attn.AttnError) as e:
        attn.attn_fwd(q, q, q)
    assert e.value.status == attn.binding.ATTN_ERR_SHAPE

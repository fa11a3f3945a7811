"""GPU parity for element masks (any set of kept score entries, given as one bit per entry or as a coordinate
list: the sparse matrices of Section 4.1) on every algorithm that takes them: the fused kernels with 128- and
64-query tiles, the path without atomics and the fp32 FMA kernels.  The oracle's element mask is an explicit
n x n keep matrix."""
import numpy as np
import pytest

from paper_2410_09397_b200 import inputs
from tests import helpers as H

pytestmark = pytest.mark.gpu
EL = inputs.MASK_ELEMENT


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
@pytest.mark.parametrize("n,d,p", [(512, 128, 0.3), (600, 64, 0.05), (328, 128, 0.5), (392, 256, 0.2)])
def test_random_element_masks(which, n, d, p):
    """Random patterns (rows that keep nothing occur at the low density; n = 600, 328, 392 leave a ragged last
    tile and a last bitmap word that is only partly used)."""
    _skip(which, d)
    errs = H.run_case(1, 2, n, d, "bf16", EL, seed=91, keep_prob=p, cfg=cfgs()[which])
    H.assert_within(errs, "bf16")


@pytest.mark.parametrize("which", ["fused128", "no_atomics"])
def test_structured_element_masks_per_head(which):
    """Head 0: a causal band of width 100 (most 128 x 128 tiles keep nothing and are never visited); head 1: a
    single kept entry per row on a permutation plus one empty row and one empty column; head 2: everything."""
    n, b, h = 640, 1, 3
    keep = np.zeros((b * h, n, n), dtype=np.uint8)
    i, j = np.indices((n, n))
    keep[0] = ((j <= i) & (i - j < 100)).astype(np.uint8)
    perm = np.random.default_rng(5).permutation(n)
    keep[1, np.arange(n), perm] = 1
    keep[1, 77, :] = 0
    keep[1, :, perm[300]] = 0
    keep[2] = 1
    errs = H.run_case(b, h, n, 128, "bf16", EL, seed=92, bmask=keep, cfg=cfgs()[which])
    H.assert_within(errs, "bf16")


@pytest.mark.parametrize("n,d", [(96, 64), (200, 40)])
def test_element_mask_fp32_path(n, d):
    errs = H.run_case(1, 2, n, d, "f32", EL, seed=93, keep_prob=0.4)
    H.assert_within(errs, "f32")


def test_mask_from_coordinate_list_is_the_bitmap():
    """attn_mask_from_coo: bit-exact against the packed keep matrix (integer work), entries out of range and
    duplicates ignored, per-head lists; then one run through the kernels with the bitmap it built."""
    import torch
    import paper_2410_09397_b200 as attn
    from paper_2410_09397_b200 import binding as B
    n, heads = 300, 2
    keep = inputs.element_mask(94, n, 0.1, heads=heads)
    hh, ii, jj = np.nonzero(keep)
    order = np.random.default_rng(6).permutation(len(hh))
    hh, ii, jj = hh[order], ii[order], jj[order]
    # append duplicates and invalid coordinates
    hh = np.concatenate([hh, hh[:50], [0, 0, 5, -1]]); ii = np.concatenate([ii, ii[:50], [n, -1, 0, 0]])
    jj = np.concatenate([jj, jj[:50], [0, 3, 0, 0]])
    dev = lambda x: torch.from_numpy(x.astype(np.int32)).cuda()
    bitmap = attn.attn_mask_from_coo(dev(ii), dev(jj), dev(hh), n, heads)
    torch.cuda.synchronize()
    assert np.array_equal(bitmap.cpu().numpy(), inputs.pack_element_mask(keep))
    # heads = NULL: everything goes into mask 0; an empty list clears the bitmap
    b0 = attn.attn_mask_from_coo(dev(ii[:100]), dev(jj[:100]), None, n, 1)
    k0 = np.zeros((1, n, n), np.uint8); k0[0, ii[:100], jj[:100]] = 1
    assert np.array_equal(b0.cpu().numpy(), inputs.pack_element_mask(k0))
    empty = attn.attn_mask_from_coo(dev(ii[:0]), dev(jj[:0]), None, n, 1, bitmap=b0)
    assert int(empty.abs().sum()) == 0
    # the bitmap drives the kernels
    x = H.make_inputs(95, 1, heads, n + 4, 64, "bf16")   # n + 4 = 304, a multiple of 8
    n2 = n + 4
    keep2 = np.zeros((heads, n2, n2), np.uint8); keep2[:, :n, :n] = keep; keep2[:, n:, 0] = 1
    from oracle import oracle as orc
    O_ref, LSE_ref = orc.attn_fwd(x["Q"], x["K"], x["V"], mask_kind=orc.MASK_ELEMENT, mask_bits=keep2)
    h2, i2, j2 = np.nonzero(keep2)
    bm = attn.attn_mask_from_coo(dev(i2), dev(j2), dev(h2), n2, heads)
    d_ = {k: H.to_dev(v, "bf16") for k, v in x.items()}
    O, LSE = attn.attn_fwd(d_["Q"], d_["K"], d_["V"], mask=B.Mask(kind=B.ATTN_MASK_ELEMENT, block_mask=bm))
    torch.cuda.synchronize()
    assert H.rel_err(H.to_np(O), O_ref) <= 2e-2 and H.rel_err(H.to_np(LSE), LSE_ref) <= 2e-2


def test_element_mask_is_refused_where_it_is_not_built():
    import torch
    import paper_2410_09397_b200 as attn
    from paper_2410_09397_b200 import binding as B
    bm = torch.zeros(1, 256, 8, dtype=torch.int32, device="cuda")
    mask = attn.Mask(kind=attn.ATTN_MASK_ELEMENT, block_mask=bm)
    assert attn.attn_bwd_workspace_bytes(256, 256, 1, 1, mask, attn.ATTN_BF16, B.Cfg(algo=B.ATTN_ALGO_MATERIALIZED)) == 0
    assert attn.attn_bwd_workspace_bytes(256, 128, 1, 1, mask, attn.ATTN_BF16, None) > 0

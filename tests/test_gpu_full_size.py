"""Parity at the full benchmark sizes, in the launch configuration bench.py times.

The whole workload runs on the GPU; the float64 oracle recomputes a sample of
(batch, head) units -- heads are independent, so a sampled head is checked on every one
of its outputs (O, LSE, dQ, dK, dV).  Sampled heads carry the repository generator's
data; the other heads are filled with seeded device noise of the same distribution
(they are computed but not compared).
"""
import numpy as np
import pytest

from oracle import oracle as orc
from paper_2410_09397_b200 import inputs
from tests import helpers as H

pytestmark = pytest.mark.gpu


def run_full(name, sample_heads, cfg=None, backward=True, w=None, element_keep=None):
    """`w`: a variant of the named workload (other head count, block edge or mask kind); `element_keep`: run with the
    element mask given as a keep matrix [1][n][n] instead of the workload's own mask."""
    import torch
    import paper_2410_09397_b200 as attn
    w = w or inputs.WORKLOADS[name]
    BH = w.batch * w.heads
    tdt = torch.bfloat16 if w.bf16 else torch.float32
    gen = torch.Generator(device="cuda").manual_seed(1234 + w.seed)
    dev = {}
    for k in ("Q", "K", "V", "dO"):
        t = torch.randn((BH, w.n, w.d), generator=gen, device="cuda", dtype=torch.float32).to(tdt)
        dev[k] = t
    host = {}
    for h in sample_heads:
        host[h] = w.tensors(head_slice=(h, h + 1))
        for k in dev:
            dev[k][h].copy_(torch.from_numpy(host[h][k][0]).to(tdt))
    bmask = w.block_mask()
    mask = None
    mask_kind = w.mask
    if element_keep is not None:
        mask_kind, bmask = inputs.MASK_ELEMENT, element_keep
        mask = attn.Mask(kind=attn.ATTN_MASK_ELEMENT, block_mask=torch.from_numpy(inputs.pack_element_mask(element_keep)).cuda())
    elif w.mask != inputs.MASK_NONE:
        mask = attn.Mask(kind=w.mask, block=w.block, block_mask=torch.from_numpy(bmask).cuda() if bmask is not None else None)
    view = {k: v.view(w.batch, w.heads, w.n, w.d) for k, v in dev.items()}
    O, LSE = attn.attn_fwd(view["Q"], view["K"], view["V"], mask=mask, cfg=cfg)
    if backward:
        dQ, dK, dV = attn.attn_bwd(view["Q"], view["K"], view["V"], O, view["dO"], LSE, mask=mask, cfg=cfg)
    torch.cuda.synchronize()
    assert torch.isfinite(O.float()).all()
    mk = H.oracle_mask_kwargs(mask_kind, w.block, bmask)
    tol = H.TOL[w.dtype]
    for h in sample_heads:
        x = {k: v.astype(np.float64)[None] for k, v in host[h].items()}
        O_ref, LSE_ref = orc.attn_fwd(x["Q"], x["K"], x["V"], **mk)
        b, hh = divmod(h, w.heads)
        errs = {"O": H.rel_err(H.to_np(O[b, hh]), O_ref[0, 0]), "LSE": H.rel_err(H.to_np(LSE[b, hh]), LSE_ref[0, 0])}
        if backward:
            g = orc.attn_bwd(x["Q"], x["K"], x["V"], O_ref, x["dO"], LSE_ref, **mk)
            for nm, got, ref in zip(("dQ", "dK", "dV"), (dQ, dK, dV), g):
                errs[nm] = H.rel_err(H.to_np(got[b, hh]), ref[0, 0])
        bad = {k: v for k, v in errs.items() if not v <= tol}
        assert not bad, f"{name} head {h}: over tolerance {tol}: {bad} (all {errs})"


def test_config2_full():
    run_full("C2", [0, 21, 63])


def test_config3_full_headline():
    run_full("C3", [0, 31])


def test_config5_full_block_sparse():
    # one head from the first, a middle and the last launch group of the backward
    run_full("C5", [0, 17, 31])


def test_config5_shape_with_64_wide_blocks_and_with_the_causal_mask_on_top():
    """C5's sequence length (n = 32768, 8 heads) with the mask redrawn on 64 x 64 blocks, and with the 128 x 128
    block mask combined with the causal mask: one head each against the oracle."""
    base = inputs.WORKLOADS["C5"]
    w64 = inputs.Workload(**{**base.__dict__, "heads": 8, "block": 64})
    run_full("C5", [3], w=w64)
    wbc = inputs.Workload(**{**base.__dict__, "heads": 8, "mask": inputs.MASK_BLOCK_SPARSE_CAUSAL})
    run_full("C5", [6], w=wbc)


def test_config3_shape_with_an_element_mask():
    """The headline shape (n = 8192, d = 128, 4 heads) under an element mask: a causal band of 1000 keys plus 2 %
    of all other causal entries at random, so that tiles are empty, partly kept and full; one head against the oracle,
    on the fused path and on the path without atomics."""
    import paper_2410_09397_b200 as attn
    base = inputs.WORKLOADS["C3"]
    w = inputs.Workload(**{**base.__dict__, "batch": 1, "heads": 4, "mask": inputs.MASK_NONE})
    n = w.n
    i, j = np.indices((n, n), dtype=np.int32)
    keep = ((j <= i) & ((i - j < 1000) | (inputs.element_mask(7, n, 0.02)[0] != 0))).astype(np.uint8)[None]
    del i, j
    run_full("C3", [2], w=w, element_keep=keep)
    run_full("C3", [1], w=w, element_keep=keep, cfg=attn.Cfg(deterministic=1))


def test_config3_full_without_atomics():
    """The path without atomics (deterministic = 1) at the headline size, two heads against the oracle."""
    import paper_2410_09397_b200 as attn
    run_full("C3", [5, 26], cfg=attn.Cfg(deterministic=1))


def test_config3_every_head_fused_against_the_path_without_atomics():
    """The oracle can afford a few heads at this size; this covers the others: every head of dQ, dK, dV from
    the fused backward against the two-kernel path without atomics.  Both are oracle-checked on sampled heads
    above; they differ in kernels, loop order (dQ) and launch grouping, so a fault tied to a head index or a
    group boundary in either one shows up as a disagreement.  dK and dV have the same summation order in both
    paths: within two bf16 steps of the head's maximum; dQ is summed in a different order and rounded from
    different partial sums: within the bf16 tolerance."""
    import torch
    import paper_2410_09397_b200 as attn
    w = inputs.WORKLOADS["C3"]
    gen = torch.Generator(device="cuda").manual_seed(99)
    Q, K, V, dO = (torch.randn((w.batch, w.heads, w.n, w.d), generator=gen, device="cuda").to(torch.bfloat16) for _ in range(4))
    mask = attn.Mask(kind=w.mask)
    O, LSE = attn.attn_fwd(Q, K, V, mask=mask)
    a = attn.attn_bwd(Q, K, V, O, dO, LSE, mask=mask)
    b = attn.attn_bwd(Q, K, V, O, dO, LSE, mask=mask, cfg=attn.Cfg(deterministic=1))
    torch.cuda.synchronize()
    for name, x, y in zip(("dQ", "dK", "dV"), a, b):
        x, y = x.float(), y.float()
        assert torch.isfinite(x).all() and torch.isfinite(y).all()
        per_head = (x - y).abs().amax(dim=(2, 3)) / y.abs().amax(dim=(2, 3))
        assert float(per_head.max()) <= (H.TOL["bf16"] if name == "dQ" else 2 ** -7), (name, per_head)


@pytest.mark.parametrize("tile_q,tile_k", [(128, 128), (128, 64), (128, 32), (256, 128), (256, 32)])
def test_config4_full_small_cache_regime_tile_sweep(tile_q, tile_k):
    """d = 256: fused forward, materialised (small-cache) backward, block edges swept."""
    import paper_2410_09397_b200 as attn
    run_full("C4", [0, 7] if tile_k == 128 else [5],
             cfg=attn.Cfg(tile_q=tile_q, tile_k=tile_k, algo=attn.ATTN_ALGO_MATERIALIZED))


def test_config4_full_default_cfg():
    """d = 256 with the default configuration: fused forward and the fused backward with 64-query tiles."""
    run_full("C4", [0, 3, 7])

"""GPU parity on seeded random problems: sizes, head counts, masks and algorithms drawn at random, so that shapes
nobody wrote down by hand (odd numbers of tiles, tails of 8 to 120 rows, one-tile problems, single heads) go through
every tensor-core path against the oracle."""
import numpy as np
import pytest

from paper_2410_09397_b200 import inputs
from tests import helpers as H

pytestmark = pytest.mark.gpu


def draw(seed):
    from paper_2410_09397_b200 import binding as B
    rng = np.random.default_rng(1000 + seed)
    d = int(rng.choice([64, 128, 256]))
    n = int(rng.integers(1, 150)) * 8                      # 8 .. 1192
    b, h = int(rng.integers(1, 3)), int(rng.integers(1, 4))
    kind = int(rng.choice([inputs.MASK_NONE, inputs.MASK_CAUSAL, inputs.MASK_BLOCK_SPARSE, inputs.MASK_BLOCK_SPARSE_CAUSAL,
                           inputs.MASK_ELEMENT]))
    block = int(rng.choice([32, 64, 128, 256]))
    algos = ["fused"]
    if d != 256:
        algos.append("no_atomics")
    if d == 128:
        algos.append("fused64")
    if kind in (inputs.MASK_NONE, inputs.MASK_CAUSAL):
        algos.append("materialised")
    algo = str(rng.choice(algos))
    cfg = {"fused": B.Cfg(algo=B.ATTN_ALGO_FUSED), "no_atomics": B.Cfg(algo=B.ATTN_ALGO_FUSED, deterministic=1),
           "fused64": B.Cfg(tile_q=64, algo=B.ATTN_ALGO_FUSED),
           "materialised": B.Cfg(tile_q=int(rng.choice([128, 256])), tile_k=int(rng.choice([32, 64, 128])),
                                 algo=B.ATTN_ALGO_MATERIALIZED)}[algo]
    return dict(b=b, h=h, n=n, d=d, kind=kind, block=block, keep=float(rng.choice([0.1, 0.4, 0.8])), cfg=cfg, algo=algo)


@pytest.mark.parametrize("seed", range(32))
def test_random_problem(seed):
    c = draw(seed)
    bmask = None
    if inputs.is_block_mask(c["kind"]):
        bmask = inputs.block_mask(seed, (c["n"] + c["block"] - 1) // c["block"], c["keep"], heads=c["b"] * c["h"] if seed % 2 else 1)
    elif c["kind"] == inputs.MASK_ELEMENT:
        bmask = inputs.element_mask(seed, c["n"], c["keep"], heads=c["b"] * c["h"] if seed % 2 else 1)
    errs = H.run_case(c["b"], c["h"], c["n"], c["d"], "bf16", c["kind"], seed=200 + seed, block=c["block"], bmask=bmask,
                      cfg=c["cfg"], check_bwd_only=False)
    bad = {k: v for k, v in errs.items() if not v <= H.TOL["bf16"]}
    assert not bad, f"{c}: over tolerance: {bad} (all {errs})"

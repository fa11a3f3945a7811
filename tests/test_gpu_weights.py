"""GPU parity of the attention-weight entry points (S = A1 X, h = A3 Y of Appendix D phase 1;
dL/dX = A1^T p A2 of Definition 3.2 and dL/dY) against the float64 oracle, through the C ABI."""
import numpy as np
import pytest

from oracle import oracle as orc
from paper_2410_09397_b200 import inputs

from tests.helpers import TOL, rel_err, to_dev, to_np

pytestmark = pytest.mark.gpu


def weights(seed, tid, units, d, dtype):
    """d x d weights of standard deviation 1/sqrt(d): the projections of N(0, 1) rows are N(0, 1) again."""
    w = inputs.normal_tensor(seed, tid, (units, d, d), bf16=False).astype(np.float64) / np.sqrt(d)
    return inputs.round_to_bf16(w.astype(np.float32)) if dtype == "bf16" else w.astype(np.float32)


def units_of(wu, b, h):
    return {"one": 1, "heads": h, "all": b * h}[wu]


PROJ_CASES = [
    # b, h, n, d, dtype, weight sharing
    (1, 1, 128, 64, "f32", "one"),          # the smallest workload's shape
    (2, 3, 300, 64, "bf16", "heads"),       # several 128-row tiles and a ragged tail
    (2, 3, 300, 128, "bf16", "all"),
    (1, 2, 392, 256, "bf16", "one"),
    (1, 1, 8, 128, "bf16", "one"),          # a single partial tile
    (2, 2, 200, 40, "bf16", "heads"),       # head size without a tensor-core kernel
    (1, 2, 100, 24, "f32", "all"),
]


@pytest.mark.parametrize("b,h,n,d,dtype,wu", PROJ_CASES)
def test_project_matches_oracle(b, h, n, d, dtype, wu):
    import torch
    import paper_2410_09397_b200 as attn
    A = inputs.normal_tensor(31, 0, (b, h, n, d), bf16=dtype == "bf16")
    W = weights(31, 4, units_of(wu, b, h), d, dtype)
    ref = orc.project(A, W)
    ws = torch.zeros(256, dtype=torch.uint8, device="cuda")
    out = attn.attn_project(to_dev(A, dtype), to_dev(W, dtype), workspace=ws)
    torch.cuda.synchronize()
    assert attn.attn_workspace_status(ws) == attn.ATTN_OK
    assert rel_err(to_np(out), ref) <= TOL[dtype]


GRAD_CASES = [
    (1, 1, 128, 64, "f32", "one"),
    (2, 3, 300, 64, "bf16", "heads"),
    (2, 3, 300, 128, "bf16", "all"),
    (1, 2, 392, 256, "bf16", "one"),
    (1, 1, 8, 128, "bf16", "one"),
    (2, 3, 4096, 64, "bf16", "heads"),      # more tiles than SMs: CTAs run through several tiles and weights
    (2, 3, 4096, 128, "bf16", "all"),
    (2, 3, 4096, 128, "bf16", "one"),
    (2, 3, 2048, 256, "bf16", "heads"),
    (2, 2, 200, 40, "bf16", "heads"),
    (1, 2, 100, 24, "f32", "all"),
]


@pytest.mark.parametrize("b,h,n,d,dtype,wu", GRAD_CASES)
def test_weight_grad_matches_oracle(b, h, n, d, dtype, wu):
    import torch
    import paper_2410_09397_b200 as attn
    A = inputs.normal_tensor(32, 0, (b, h, n, d), bf16=dtype == "bf16")
    G = inputs.normal_tensor(32, 3, (b, h, n, d), bf16=dtype == "bf16")
    units = units_of(wu, b, h)
    ref = orc.weight_grad(A, G, units)
    ws = torch.zeros(256, dtype=torch.uint8, device="cuda")
    dA, dG = to_dev(A, dtype), to_dev(G, dtype)
    g = torch.full((units, d, d), 7.0, dtype=torch.float32, device="cuda")      # must be overwritten, not added to
    for _ in range(2):                                                         # and a second call gives the same
        attn.attn_weight_grad(dA, dG, units, g, workspace=ws)
        torch.cuda.synchronize()
        assert attn.attn_workspace_status(ws) == attn.ATTN_OK
        assert rel_err(to_np(g), ref) <= TOL[dtype]


E2E_CASES = [
    # b, h, n, d, dtype, sharing, mask
    (1, 1, 128, 64, "f32", "one", inputs.MASK_NONE),
    (2, 2, 300, 64, "bf16", "heads", inputs.MASK_CAUSAL),
    (2, 2, 392, 128, "bf16", "heads", inputs.MASK_NONE),
    (1, 2, 392, 128, "bf16", "all", inputs.MASK_CAUSAL),
    (1, 2, 264, 256, "bf16", "one", inputs.MASK_NONE),     # backward with 64-query tiles
]


@pytest.mark.parametrize("b,h,n,d,dtype,wu,mask_kind", E2E_CASES)
def test_weight_gradients_of_the_whole_path(b, h, n, d, dtype, wu, mask_kind):
    """A1, A2, A3, X, Y, dO in; gX, gY out: projections, forward, phase 2 all on the GPU, against the oracle
    run in float64 on the same (storage-rounded) inputs."""
    import torch
    import paper_2410_09397_b200 as attn
    from paper_2410_09397_b200 import binding as B
    bf = dtype == "bf16"
    A1, A2, A3, dO = (inputs.normal_tensor(33, t, (b, h, n, d), bf16=bf) for t in range(4))
    units = units_of(wu, b, h)
    X, Y = weights(33, 4, units, d, dtype), weights(33, 5, units, d, dtype)
    ref = orc.attn_weights_bwd(A1, A2, A3, X, Y, dO, mask_kind=mask_kind)

    dev = {k: to_dev(v, dtype) for k, v in dict(A1=A1, A2=A2, A3=A3, dO=dO, X=X, Y=Y).items()}
    mask = None if mask_kind == inputs.MASK_NONE else B.Mask(kind=mask_kind)
    S, hh = attn.attn_project(dev["A1"], dev["X"]), attn.attn_project(dev["A3"], dev["Y"])
    O, LSE = attn.attn_fwd(S, dev["A2"], hh, mask=mask)
    dt = B.ATTN_BF16 if bf else B.ATTN_F32
    ws = torch.zeros(B.attn_weights_bwd_workspace_bytes(n, d, h, b, mask, dt, None), dtype=torch.uint8, device="cuda")
    gX, gY = attn.attn_weights_bwd(dev["A1"], dev["A2"], dev["A3"], S, hh, O, dev["dO"], LSE, units, mask=mask,
                                   workspace=ws)
    torch.cuda.synchronize()
    assert attn.attn_workspace_status(ws) == attn.ATTN_OK
    errs = {"S": rel_err(to_np(S), ref["S"]), "h": rel_err(to_np(hh), ref["h"]), "O": rel_err(to_np(O), ref["O"]),
            "gX": rel_err(to_np(gX), ref["gX"]), "gY": rel_err(to_np(gY), ref["gY"])}
    assert all(v <= TOL[dtype] for v in errs.values()), errs
    # Y fixed, as in the paper's statement: only gX is produced
    gX2, none = attn.attn_weights_bwd(dev["A1"], dev["A2"], None, S, hh, O, dev["dO"], LSE, units, want_gY=False,
                                      mask=mask, workspace=ws)
    torch.cuda.synchronize()
    assert none is None and rel_err(to_np(gX2), ref["gX"]) <= TOL[dtype]


def test_weight_kernels_at_headline_size_on_sampled_units():
    """batch 2 x 16 heads, n = 8192, d = 128, bf16: the launch shape the benchmark times; the oracle checks
    two sampled units of the projection and of the per-unit weight gradient."""
    import torch
    import paper_2410_09397_b200 as attn
    w = inputs.WORKLOADS["C3"]
    b, h, n, d = w.batch, w.heads, w.n, w.d
    sample = [3, 29]
    gen = torch.Generator(device="cuda").manual_seed(5)
    A = torch.randn((b, h, n, d), generator=gen, device="cuda").to(torch.bfloat16)
    G = torch.randn((b, h, n, d), generator=gen, device="cuda").to(torch.bfloat16)
    for u in sample:      # the sampled units get the repository's own seeded values
        bi, hi = divmod(u, h)
        A[bi, hi] = to_dev(inputs.normal_tensor(34, 0, (n, d), bf16=True), "bf16")
        G[bi, hi] = to_dev(inputs.normal_tensor(34 + u, 3, (n, d), bf16=True), "bf16")
    W = to_dev(weights(34, 4, h, d, "bf16"), "bf16")
    ws = torch.zeros(256, dtype=torch.uint8, device="cuda")
    out = attn.attn_project(A, W, workspace=ws)
    g = attn.attn_weight_grad(A, G, b * h, workspace=ws)
    torch.cuda.synchronize()
    assert attn.attn_workspace_status(ws) == attn.ATTN_OK
    for u in sample:
        bi, hi = divmod(u, h)
        a, gg = to_np(A[bi, hi])[None, None], to_np(G[bi, hi])[None, None]
        assert rel_err(to_np(out[bi, hi]), orc.project(a, to_np(W[hi])[None])[0, 0]) <= TOL["bf16"]
        assert rel_err(to_np(g[u]), orc.weight_grad(a, gg, 1)[0]) <= TOL["bf16"]


def test_weight_gradients_through_a_block_sparse_mask():
    """The whole path with the 128 x 128 block mask of the sparse workload's kind (diagonal kept, others with
    probability 0.3), one weight per head, against the oracle."""
    import torch
    import paper_2410_09397_b200 as attn
    from paper_2410_09397_b200 import binding as B
    b, h, n, d, block = 1, 2, 640, 128, 128
    A1, A2, A3, dO = (inputs.normal_tensor(35, t, (b, h, n, d), bf16=True) for t in range(4))
    X, Y = weights(35, 4, h, d, "bf16"), weights(35, 5, h, d, "bf16")
    bm = inputs.block_mask(36, n // block, 0.3)
    ref = orc.attn_weights_bwd(A1, A2, A3, X, Y, dO, mask_kind=orc.MASK_BLOCK, block=block, mask_bits=bm)
    dev = {k: to_dev(v, "bf16") for k, v in dict(A1=A1, A2=A2, A3=A3, dO=dO, X=X, Y=Y).items()}
    mask = B.Mask(kind=inputs.MASK_BLOCK_SPARSE, block=block, block_mask=torch.from_numpy(bm).cuda())
    S, hh = attn.attn_project(dev["A1"], dev["X"]), attn.attn_project(dev["A3"], dev["Y"])
    O, LSE = attn.attn_fwd(S, dev["A2"], hh, mask=mask)
    ws = torch.zeros(B.attn_weights_bwd_workspace_bytes(n, d, h, b, mask, B.ATTN_BF16, None), dtype=torch.uint8,
                     device="cuda")
    gX, gY = attn.attn_weights_bwd(dev["A1"], dev["A2"], dev["A3"], S, hh, O, dev["dO"], LSE, h, mask=mask, workspace=ws)
    torch.cuda.synchronize()
    assert attn.attn_workspace_status(ws) == attn.ATTN_OK
    assert rel_err(to_np(gX), ref["gX"]) <= TOL["bf16"] and rel_err(to_np(gY), ref["gY"]) <= TOL["bf16"]


ALGO_CASES = [
    # d, n, configuration of the attention backward inside attn_weights_bwd
    (128, 392, dict()),                                   # fused, 128-query tiles: gX read from the fp32 dQ accumulator
    (64, 300, dict()),
    (128, 392, dict(algo="fused", tile_q=64)),            # fused, 64-query tiles: the accumulator as well
    (128, 392, dict(deterministic=1)),                    # no accumulator: gX from the stored dQ
    (64, 300, dict(deterministic=1)),
    (128, 264, dict(algo="materialized")),
    (256, 264, dict()),                                   # 64-query tiles with the head dimension split: accumulator too
]


@pytest.mark.parametrize("d,n,cfg_kw", ALGO_CASES)
def test_weight_gradients_for_every_backward_algorithm(d, n, cfg_kw):
    """gX and gY through attn_weights_bwd with each algorithm of the attention backward (causal mask, one weight
    per head, a ragged last tile), against the oracle; where dQ is accumulated in fp32 the result must also agree
    with the product formed from the stored bf16 dQ of attn_bwd to within the storage rounding."""
    import torch
    import paper_2410_09397_b200 as attn
    from paper_2410_09397_b200 import binding as B
    b, h = 2, 2
    A1, A2, A3, dO = (inputs.normal_tensor(41, t, (b, h, n, d), bf16=True) for t in range(4))
    X, Y = weights(41, 4, h, d, "bf16"), weights(41, 5, h, d, "bf16")
    ref = orc.attn_weights_bwd(A1, A2, A3, X, Y, dO, mask_kind=inputs.MASK_CAUSAL)
    dev = {k: to_dev(v, "bf16") for k, v in dict(A1=A1, A2=A2, A3=A3, dO=dO, X=X, Y=Y).items()}
    mask = B.Mask(kind=inputs.MASK_CAUSAL)
    kw = dict(cfg_kw)
    if "algo" in kw:
        kw["algo"] = {"fused": B.ATTN_ALGO_FUSED, "materialized": B.ATTN_ALGO_MATERIALIZED}[kw["algo"]]
    cfg = B.Cfg(**kw) if kw else None
    S, hh = attn.attn_project(dev["A1"], dev["X"]), attn.attn_project(dev["A3"], dev["Y"])
    O, LSE = attn.attn_fwd(S, dev["A2"], hh, mask=mask)
    ws = torch.zeros(B.attn_weights_bwd_workspace_bytes(n, d, h, b, mask, B.ATTN_BF16, cfg), dtype=torch.uint8,
                     device="cuda")
    for _ in range(2):      # the second call finds the workspace as the first left it
        gX, gY = attn.attn_weights_bwd(dev["A1"], dev["A2"], dev["A3"], S, hh, O, dev["dO"], LSE, h, mask=mask, cfg=cfg,
                                       workspace=ws)
        torch.cuda.synchronize()
        assert attn.attn_workspace_status(ws) == attn.ATTN_OK
        errs = {"gX": rel_err(to_np(gX), ref["gX"]), "gY": rel_err(to_np(gY), ref["gY"])}
        assert all(v <= TOL["bf16"] for v in errs.values()), errs
    dQ, dK, dV = attn.attn_bwd(S, dev["A2"], hh, O, dev["dO"], LSE, mask=mask, cfg=cfg)
    g2 = attn.attn_weight_grad(dev["A1"], dQ, h)
    torch.cuda.synchronize()
    assert rel_err(to_np(gX), to_np(g2)) <= 1e-2


def test_weights_bwd_at_headline_size_on_sampled_units():
    """attn_weights_bwd on the launch shape the benchmark times (batch 2 x 16 heads, n = 8192, d = 128, causal, one
    weight per unit so that every unit's gradient can be read on its own, S = A1 and h = A3 as in the benchmark):
    for two sampled units the oracle's attention backward followed by its weight-gradient product gives gX and gY."""
    import torch
    import paper_2410_09397_b200 as attn
    from paper_2410_09397_b200 import binding as B
    w = inputs.WORKLOADS["C3"]
    b, h, n, d = w.batch, w.heads, w.n, w.d
    sample = [5, 30]
    gen = torch.Generator(device="cuda").manual_seed(77)
    dev = {k: torch.randn((b * h, n, d), generator=gen, device="cuda").to(torch.bfloat16) for k in ("Q", "K", "V", "dO")}
    host = {}
    for u in sample:
        host[u] = w.tensors(head_slice=(u, u + 1))
        for k in dev:
            dev[k][u].copy_(torch.from_numpy(host[u][k][0]).to(torch.bfloat16))
    view = {k: v.view(b, h, n, d) for k, v in dev.items()}
    mask = B.Mask(kind=inputs.MASK_CAUSAL)
    O, LSE = attn.attn_fwd(view["Q"], view["K"], view["V"], mask=mask)
    ws = torch.zeros(B.attn_weights_bwd_workspace_bytes(n, d, h, b, mask, B.ATTN_BF16, None), dtype=torch.uint8,
                     device="cuda")
    gX, gY = attn.attn_weights_bwd(view["Q"], view["K"], view["V"], view["Q"], view["V"], O, view["dO"], LSE, b * h,
                                   mask=mask, workspace=ws)
    torch.cuda.synchronize()
    assert attn.attn_workspace_status(ws) == attn.ATTN_OK
    for u in sample:
        x = {k: v.astype(np.float64)[None] for k, v in host[u].items()}
        O_ref, LSE_ref = orc.attn_fwd(x["Q"], x["K"], x["V"], mask_kind=orc.MASK_CAUSAL)
        dQ, dK, dV = orc.attn_bwd(x["Q"], x["K"], x["V"], O_ref, x["dO"], LSE_ref, mask_kind=orc.MASK_CAUSAL)
        errs = {"gX": rel_err(to_np(gX[u]), orc.weight_grad(x["Q"], dQ, 1)[0]),
                "gY": rel_err(to_np(gY[u]), orc.weight_grad(x["V"], dV, 1)[0])}
        assert all(v <= TOL["bf16"] for v in errs.values()), (u, errs)

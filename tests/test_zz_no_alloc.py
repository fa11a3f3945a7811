"""attn_bwd_noalloc: the backward for callers that cannot allocate device memory.

Some users of the library are handed tensors but may not call cudaMalloc at that point
(a frozen memory pool, a real-time loop, a plug-in without an allocator), so they cannot
supply attn_bwd's workspace.  The entry point tested here keeps its scratch in a fixed
8 MiB array inside the library instead.  It must give the same dQ, dK, dV as attn_bwd
(which the parity tests check against the float64 oracle on these shapes and larger ones),
also on a second call (the array keeps the first call's contents), and must refuse
problems that do not fit.  This file sorts last on purpose: a run that stops at the
first failure has then already run every other test.
"""
import pytest

from paper_2410_09397_b200 import inputs
from tests import helpers as H

pytestmark = pytest.mark.gpu


@pytest.mark.parametrize("dtype,algo_name", [("bf16", "fused"), ("f32", "simt")])
def test_noalloc_matches_attn_bwd_twice(dtype, algo_name):
    import torch
    import paper_2410_09397_b200 as attn
    algo = attn.ATTN_ALGO_FUSED if algo_name == "fused" else attn.ATTN_ALGO_SIMT
    cfg = attn.Cfg(algo=algo)
    b, h, n, d = 1, 2, 384, 128
    mask = attn.Mask(kind=attn.ATTN_MASK_CAUSAL)
    tol = H.TOL[dtype]
    for call, seed in enumerate((41, 42)):          # two calls in a row, different data
        x = H.make_inputs(seed, b, h, n, d, dtype)
        dev = {k: H.to_dev(v, dtype) for k, v in x.items()}
        O, LSE = attn.attn_fwd(dev["Q"], dev["K"], dev["V"], mask=mask, cfg=cfg)
        ref = attn.attn_bwd(dev["Q"], dev["K"], dev["V"], O, dev["dO"], LSE, mask=mask, cfg=cfg)
        out = tuple(torch.full_like(dev["Q"], float("nan")) for _ in range(3))
        attn.attn_bwd_noalloc(dev["Q"], dev["K"], dev["V"], O, dev["dO"], LSE, *out, mask=mask, cfg=cfg)
        assert attn.attn_noalloc_status() == attn.ATTN_OK     # synchronises; no bounded wait ran out
        for name, got, want in zip(("dQ", "dK", "dV"), out, ref):
            err = H.rel_err(H.to_np(got), H.to_np(want))
            assert err <= tol, (call, name, err)


def test_noalloc_rejects_problems_beyond_its_scratch():
    import torch
    import paper_2410_09397_b200 as attn
    assert attn.attn_noalloc_scratch_bytes() == 8 << 20
    b, h, n, d = 1, 8, 4096, 128          # fused workspace: 16 MiB accumulator > 8 MiB
    cfg = attn.Cfg(algo=attn.ATTN_ALGO_FUSED)
    assert attn.attn_bwd_workspace_bytes(n, d, h, b, None, attn.ATTN_BF16, cfg) > attn.attn_noalloc_scratch_bytes()
    t = torch.zeros(b, h, n, d, dtype=torch.bfloat16, device="cuda")
    lse = torch.zeros(b, h, n, dtype=torch.float32, device="cuda")
    with pytest.raises(attn.AttnError) as e:
        attn.attn_bwd_noalloc(t, t, t, t, t, lse, torch.empty_like(t), torch.empty_like(t), torch.empty_like(t), cfg=cfg)
    assert e.value.status == attn.binding.ATTN_ERR_WORKSPACE

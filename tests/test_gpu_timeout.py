"""The bounded waits of the tensor-core kernels, made to run out on purpose -- safely.

Every mbarrier wait in the library polls under a time limit; when it runs out the CTA sets
the workspace status word and the kernel still runs to its normal end.  The self-test
entry point launches one warp that waits a few milliseconds on a barrier nothing arrives
at.  Nothing faults and nothing hangs: the wait ends by itself, the status says
ATTN_ERR_DEVICE_TIMEOUT, and the next ordinary call on the same context is clean.
"""
import pytest

from paper_2410_09397_b200 import inputs
from tests import helpers as H

pytestmark = pytest.mark.gpu


def test_wait_that_runs_out_sets_the_status_and_leaves_the_context_usable():
    import torch
    import paper_2410_09397_b200 as attn
    from paper_2410_09397_b200 import binding as B
    ws = torch.zeros(256, dtype=torch.uint8, device="cuda")
    assert attn.attn_workspace_status(ws) == B.ATTN_OK
    attn.attn_selftest_wait_timeout(ws, limit_us=3000)
    assert attn.attn_workspace_status(ws) == B.ATTN_ERR_DEVICE_TIMEOUT
    words = ws.view(torch.int32)[:2].cpu().tolist()
    assert words[0] == B.ATTN_ERR_DEVICE_TIMEOUT
    assert words[1] == 0, "a wait on a barrier nobody arrives at reported success"
    # the context is as usable as before: an ordinary forward + backward, checked against the oracle
    errs = H.run_case(1, 2, 256, 128, "bf16", inputs.MASK_CAUSAL, seed=5)
    H.assert_within(errs, "bf16")


def test_selftest_rejects_bad_arguments_before_any_launch():
    import torch
    import paper_2410_09397_b200 as attn
    from paper_2410_09397_b200 import binding as B
    ws = torch.zeros(256, dtype=torch.uint8, device="cuda")
    for bad in (0, 200000):
        with pytest.raises(attn.AttnError) as e:
            attn.attn_selftest_wait_timeout(ws, limit_us=bad)
        assert e.value.status == B.ATTN_ERR_WORKSPACE
    assert attn.attn_workspace_status(ws) == B.ATTN_OK

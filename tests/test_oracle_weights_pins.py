"""Pins for the oracle's attention-weight functions (S = A1 X, h = A3 Y of Appendix D phase 1;
dL/dX = A1^T p A2 of Definition 3.2; dL/dY): checked against library products, against the
dense form written with the n x n matrix p, and against central differences of the loss in
the weights themselves.  Nothing here touches the CUDA path.
"""
import numpy as np
import pytest

from oracle import oracle as orc
from paper_2410_09397_b200 import inputs


def rnd(seed, tid, *shape):
    return inputs.normal_tensor(seed, tid, shape, bf16=False).astype(np.float64)


@pytest.mark.parametrize("wu", ["one", "heads", "all"])
def test_project_is_the_plain_product(wu):
    """A transposed weight (A W^T), a wrong unit-to-weight map or a dropped term fails here."""
    b, h, n, d = 2, 3, 5, 4
    A = rnd(21, 0, b, h, n, d)
    W = rnd(21, 1, {"one": 1, "heads": h, "all": b * h}[wu], d, d)
    out = orc.project(A, W)
    for bi in range(b):
        for hi in range(h):
            w = W[{"one": 0, "heads": hi, "all": bi * h + hi}[wu]]
            np.testing.assert_allclose(out[bi, hi], A[bi, hi] @ w, rtol=1e-13, atol=1e-14)
    # a non-symmetric weight tells A W from A W^T
    assert np.abs(out[0, 0] - A[0, 0] @ W[0].T).max() > 1e-3


@pytest.mark.parametrize("wu", ["one", "heads", "all"])
def test_weight_grad_is_A_transpose_G_summed_over_sharing_units(wu):
    b, h, n, d = 2, 3, 6, 4
    A, G = rnd(22, 0, b, h, n, d), rnd(22, 1, b, h, n, d)
    units = {"one": 1, "heads": h, "all": b * h}[wu]
    g = orc.weight_grad(A, G, units)
    ref = np.zeros((units, d, d))
    for bi in range(b):
        for hi in range(h):
            ref[{"one": 0, "heads": hi, "all": bi * h + hi}[wu]] += np.einsum("ia,ib->ab", A[bi, hi], G[bi, hi])
    np.testing.assert_allclose(g, ref, rtol=1e-13, atol=1e-13)
    assert np.abs(g[0] - g[0].T).max() > 1e-3          # A^T G, not G^T A


def test_gradient_in_X_equals_dense_form_of_the_definition():
    """Definition 3.2 literally: A1^T p A2 with the n x n matrix p of the no-cache algorithm."""
    n, d = 9, 4
    A1, A2, A3, G = (rnd(23, t, 1, 1, n, d) for t in range(4))
    X, Y = rnd(23, 4, 1, d, d) * 0.4, rnd(23, 5, 1, d, d) * 0.5
    r = orc.attn_weights_bwd(A1, A2, A3, X, Y, G, scale=1.0)
    p = orc.attn_dense(r["S"][0, 0], A2[0, 0], r["h"][0, 0], G[0, 0], scale=1.0)["p"]
    np.testing.assert_allclose(r["gX"][0], A1[0, 0].T @ p @ A2[0, 0], rtol=1e-11, atol=1e-13)
    f = orc.attn_dense(r["S"][0, 0], A2[0, 0], r["h"][0, 0], G[0, 0], scale=1.0)["f"]
    np.testing.assert_allclose(r["gY"][0], A3[0, 0].T @ f.T @ G[0, 0], rtol=1e-11, atol=1e-13)


@pytest.mark.parametrize("mask_kind", [orc.MASK_NONE, orc.MASK_CAUSAL])
@pytest.mark.parametrize("wu", ["heads", "all"])
def test_weight_gradients_match_central_differences(mask_kind, wu):
    """L = sum(O o G) as a function of X and Y, with the projections done by numpy: the finite
    differences know nothing of the oracle's project / weight_grad, so a wrong sign, a missing
    scale, a transposed product or gradients not added over the batch all fail."""
    b, h, n, d = 2, 2, 6, 3
    A1, A2, A3, G = (rnd(24, t, b, h, n, d) for t in range(4))
    units = h if wu == "heads" else b * h
    X, Y = rnd(24, 4, units, d, d) * 0.5, rnd(24, 5, units, d, d) * 0.5
    scale = 0.7

    def widx(bi, hi):
        return hi if wu == "heads" else bi * h + hi

    def L(Xm, Ym):
        S = np.stack([np.stack([A1[bi, hi] @ Xm[widx(bi, hi)] for hi in range(h)]) for bi in range(b)])
        hh = np.stack([np.stack([A3[bi, hi] @ Ym[widx(bi, hi)] for hi in range(h)]) for bi in range(b)])
        O, _ = orc.attn_fwd(S, A2, hh, mask_kind=mask_kind, scale=scale)
        return float((O * G).sum())

    r = orc.attn_weights_bwd(A1, A2, A3, X, Y, G, mask_kind=mask_kind, scale=scale)
    eps = 1e-5
    for name, W, g in (("X", X, r["gX"]), ("Y", Y, r["gY"])):
        num = np.zeros_like(W)
        for idx in np.ndindex(*W.shape):
            Wp, Wm = W.copy(), W.copy()
            Wp[idx] += eps
            Wm[idx] -= eps
            num[idx] = (L(Wp, Y) - L(Wm, Y)) / (2 * eps) if name == "X" else (L(X, Wp) - L(X, Wm)) / (2 * eps)
        assert np.abs(num - g).max() <= 2e-8 * max(1.0, np.abs(num).max()), name


def test_identity_weights_reduce_to_plain_attention():
    """X = Y = I: S = A1, h = A3 and the weight gradients are A1^T dQ and A3^T dV of the plain path."""
    b, h, n, d = 1, 2, 7, 4
    A1, A2, A3, G = (rnd(25, t, b, h, n, d) for t in range(4))
    I = np.eye(d)[None]
    r = orc.attn_weights_bwd(A1, A2, A3, I, I, G)
    O, LSE = orc.attn_fwd(A1, A2, A3)
    dQ, dK, dV = orc.attn_bwd(A1, A2, A3, O, G, LSE)
    np.testing.assert_allclose(r["O"], O, rtol=1e-13, atol=1e-14)
    np.testing.assert_allclose(r["gX"][0], sum(A1[0, k].T @ dQ[0, k] for k in range(h)), rtol=1e-12, atol=1e-13)
    np.testing.assert_allclose(r["gY"][0], sum(A3[0, k].T @ dV[0, k] for k in range(h)), rtol=1e-12, atol=1e-13)

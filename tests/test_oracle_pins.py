"""Pins for the float64 CPU oracle: everything here checks ``oracle/`` against facts
fixed by the paper or by mathematics, never against the CUDA path.

Each test names the plausible mistake it would catch.
"""
import itertools
import math

import numpy as np
import pytest

from oracle import oracle as orc
from paper_2410_09397_b200 import inputs


def rnd(seed, *shape):
    return inputs.normal_tensor(seed, 0, shape, bf16=False).astype(np.float64)


def make(seed, n, d, b=1, h=1):
    return tuple(inputs.normal_tensor(seed, t, (b, h, n, d), bf16=False).astype(np.float64) for t in range(4))


def masks_for(n, block=2, seed=11):
    nb = (n + block - 1) // block
    bm = inputs.block_mask(seed, nb, 0.4)
    return [
        dict(mask_kind=orc.MASK_NONE),
        dict(mask_kind=orc.MASK_CAUSAL),
        dict(mask_kind=orc.MASK_BLOCK, block=block, mask_bits=bm),
        # block mask AND causal; the diagonal blocks are kept so that every row keeps its own key
        dict(mask_kind=orc.MASK_BLOCK_CAUSAL, block=block, mask_bits=bm | np.eye(nb, dtype=bm.dtype)[None]),
    ]


def loss(Q, K, V, G, **mk):
    O, _ = orc.attn_fwd(Q, K, V, **mk)
    return float((O * G).sum())


# ---------------------------------------------------------------- finite differences

@pytest.mark.parametrize("n,d", [(1, 1), (2, 4), (5, 8), (8, 4), (16, 8)])
def test_gradients_match_central_differences(n, d):
    """dQ, dK, dV are the derivatives of L = sum(O o G) (wrong sign, dropped scale,
    transposed operand or a missing -D term all fail here)."""
    Q, K, V, G = make(3, n, d)
    for mk in masks_for(n):
        O, LSE = orc.attn_fwd(Q, K, V, **mk)
        dQ, dK, dV = orc.attn_bwd(Q, K, V, O, G, LSE, **mk)
        h = 1e-5
        for name, X, dX in (("Q", Q, dQ), ("K", K, dK), ("V", V, dV)):
            num = np.zeros_like(X)
            for idx in itertools.product(*(range(s) for s in X.shape)):
                old = X[idx]
                X[idx] = old + h
                lp = loss(Q, K, V, G, **mk)
                X[idx] = old - h
                lm = loss(Q, K, V, G, **mk)
                X[idx] = old
                num[idx] = (lp - lm) / (2 * h)
            scale_ = max(np.abs(num).max(), 1e-30)
            assert np.abs(num - dX).max() <= 2e-8 * max(scale_, 1.0), (name, mk["mask_kind"])


def test_weight_gradient_of_the_paper():
    """Definition 3.2: dL/dX = A1^T p(X) A2.  With Q = A1 X, K = A2 and scale = 1 (the
    paper folds the scale into X) this is A1^T dQ; checked by differences in X."""
    n, d = 7, 3
    A1, A2, V, G = (a[0, 0] for a in make(5, n, d))
    X = rnd(9, d, d) * 0.3

    def L(Xm):
        O, _ = orc.attn_fwd((A1 @ Xm)[None, None], A2[None, None], V[None, None], scale=1.0)
        return float((O[0, 0] * G).sum())

    Q = A1 @ X
    O, LSE = orc.attn_fwd(Q[None, None], A2[None, None], V[None, None], scale=1.0)
    dQ, _, _ = orc.attn_bwd(Q[None, None], A2[None, None], V[None, None], O, G[None, None], LSE, scale=1.0)
    g = A1.T @ dQ[0, 0]
    # the same gradient through the dense intermediates: A1^T p A2
    p = orc.attn_dense(Q, A2, V, G, scale=1.0)["p"]
    np.testing.assert_allclose(A1.T @ p @ A2, g, rtol=1e-11, atol=1e-13)
    h = 1e-5
    for a in range(d):
        for b in range(d):
            Xp, Xm = X.copy(), X.copy()
            Xp[a, b] += h
            Xm[a, b] -= h
            assert abs((L(Xp) - L(Xm)) / (2 * h) - g[a, b]) < 2e-8


# ---------------------------------------------------------------- closed forms, invariants

def ref_forward_numpy(Q, K, V, keep, scale):
    """Textbook softmax attention with numpy library routines (one head)."""
    S = scale * (Q @ K.T)
    S = np.where(keep, S, -np.inf)
    m = S.max(axis=1, keepdims=True)
    E = np.exp(S - m)
    l = E.sum(axis=1, keepdims=True)
    P = E / l
    return P, P @ V, (m + np.log(l))[:, 0]


def keep_matrix(n, mk):
    kind = mk["mask_kind"]
    if kind == orc.MASK_NONE:
        return np.ones((n, n), bool)
    if kind == orc.MASK_CAUSAL:
        return np.tril(np.ones((n, n), bool))
    blk = mk["block"]
    keep = np.kron(mk["mask_bits"][0].astype(bool), np.ones((blk, blk), bool))[:n, :n]
    return keep & np.tril(np.ones((n, n), bool)) if kind == orc.MASK_BLOCK_CAUSAL else keep


@pytest.mark.parametrize("n,d", [(6, 4), (12, 8), (33, 16)])
def test_forward_and_dV_against_library_routines(n, d):
    """O and LSE against numpy's matmul/exp/log; dV against the closed form P^T dO by
    an independent triple loop (catches a transposed P or a wrong normaliser)."""
    Q, K, V, G = make(4, n, d)
    for mk in masks_for(n, block=3):
        keep = keep_matrix(n, mk)
        P, O_ref, LSE_ref = ref_forward_numpy(Q[0, 0], K[0, 0], V[0, 0], keep, 1 / math.sqrt(d))
        O, LSE = orc.attn_fwd(Q, K, V, **mk)
        np.testing.assert_allclose(O[0, 0], O_ref, rtol=1e-12, atol=1e-14)
        np.testing.assert_allclose(LSE[0, 0], LSE_ref, rtol=1e-13, atol=1e-14)
        _, _, dV = orc.attn_bwd(Q, K, V, O, G, LSE, **mk)
        dV_ref = np.zeros((n, d))
        for j in range(n):
            for c in range(d):
                for i in range(n):
                    dV_ref[j, c] += P[i, j] * G[0, 0, i, c]
        np.testing.assert_allclose(dV[0, 0], dV_ref, rtol=1e-12, atol=1e-14)


def test_gradients_against_torch_autograd_float64():
    """A library's reverse-mode derivative of the textbook formula (float64)."""
    torch = pytest.importorskip("torch")
    n, d = 24, 8
    Q, K, V, G = make(6, n, d, b=2, h=2)
    for mk in masks_for(n, block=4):
        keep = torch.from_numpy(keep_matrix(n, mk))
        q, k, v = (torch.tensor(a, dtype=torch.float64, requires_grad=True) for a in (Q, K, V))
        s = (q @ k.transpose(-1, -2)) / math.sqrt(d)
        s = s.masked_fill(~keep, float("-inf"))
        o = torch.softmax(s, dim=-1) @ v
        (o * torch.from_numpy(G)).sum().backward()
        O, LSE = orc.attn_fwd(Q, K, V, **mk)
        np.testing.assert_allclose(O, o.detach().numpy(), rtol=1e-12, atol=1e-14)
        np.testing.assert_allclose(LSE, torch.logsumexp(s, -1).detach().numpy(), rtol=1e-13)
        dQ, dK, dV = orc.attn_bwd(Q, K, V, O, G, LSE, **mk)
        for mine, theirs in ((dQ, q.grad), (dK, k.grad), (dV, v.grad)):
            np.testing.assert_allclose(mine, theirs.numpy(), rtol=1e-10, atol=1e-13)


def test_element_mask_against_autograd_and_central_differences():
    """An arbitrary set of kept entries, a different one per head, with a row and a column that keep nothing
    (the coordinate-list sparsity of Section 4.1 as an explicit keep matrix): the textbook formula with the
    dropped scores at minus infinity, differentiated by a library in float64, and central differences of
    L = sum(O o G) (an index swap between rows and columns of the mask, or between the heads' masks, fails)."""
    torch = pytest.importorskip("torch")
    n, d = 11, 5
    Q, K, V, G = make(16, n, d, b=1, h=2)
    keep = inputs.element_mask(17, n, 0.45, heads=2)
    keep[0, 3, :] = 0
    keep[1, :, 6] = 0
    keep[1, 0, 0] = 1
    mk = dict(mask_kind=orc.MASK_ELEMENT, mask_bits=keep)
    O, LSE = orc.attn_fwd(Q, K, V, **mk)
    dQ, dK, dV = orc.attn_bwd(Q, K, V, O, G, LSE, **mk)
    q, k, v = (torch.tensor(a, dtype=torch.float64, requires_grad=True) for a in (Q, K, V))
    s = (q @ k.transpose(-1, -2)) / math.sqrt(d)
    s = s.masked_fill(~torch.from_numpy(keep.astype(bool))[None], float("-inf"))
    pr = torch.nan_to_num(torch.softmax(s, dim=-1), nan=0.0)       # a row that keeps nothing: all zeros
    o = pr @ v
    (o * torch.from_numpy(G)).sum().backward()
    np.testing.assert_allclose(O, o.detach().numpy(), rtol=1e-12, atol=1e-14)
    assert np.all(O[0, 0, 3] == 0) and LSE[0, 0, 3] == -np.inf
    np.testing.assert_allclose(dV, v.grad.numpy(), rtol=1e-10, atol=1e-13)
    assert np.all(dV[0, 1, 6] == 0) and np.all(dK[0, 1, 6] == 0)
    h = 1e-5
    rng = np.random.default_rng(18)
    for name, X, g in (("Q", Q, dQ), ("K", K, dK), ("V", V, dV)):
        for _ in range(12):
            idx = tuple(int(rng.integers(0, sz)) for sz in X.shape)
            old = X[idx]
            X[idx] = old + h; lp = loss(Q, K, V, G, **mk)
            X[idx] = old - h; lm = loss(Q, K, V, G, **mk)
            X[idx] = old
            assert abs((lp - lm) / (2 * h) - g[idx]) <= 1e-7 * max(1.0, abs(g[idx])), (name, idx)


def test_dense_intermediates_invariants():
    """Rows of f sum to 1; rows of p sum to 0; (f o q) 1 = (O o dO) 1 (the two matrix
    forms of Definition B.9); p equals the row form (diag(f_i) - f_i f_i^T) q_i;
    ln l equals the saved LSE (the paper's unshifted form)."""
    n, d = 10, 6
    Q, K, V, G = make(7, n, d)
    for mk in masks_for(n):
        dn = orc.attn_dense(Q[0, 0], K[0, 0], V[0, 0], G[0, 0], **mk)
        f, q, p = dn["f"], dn["q"], dn["p"]
        np.testing.assert_allclose(f.sum(1), 1.0, rtol=1e-14)
        assert np.abs(p.sum(1)).max() <= 1e-13 * np.abs(p).sum(1).max()
        O, LSE = orc.attn_fwd(Q, K, V, **mk)
        np.testing.assert_allclose(np.log(dn["l"]), LSE[0, 0], rtol=1e-13, atol=1e-14)
        np.testing.assert_allclose(dn["v_fq"], (O[0, 0] * G[0, 0]).sum(1), rtol=1e-11, atol=1e-13)
        np.testing.assert_allclose(q, G[0, 0] @ V[0, 0].T, rtol=1e-13, atol=1e-14)
        for i in range(n):
            row = (np.diag(f[i]) - np.outer(f[i], f[i])) @ q[i]
            np.testing.assert_allclose(p[i], row, rtol=1e-10, atol=1e-14)
        # the streaming backward agrees with products of the dense intermediates
        dQ, dK, dV = orc.attn_bwd(Q, K, V, O, G, LSE, **mk)
        s = 1 / math.sqrt(d)
        np.testing.assert_allclose(dQ[0, 0], s * p @ K[0, 0], rtol=1e-10, atol=1e-13)
        np.testing.assert_allclose(dK[0, 0], s * p.T @ Q[0, 0], rtol=1e-10, atol=1e-13)
        np.testing.assert_allclose(dV[0, 0], f.T @ G[0, 0], rtol=1e-10, atol=1e-13)


def test_special_cases():
    d = 5
    Q, K, V, G = make(8, 1, d)
    O, LSE = orc.attn_fwd(Q, K, V)
    dQ, dK, dV = orc.attn_bwd(Q, K, V, O, G, LSE)
    # n = 1: P = [1]
    np.testing.assert_allclose(O, V, rtol=1e-15)
    np.testing.assert_allclose(dV, G, rtol=1e-15)
    assert np.abs(dQ).max() < 1e-15 and np.abs(dK).max() < 1e-15
    np.testing.assert_allclose(LSE[0, 0, 0], (Q * K).sum() / math.sqrt(d), rtol=1e-14)
    # Q = 0: uniform attention over kept keys
    n = 9
    Q, K, V, G = make(8, n, d)
    Q[:] = 0
    O, LSE = orc.attn_fwd(Q, K, V)
    np.testing.assert_allclose(O[0, 0], np.tile(V[0, 0].mean(0), (n, 1)), rtol=1e-13)
    np.testing.assert_allclose(LSE, math.log(n), rtol=1e-14)
    O, LSE = orc.attn_fwd(Q, K, V, mask_kind=orc.MASK_CAUSAL)
    for i in range(n):
        np.testing.assert_allclose(O[0, 0, i], V[0, 0, : i + 1].mean(0), rtol=1e-13, atol=1e-15)
    # causal row 0 sees only key 0
    Q, K, V, G = make(9, n, d)
    O, _ = orc.attn_fwd(Q, K, V, mask_kind=orc.MASK_CAUSAL)
    np.testing.assert_allclose(O[0, 0, 0], V[0, 0, 0], rtol=1e-14)


def test_invariances():
    n, d = 11, 4
    Q, K, V, G = make(10, n, d)
    O, LSE = orc.attn_fwd(Q, K, V)
    dQ, dK, dV = orc.attn_bwd(Q, K, V, O, G, LSE)
    # adding the same vector to every key shifts each score row by a constant
    u = rnd(12, d)
    O2, LSE2 = orc.attn_fwd(Q, K + u, V)
    dQ2, _, dV2 = orc.attn_bwd(Q, K + u, V, O2, G, LSE2)
    np.testing.assert_allclose(O2, O, rtol=1e-11, atol=1e-13)
    np.testing.assert_allclose(dQ2, dQ, rtol=1e-9, atol=1e-12)
    np.testing.assert_allclose(dV2, dV, rtol=1e-10, atol=1e-13)
    # joint permutation of keys and values
    perm = np.array([(3 * i + 5) % n for i in range(n)])
    O3, LSE3 = orc.attn_fwd(Q, K[:, :, perm], V[:, :, perm])
    dQ3, dK3, dV3 = orc.attn_bwd(Q, K[:, :, perm], V[:, :, perm], O3, G, LSE3)
    np.testing.assert_allclose(O3, O, rtol=1e-12, atol=1e-14)
    np.testing.assert_allclose(dQ3, dQ, rtol=1e-10, atol=1e-13)
    np.testing.assert_allclose(dK3, dK[:, :, perm], rtol=1e-10, atol=1e-13)
    np.testing.assert_allclose(dV3, dV[:, :, perm], rtol=1e-10, atol=1e-13)
    # Q -> aQ, K -> K/a
    O4, _ = orc.attn_fwd(2.5 * Q, K / 2.5, V)
    np.testing.assert_allclose(O4, O, rtol=1e-12, atol=1e-14)
    # explicit scale: scale s on (Q, K) equals scale 1 on (sQ, K)
    O5, LSE5 = orc.attn_fwd(Q / math.sqrt(d), K, V, scale=1.0)
    np.testing.assert_allclose(O5, O, rtol=1e-12, atol=1e-14)
    np.testing.assert_allclose(LSE5, LSE, rtol=1e-12, atol=1e-14)


@pytest.mark.parametrize("n,block", [(8, 2), (12, 4), (10, 4)])
def test_masks_equal_brute_force_element_mask(n, block):
    """Causal and block masks equal the same computation under an explicit n x n mask
    (ragged last block included)."""
    d = 4
    Q, K, V, G = make(13, n, d, b=1, h=2)
    for mk in masks_for(n, block=block)[1:]:
        keep = keep_matrix(n, mk).astype(np.uint8)[None]
        O, LSE = orc.attn_fwd(Q, K, V, **mk)
        Oe, LSEe = orc.attn_fwd(Q, K, V, mask_kind=orc.MASK_ELEMENT, mask_bits=keep)
        assert np.array_equal(O, Oe) and np.array_equal(LSE, LSEe)
        g = orc.attn_bwd(Q, K, V, O, G, LSE, **mk)
        ge = orc.attn_bwd(Q, K, V, O, G, LSE, mask_kind=orc.MASK_ELEMENT, mask_bits=keep)
        for a, b in zip(g, ge):
            assert np.array_equal(a, b)


def test_per_head_masks_and_empty_rows():
    """mask_heads > 1 selects a mask per (batch, head); a row with no kept entry gives
    O = 0, LSE = -inf and no gradient."""
    n, d = 6, 3
    Q, K, V, G = make(14, n, d, b=1, h=2)
    keep = np.ones((2, n, n), np.uint8)
    keep[1] = np.tril(np.ones((n, n), np.uint8))
    keep[0, 2, :] = 0
    O, LSE = orc.attn_fwd(Q, K, V, mask_kind=orc.MASK_ELEMENT, mask_bits=keep)
    assert np.all(O[0, 0, 2] == 0) and LSE[0, 0, 2] == -np.inf
    Oc, LSEc = orc.attn_fwd(Q[:, 1:], K[:, 1:], V[:, 1:], mask_kind=orc.MASK_CAUSAL)
    assert np.array_equal(O[:, 1:], Oc) and np.array_equal(LSE[:, 1:], LSEc)
    dQ, dK, dV = orc.attn_bwd(Q, K, V, O, G, LSE, mask_kind=orc.MASK_ELEMENT, mask_bits=keep)
    assert np.all(np.isfinite(dQ)) and np.all(np.isfinite(dK)) and np.all(np.isfinite(dV))
    assert np.all(dQ[0, 0, 2] == 0)
    # dropping the empty row from the problem changes nothing for the others
    sel = [0, 1, 3, 4, 5]
    keep2 = keep[:1][:, sel]
    Q2, G2 = Q[:, :1, sel], G[:, :1, sel]
    # keys stay n long, so use the element mask with a rectangular trick: pad queries back
    Qp = np.zeros_like(Q[:, :1]); Qp[:, :, : len(sel)] = Q2
    Gp = np.zeros_like(Qp); Gp[:, :, : len(sel)] = G2
    kp = np.zeros((1, n, n), np.uint8); kp[:, : len(sel)] = keep2; kp[:, len(sel):] = 1
    Op, LSEp = orc.attn_fwd(Qp, K[:, :1], V[:, :1], mask_kind=orc.MASK_ELEMENT, mask_bits=kp)
    _, dKp, dVp = orc.attn_bwd(Qp, K[:, :1], V[:, :1], Op, Gp, LSEp, mask_kind=orc.MASK_ELEMENT, mask_bits=kp)
    np.testing.assert_allclose(dKp, dK[:, :1], rtol=1e-12, atol=1e-14)
    np.testing.assert_allclose(dVp, dV[:, :1], rtol=1e-12, atol=1e-14)


def test_heads_are_independent():
    n, d = 9, 4
    Q, K, V, G = make(15, n, d, b=2, h=3)
    O, LSE = orc.attn_fwd(Q, K, V, mask_kind=orc.MASK_CAUSAL)
    g = orc.attn_bwd(Q, K, V, O, G, LSE, mask_kind=orc.MASK_CAUSAL)
    for b in range(2):
        for h in range(3):
            sl = (slice(b, b + 1), slice(h, h + 1))
            O1, LSE1 = orc.attn_fwd(Q[sl], K[sl], V[sl], mask_kind=orc.MASK_CAUSAL)
            assert np.array_equal(O1, O[sl]) and np.array_equal(LSE1, LSE[sl])
            g1 = orc.attn_bwd(Q[sl], K[sl], V[sl], O1, G[sl], LSE1, mask_kind=orc.MASK_CAUSAL)
            for a, c in zip(g1, g):
                assert np.array_equal(a, c[sl])


# ---------------------------------------------------------------- I/O bound closed forms

def test_io_bound_pins():
    """Section 4: at M = d^2 both branches of Theorem 1.1 equal n^2 + n d; the sparse
    bound with dense counts equals the dense bound; dividing point Z_input^2 / Z_QK."""
    for n, d in ((8192, 128), (4096, 256), (1000, 10)):
        M = d * d
        a = (n * n * d * d + n * d ** 3) / M
        b = (n * n * d + n * d * d) / math.sqrt(M)
        assert a == pytest.approx(n * n + n * d) and b == pytest.approx(n * n + n * d)
        assert orc.io_bound_backward(n, d, M) == pytest.approx(n * n + n * d)
        for M in (d * d / 16, d * d, 16 * d * d):
            assert orc.io_bound_sparse(n * d, n * n, M) == pytest.approx(orc.io_bound_forward(n, d, M))
            assert orc.io_bound_sparse_formal(n * d, d * d, n * d, n * n, M) == pytest.approx(
                orc.io_bound_backward(n, d, M))
        # small cache uses the sqrt branch, large cache the 1/M branch
        assert orc.io_bound_backward(n, d, d * d / 4) == pytest.approx((n * n * d + n * d * d) / (d / 2))
        assert orc.io_bound_backward(n, d, 4 * d * d) == pytest.approx((n * n * d * d + n * d ** 3) / (4 * d * d))
    z_in, z_qk = 4194304.0, 111149056.0
    M_star = z_in ** 2 / z_qk
    assert z_in ** 2 / M_star == pytest.approx(z_in * math.sqrt(z_qk) / math.sqrt(M_star))

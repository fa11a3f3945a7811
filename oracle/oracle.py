"""Python face of the float64 CPU oracle (``attn_oracle.c``).

THIS IS TEST INFRASTRUCTURE: only the tests, the smoke check and the benchmark's
CPU-baseline leg may import it.  It shares nothing with the CUDA library.

All tensors are numpy float64 arrays shaped ``[batch, heads, n, d]`` (LSE
``[batch, heads, n]``).  Mask kinds: 0 none, 1 causal (keep j <= i), 2 block mask
(uint8 ``[mask_heads, nb, nb]``), 3 explicit element mask (uint8 ``[mask_heads, n, n]``,
the reference for ATTN_MASK_ELEMENT and the brute-force check of the other kinds).

``project`` / ``weight_grad`` / ``attn_weights_bwd`` cover the paper's own gradient target,
the attention weights X and Y (Definition 3.2, Appendix D).

Also here: ``io_bound_*`` -- the paper's closed-form I/O bounds (Theorem 1.1 and the
sparse lower bound, Theorem 1.2 / 4.5) as plain expressions, used to check the
library's bound calculators.
"""
from __future__ import annotations

import ctypes
import math
import os
import subprocess

import numpy as np

_HERE = os.path.dirname(os.path.abspath(__file__))
_SRC = os.path.join(_HERE, "attn_oracle.c")
_LIB = os.path.join(_HERE, "liboracle.so")

MASK_NONE, MASK_CAUSAL, MASK_BLOCK, MASK_ELEMENT, MASK_BLOCK_CAUSAL = 0, 1, 2, 3, 4


def build(force: bool = False) -> str:
    """Compile ``attn_oracle.c`` into ``liboracle.so`` beside it (gcc, OpenMP, no fast-math)."""
    if force or not os.path.exists(_LIB) or os.path.getmtime(_LIB) < os.path.getmtime(_SRC):
        tmp = _LIB + f".tmp{os.getpid()}"
        subprocess.check_call(["gcc", "-O2", "-fopenmp", "-shared", "-fPIC", "-std=c11", "-o", tmp, _SRC, "-lm"])
        os.replace(tmp, _LIB)
    return _LIB


_lib = None


def _load():
    global _lib
    if _lib is None:
        _lib = ctypes.CDLL(build())
        _lib.attn_oracle_threads.restype = ctypes.c_int
    return _lib


def threads() -> int:
    return int(_load().attn_oracle_threads())


def _p(a):
    return None if a is None else a.ctypes.data_as(ctypes.c_void_p)


def _f64(a):
    return np.ascontiguousarray(a, dtype=np.float64)


def _mask_args(mask_kind, block, mask_bits):
    if mask_kind in (MASK_BLOCK, MASK_ELEMENT, MASK_BLOCK_CAUSAL):
        mask_bits = np.ascontiguousarray(mask_bits, dtype=np.uint8)
        assert mask_bits.ndim == 3
        return mask_bits, int(mask_bits.shape[0])
    return None, 1


def attn_fwd(Q, K, V, *, mask_kind=MASK_NONE, block=128, mask_bits=None, scale=None):
    """Returns (O, LSE) for ``[batch, heads, n, d]`` inputs."""
    Q, K, V = _f64(Q), _f64(K), _f64(V)
    b, h, n, d = Q.shape
    scale = 1.0 / math.sqrt(d) if scale is None else float(scale)
    bits, mh = _mask_args(mask_kind, block, mask_bits)
    O = np.empty_like(Q)
    LSE = np.empty((b, h, n), dtype=np.float64)
    _load().attn_oracle_fwd(_p(Q), _p(K), _p(V), n, d, h, b, int(mask_kind), int(block), _p(bits), mh,
                            ctypes.c_double(scale), _p(O), _p(LSE))
    return O, LSE


def attn_bwd(Q, K, V, O, dO, LSE, *, mask_kind=MASK_NONE, block=128, mask_bits=None, scale=None):
    """Returns (dQ, dK, dV) given the forward's O and LSE."""
    Q, K, V, O, dO, LSE = _f64(Q), _f64(K), _f64(V), _f64(O), _f64(dO), _f64(LSE)
    b, h, n, d = Q.shape
    scale = 1.0 / math.sqrt(d) if scale is None else float(scale)
    bits, mh = _mask_args(mask_kind, block, mask_bits)
    dQ, dK, dV = np.empty_like(Q), np.empty_like(Q), np.empty_like(Q)
    _load().attn_oracle_bwd(_p(Q), _p(K), _p(V), _p(O), _p(dO), _p(LSE), n, d, h, b, int(mask_kind), int(block),
                            _p(bits), mh, ctypes.c_double(scale), _p(dQ), _p(dK), _p(dV))
    return dQ, dK, dV


def attn_dense(Q, K, V, dO, *, mask_kind=MASK_NONE, block=128, mask_bits=None, scale=None):
    """One head (``[n, d]`` inputs): the dense intermediates of the no-cache algorithm.

    Returns dict with l [n], f, q, p [n, n] and v_fq = (f o q) 1 [n].
    """
    Q, K, V, dO = _f64(Q), _f64(K), _f64(V), _f64(dO)
    n, d = Q.shape
    scale = 1.0 / math.sqrt(d) if scale is None else float(scale)
    bits = None
    if mask_kind in (MASK_BLOCK, MASK_ELEMENT, MASK_BLOCK_CAUSAL):
        bits = np.ascontiguousarray(mask_bits, dtype=np.uint8)
    out = {"l": np.empty(n), "f": np.empty((n, n)), "q": np.empty((n, n)), "p": np.empty((n, n)),
           "v_fq": np.empty(n)}
    _load().attn_oracle_dense(_p(Q), _p(K), _p(V), _p(dO), n, d, int(mask_kind), int(block), _p(bits),
                              ctypes.c_double(scale), _p(out["l"]), _p(out["f"]), _p(out["q"]), _p(out["p"]),
                              _p(out["v_fq"]))
    return out


def project(A, W):
    """``out[b, h] = A[b, h] @ W[(b*heads + h) % weight_units]`` -- S = A1 X or h = A3 Y
    (Appendix D, phase 1).  ``A`` is ``[batch, heads, n, d]``, ``W`` is ``[weight_units, d, d]``."""
    A, W = _f64(A), _f64(W)
    b, h, n, d = A.shape
    assert W.shape[1:] == (d, d) and W.shape[0] in (1, h, b * h)
    out = np.empty_like(A)
    _load().attn_oracle_project(_p(A), _p(W), _p(out), n, d, ctypes.c_long(b * h), ctypes.c_long(W.shape[0]))
    return out


def weight_grad(A, G, weight_units: int):
    """``g[w] = sum over units u with u % weight_units == w of A[u]^T @ G[u]`` -- Definition 3.2
    with ``G = p A2`` (the gradient with respect to S = A1 X)."""
    A, G = _f64(A), _f64(G)
    b, h, n, d = A.shape
    assert weight_units in (1, h, b * h)
    g = np.empty((weight_units, d, d), dtype=np.float64)
    _load().attn_oracle_weight_grad(_p(A), _p(G), _p(g), n, d, ctypes.c_long(b * h), ctypes.c_long(weight_units))
    return g


def attn_weights_bwd(A1, A2, A3, X, Y, dO, *, mask_kind=MASK_NONE, block=128, mask_bits=None, scale=None):
    """The paper's backward problem with its own inputs: S = A1 X, h = A3 Y (phase 1), the forward for
    O and l, then dL/dX = A1^T p A2 and dL/dY = A3^T f^T dO.  Returns a dict with S, h, O, LSE, dS
    (the gradient of S, = scale * p A2), dK, dh, gX, gY."""
    S, h = project(A1, X), project(A3, Y)
    kw = dict(mask_kind=mask_kind, block=block, mask_bits=mask_bits, scale=scale)
    O, LSE = attn_fwd(S, A2, h, **kw)
    dS, dK, dh = attn_bwd(S, A2, h, O, dO, LSE, **kw)
    return {"S": S, "h": h, "O": O, "LSE": LSE, "dS": dS, "dK": dK, "dh": dh,
            "gX": weight_grad(A1, dS, np.asarray(X).shape[0]), "gY": weight_grad(A3, dh, np.asarray(Y).shape[0])}


# ---- closed-form I/O bounds, constants taken as 1 (Theorem 1.1; Theorem 1.2 / 4.5) ----

def io_bound_backward(n: float, d: float, M: float) -> float:
    """min{(n^2 d^2 + n d^3)/M, (n^2 d + n d^2)/sqrt(M)} (Theorem 1.1)."""
    return min((n * n * d * d + n * d ** 3) / M, (n * n * d + n * d * d) / math.sqrt(M))


def io_bound_forward(n: float, d: float, M: float) -> float:
    """min{n^2 d^2 / M, n^2 d / sqrt(M)} (Table 1, forward rows)."""
    return min(n * n * d * d / M, n * n * d / math.sqrt(M))


def io_bound_sparse(z_input: float, z_qk: float, M: float) -> float:
    """min{Z_input^2 / M, Z_input sqrt(Z_QK) / sqrt(M)} (Theorem 1.2)."""
    return min(z_input ** 2 / M, z_input * math.sqrt(z_qk) / math.sqrt(M))


def io_bound_sparse_formal(z_a: float, z_x: float, z_ax: float, z_axa: float, M: float) -> float:
    """min{(Z_A^2 + Z_A Z_X)/M, (Z_A sqrt(Z_AXA) + sqrt(Z_A Z_X Z_AX))/sqrt(M)} (Theorem 4.5)."""
    return min((z_a ** 2 + z_a * z_x) / M,
               (z_a * math.sqrt(z_axa) + math.sqrt(z_a * z_x * z_ax)) / math.sqrt(M))

"""ctypes binding of ``libattn_b200.so`` -- same names as ``include/attn.h``.

Argument marshalling only: every step of the attention path runs in the library's
CUDA kernels.  Tensors are torch CUDA tensors (torch supplies device memory and the
stream, nothing else); ``attn_fwd`` / ``attn_bwd`` enqueue on torch's current stream and
do not synchronise.  If the library is missing this module raises -- there is no
fallback of any kind.
"""
from __future__ import annotations

import ctypes
import os
from dataclasses import dataclass

HERE = os.path.dirname(os.path.abspath(__file__))
LIB_PATH = os.path.join(HERE, "libattn_b200.so")

ATTN_OK = 0
(ATTN_ERR_NULL, ATTN_ERR_SHAPE, ATTN_ERR_DTYPE, ATTN_ERR_ALIGN, ATTN_ERR_TILE, ATTN_ERR_MASK, ATTN_ERR_WORKSPACE,
 ATTN_ERR_ARCH, ATTN_ERR_LAUNCH, ATTN_ERR_DEVICE_TIMEOUT) = range(1, 11)
ATTN_F32, ATTN_BF16 = 0, 1
ATTN_MASK_NONE, ATTN_MASK_CAUSAL, ATTN_MASK_BLOCK_SPARSE, ATTN_MASK_BLOCK_SPARSE_CAUSAL, ATTN_MASK_ELEMENT = 0, 1, 2, 3, 4
ATTN_ALGO_AUTO, ATTN_ALGO_FUSED, ATTN_ALGO_MATERIALIZED, ATTN_ALGO_SIMT = 0, 1, 2, 3

# every symbol include/attn.h declares
EXPORTS = (
    "attn_fwd", "attn_bwd", "attn_bwd_preprocess", "attn_fwd_workspace_bytes", "attn_bwd_workspace_bytes",
    "attn_workspace_status", "attn_supported_cfgs", "attn_cfg_onchip_elems", "attn_io_bound_elems",
    "attn_io_bound_sparse_elems", "attn_io_replay", "attn_status_str", "attn_kernel_launches", "attn_timing_enable",
    "attn_timing_collect", "attn_bwd_noalloc", "attn_noalloc_scratch_bytes", "attn_noalloc_status",
    "attn_selftest_wait_timeout", "attn_mask_from_coo",
    "attn_project", "attn_weight_grad", "attn_weights_bwd", "attn_weights_bwd_workspace_bytes",
)


class AttnError(RuntimeError):
    def __init__(self, status: int, where: str):
        self.status = status
        super().__init__(f"{where}: {status_str(status)} (attn_status {status})")


class CMask(ctypes.Structure):
    _fields_ = [("kind", ctypes.c_int), ("block", ctypes.c_int), ("block_mask", ctypes.c_void_p),
                ("mask_heads", ctypes.c_int)]


class CCfg(ctypes.Structure):
    _fields_ = [("tile_q", ctypes.c_int), ("tile_k", ctypes.c_int), ("tile_d", ctypes.c_int),
                ("algo", ctypes.c_int), ("deterministic", ctypes.c_int)]


class CIoCount(ctypes.Structure):
    _fields_ = [("loads", ctypes.c_double), ("stores", ctypes.c_double), ("reductions", ctypes.c_double)]


@dataclass
class Mask:
    """Which score entries are kept; ``block_mask`` is a CUDA uint8 tensor ``[mask_heads, nb, nb]``, or, for
    ATTN_MASK_ELEMENT, a CUDA int32 tensor ``[mask_heads, n, ceil(n / 32)]`` of keep bits."""
    kind: int = ATTN_MASK_NONE
    block: int = 128
    block_mask: object = None

    def c(self) -> CMask | None:
        if self.kind == ATTN_MASK_ELEMENT:
            bm = self.block_mask
            return CMask(self.kind, 0, bm.data_ptr() if bm is not None else None, int(bm.shape[0]) if bm is not None else 1)
        if self.kind in (ATTN_MASK_BLOCK_SPARSE, ATTN_MASK_BLOCK_SPARSE_CAUSAL):
            bm = self.block_mask
            return CMask(self.kind, self.block, bm.data_ptr() if bm is not None else None,
                         int(bm.shape[0]) if bm is not None else 1)
        return CMask(self.kind, 0, None, 1)


@dataclass
class Cfg:
    tile_q: int = 0
    tile_k: int = 0
    tile_d: int = 0
    algo: int = ATTN_ALGO_AUTO
    deterministic: int = 0

    def c(self) -> CCfg:
        return CCfg(self.tile_q, self.tile_k, self.tile_d, self.algo, self.deterministic)


_lib = None


def lib() -> ctypes.CDLL:
    """Loads the library (once).  Raises if it has not been built."""
    global _lib
    if _lib is not None:
        return _lib
    if not os.path.exists(LIB_PATH):
        raise RuntimeError(f"{LIB_PATH} is missing: build it with `python -m paper_2410_09397_b200.build` "
                           "(there is no fallback path)")
    L = ctypes.CDLL(LIB_PATH)
    vp, ci, cf, sz = ctypes.c_void_p, ctypes.c_int, ctypes.c_float, ctypes.c_size_t
    L.attn_fwd.restype = ci
    L.attn_fwd.argtypes = [vp, vp, vp, vp, vp, ci, ci, ci, ci, ctypes.POINTER(CMask), ci, cf,
                           ctypes.POINTER(CCfg), vp, sz, vp]
    L.attn_bwd.restype = ci
    L.attn_bwd.argtypes = [vp] * 9 + [ci, ci, ci, ci, ctypes.POINTER(CMask), ci, cf, ctypes.POINTER(CCfg), vp, sz, vp]
    L.attn_bwd_noalloc.restype = ci
    L.attn_bwd_noalloc.argtypes = [vp] * 9 + [ci, ci, ci, ci, ctypes.POINTER(CMask), ci, cf, ctypes.POINTER(CCfg), vp]
    L.attn_noalloc_scratch_bytes.restype = sz
    L.attn_noalloc_scratch_bytes.argtypes = []
    L.attn_noalloc_status.restype = ci
    L.attn_noalloc_status.argtypes = [vp]
    L.attn_selftest_wait_timeout.restype = ci
    L.attn_selftest_wait_timeout.argtypes = [vp, sz, ctypes.c_uint, vp]
    L.attn_mask_from_coo.restype = ci
    L.attn_mask_from_coo.argtypes = [vp, vp, vp, sz, ci, ci, vp, vp]
    L.attn_bwd_preprocess.restype = ci
    L.attn_bwd_preprocess.argtypes = [vp, vp, vp, sz, ci, ci, vp]
    for f in (L.attn_fwd_workspace_bytes, L.attn_bwd_workspace_bytes):
        f.restype = sz
        f.argtypes = [ci, ci, ci, ci, ctypes.POINTER(CMask), ci, ctypes.POINTER(CCfg)]
    L.attn_project.restype = ci
    L.attn_project.argtypes = [vp, vp, vp, ci, ci, ci, ci, ci, ci, vp, sz, vp]
    L.attn_weight_grad.restype = ci
    L.attn_weight_grad.argtypes = [vp, vp, vp, ci, ci, ci, ci, ci, ci, vp, sz, vp]
    L.attn_weights_bwd.restype = ci
    L.attn_weights_bwd.argtypes = [vp] * 10 + [ci, ci, ci, ci, ci, ctypes.POINTER(CMask), ci, cf,
                                               ctypes.POINTER(CCfg), vp, sz, vp]
    L.attn_weights_bwd_workspace_bytes.restype = sz
    L.attn_weights_bwd_workspace_bytes.argtypes = [ci, ci, ci, ci, ctypes.POINTER(CMask), ci, ctypes.POINTER(CCfg)]
    L.attn_workspace_status.restype = ci
    L.attn_workspace_status.argtypes = [vp, vp]
    L.attn_supported_cfgs.restype = ci
    L.attn_supported_cfgs.argtypes = [ci, ci, ctypes.POINTER(CCfg), ci]
    L.attn_cfg_onchip_elems.restype = sz
    L.attn_cfg_onchip_elems.argtypes = [ci, ci, ctypes.POINTER(CCfg), ci]
    L.attn_io_bound_elems.restype = ctypes.c_double
    L.attn_io_bound_elems.argtypes = [ctypes.c_double] * 3 + [ci]
    L.attn_io_bound_sparse_elems.restype = ctypes.c_double
    L.attn_io_bound_sparse_elems.argtypes = [ctypes.c_double] * 3
    L.attn_io_replay.restype = ci
    L.attn_io_replay.argtypes = [ci, ci, ci, ci, ctypes.POINTER(CCfg), ci, ctypes.POINTER(CIoCount)]
    L.attn_kernel_launches.restype = ctypes.c_ulonglong
    L.attn_kernel_launches.argtypes = []
    L.attn_timing_enable.restype = ci
    L.attn_timing_enable.argtypes = [ci]
    L.attn_timing_collect.restype = ci
    L.attn_timing_collect.argtypes = [ctypes.POINTER(cf), ctypes.POINTER(ctypes.c_char_p), ci]
    L.attn_status_str.restype = ctypes.c_char_p
    L.attn_status_str.argtypes = [ci]
    _lib = L
    return L


def status_str(status: int) -> str:
    return lib().attn_status_str(int(status)).decode()


def _ref(x):
    return None if x is None else ctypes.byref(x)


def _dtype_code(t) -> int:
    import torch
    if t.dtype == torch.float32:
        return ATTN_F32
    if t.dtype == torch.bfloat16:
        return ATTN_BF16
    raise AttnError(ATTN_ERR_DTYPE, "binding")


def _check_tensors(*ts):
    for t in ts:
        if not t.is_cuda or not t.is_contiguous():
            raise ValueError("tensors must be contiguous CUDA tensors")


def _stream() -> int:
    import torch
    return torch.cuda.current_stream().cuda_stream


def attn_fwd_workspace_bytes(n, d, heads, batch, mask: Mask | None, dt: int, cfg: Cfg | None) -> int:
    return int(lib().attn_fwd_workspace_bytes(n, d, heads, batch, _ref(mask.c() if mask else None), dt,
                                              _ref(cfg.c() if cfg else None)))


def attn_bwd_workspace_bytes(n, d, heads, batch, mask: Mask | None, dt: int, cfg: Cfg | None) -> int:
    return int(lib().attn_bwd_workspace_bytes(n, d, heads, batch, _ref(mask.c() if mask else None), dt,
                                              _ref(cfg.c() if cfg else None)))


def _workspace(nbytes: int, like):
    import torch
    return torch.empty(max(nbytes, 256), dtype=torch.uint8, device=like.device)


def attn_fwd(Q, K, V, O=None, LSE=None, *, mask: Mask | None = None, scale: float = 0.0, cfg: Cfg | None = None,
             workspace=None):
    """O, LSE = softmax(scale * Q K^T restricted to kept entries) V.  Tensors ``[batch, heads, n, d]``."""
    import torch
    _check_tensors(Q, K, V)
    b, h, n, d = Q.shape
    dt = _dtype_code(Q)
    if O is None:
        O = torch.empty_like(Q)
    if LSE is None:
        LSE = torch.empty((b, h, n), dtype=torch.float32, device=Q.device)
    if workspace is None:
        workspace = _workspace(attn_fwd_workspace_bytes(n, d, h, b, mask, dt, cfg), Q)
    cm, cc = (mask.c() if mask else None), (cfg.c() if cfg else None)
    st = lib().attn_fwd(Q.data_ptr(), K.data_ptr(), V.data_ptr(), O.data_ptr(), LSE.data_ptr(), n, d, h, b, _ref(cm),
                        dt, scale, _ref(cc), workspace.data_ptr(), workspace.numel(), _stream())
    if st != ATTN_OK:
        raise AttnError(st, "attn_fwd")
    return O, LSE


def attn_bwd(Q, K, V, O, dO, LSE, dQ=None, dK=None, dV=None, *, mask: Mask | None = None, scale: float = 0.0,
             cfg: Cfg | None = None, workspace=None):
    """dQ, dK, dV of sum(O o G) given dO = G and the forward's O, LSE."""
    import torch
    _check_tensors(Q, K, V, O, dO, LSE)
    b, h, n, d = Q.shape
    dt = _dtype_code(Q)
    dQ = torch.empty_like(Q) if dQ is None else dQ
    dK = torch.empty_like(Q) if dK is None else dK
    dV = torch.empty_like(Q) if dV is None else dV
    if workspace is None:
        workspace = _workspace(attn_bwd_workspace_bytes(n, d, h, b, mask, dt, cfg), Q)
    cm, cc = (mask.c() if mask else None), (cfg.c() if cfg else None)
    st = lib().attn_bwd(Q.data_ptr(), K.data_ptr(), V.data_ptr(), O.data_ptr(), dO.data_ptr(), LSE.data_ptr(),
                        dQ.data_ptr(), dK.data_ptr(), dV.data_ptr(), n, d, h, b, _ref(cm), dt, scale, _ref(cc),
                        workspace.data_ptr(), workspace.numel(), _stream())
    if st != ATTN_OK:
        raise AttnError(st, "attn_bwd")
    return dQ, dK, dV


def attn_bwd_preprocess(O, dO, D=None):
    """D = rowsum(dO o O) over the last dimension; returns float32 of O.shape[:-1]."""
    import torch
    _check_tensors(O, dO)
    d = O.shape[-1]
    rows = O.numel() // d
    if D is None:
        D = torch.empty(O.shape[:-1], dtype=torch.float32, device=O.device)
    st = lib().attn_bwd_preprocess(O.data_ptr(), dO.data_ptr(), D.data_ptr(), rows, d, _dtype_code(O), _stream())
    if st != ATTN_OK:
        raise AttnError(st, "attn_bwd_preprocess")
    return D


def attn_project(A, W, out=None, *, workspace=None):
    """out[b, h] = A[b, h] @ W[(b * heads + h) % weight_units]; ``W`` is ``[weight_units, d, d]``."""
    import torch
    _check_tensors(A, W)
    b, h, n, d = A.shape
    out = torch.empty_like(A) if out is None else out
    workspace = _workspace(256, A) if workspace is None else workspace
    st = lib().attn_project(A.data_ptr(), W.data_ptr(), out.data_ptr(), n, d, h, b, W.shape[0], _dtype_code(A),
                            workspace.data_ptr(), workspace.numel(), _stream())
    if st != ATTN_OK:
        raise AttnError(st, "attn_project")
    return out


def attn_weight_grad(A, G, weight_units: int, g=None, *, workspace=None):
    """g[w] = sum of A[u]^T @ G[u] over the units u with u % weight_units == w; float32 ``[weight_units, d, d]``."""
    import torch
    _check_tensors(A, G)
    b, h, n, d = A.shape
    g = torch.empty((weight_units, d, d), dtype=torch.float32, device=A.device) if g is None else g
    workspace = _workspace(256, A) if workspace is None else workspace
    st = lib().attn_weight_grad(A.data_ptr(), G.data_ptr(), g.data_ptr(), n, d, h, b, weight_units, _dtype_code(A),
                                workspace.data_ptr(), workspace.numel(), _stream())
    if st != ATTN_OK:
        raise AttnError(st, "attn_weight_grad")
    return g


def attn_weights_bwd_workspace_bytes(n, d, heads, batch, mask: Mask | None, dt: int, cfg: Cfg | None) -> int:
    return int(lib().attn_weights_bwd_workspace_bytes(n, d, heads, batch, _ref(mask.c() if mask else None), dt,
                                                      _ref(cfg.c() if cfg else None)))


def attn_weights_bwd(A1, A2, A3, S, h, O, dO, LSE, weight_units: int, gX=None, gY=None, *, want_gY: bool = True,
                     mask: Mask | None = None, scale: float = 0.0, cfg: Cfg | None = None, workspace=None):
    """gX = dL/dX, gY = dL/dY (None when ``want_gY`` is false) given S = A1 X, h = A3 Y and the forward's O, LSE."""
    import torch
    _check_tensors(A1, A2, S, h, O, dO, LSE)
    b, nh, n, d = S.shape
    dt = _dtype_code(S)
    gX = torch.empty((weight_units, d, d), dtype=torch.float32, device=S.device) if gX is None else gX
    if want_gY:
        _check_tensors(A3)
        gY = torch.empty((weight_units, d, d), dtype=torch.float32, device=S.device) if gY is None else gY
    else:
        gY = None
    if workspace is None:
        workspace = _workspace(attn_weights_bwd_workspace_bytes(n, d, nh, b, mask, dt, cfg), S)
    cm, cc = (mask.c() if mask else None), (cfg.c() if cfg else None)
    st = lib().attn_weights_bwd(A1.data_ptr(), A2.data_ptr(), A3.data_ptr() if A3 is not None else None, S.data_ptr(),
                                h.data_ptr(), O.data_ptr(), dO.data_ptr(), LSE.data_ptr(), gX.data_ptr(),
                                gY.data_ptr() if gY is not None else None, n, d, nh, b, weight_units, _ref(cm), dt,
                                scale, _ref(cc), workspace.data_ptr(), workspace.numel(), _stream())
    if st != ATTN_OK:
        raise AttnError(st, "attn_weights_bwd")
    return gX, gY


def attn_workspace_status(workspace) -> int:
    return int(lib().attn_workspace_status(workspace.data_ptr(), _stream()))


def attn_supported_cfgs(d: int, dt: int) -> list[Cfg]:
    buf = (CCfg * 64)()
    cnt = lib().attn_supported_cfgs(d, dt, buf, 64)
    return [Cfg(buf[i].tile_q, buf[i].tile_k, buf[i].tile_d, buf[i].algo, 0) for i in range(min(cnt, 64))]


def attn_cfg_onchip_elems(d: int, dt: int, cfg: Cfg | None, backward: bool) -> int:
    return int(lib().attn_cfg_onchip_elems(d, dt, _ref(cfg.c() if cfg else None), int(backward)))


def attn_io_replay(n: int, d: int, mask_kind: int, dt: int, cfg: Cfg | None, backward: bool) -> dict:
    """Elements one head moves across the SM boundary under ``cfg``: {"loads", "stores", "reductions", "total"}."""
    out = CIoCount()
    st = lib().attn_io_replay(n, d, mask_kind, dt, _ref(cfg.c() if cfg else None), int(backward), ctypes.byref(out))
    if st != ATTN_OK:
        raise AttnError(st, "attn_io_replay")
    return {"loads": out.loads, "stores": out.stores, "reductions": out.reductions,
            "total": out.loads + out.stores + out.reductions}


def attn_mask_from_coo(rows, cols, heads, n: int, mask_heads: int = 1, bitmap=None):
    """Bitmap of an ATTN_MASK_ELEMENT mask from CUDA int32 coordinate tensors (``heads`` may be None)."""
    import torch
    nnz = int(rows.numel())
    if bitmap is None:
        bitmap = torch.empty((mask_heads, n, (n + 31) // 32), dtype=torch.int32, device=rows.device)
    st = lib().attn_mask_from_coo(rows.data_ptr() if nnz else None, cols.data_ptr() if nnz else None,
                                  heads.data_ptr() if heads is not None else None, nnz, n, mask_heads, bitmap.data_ptr(),
                                  _stream())
    if st != ATTN_OK:
        raise AttnError(st, "attn_mask_from_coo")
    return bitmap


def attn_io_bound_elems(n, d, M, backward: bool) -> float:
    return float(lib().attn_io_bound_elems(float(n), float(d), float(M), int(backward)))


def attn_io_bound_sparse_elems(z_input, z_qk, M) -> float:
    return float(lib().attn_io_bound_sparse_elems(float(z_input), float(z_qk), float(M)))


def attn_kernel_launches() -> int:
    return int(lib().attn_kernel_launches())


def attn_timing_enable(on: bool) -> None:
    st = lib().attn_timing_enable(int(on))
    if st != ATTN_OK:
        raise AttnError(st, "attn_timing_enable")


def attn_timing_collect(max_entries: int = 256) -> list[tuple[str, float]]:
    """[(kernel name, milliseconds), ...] for the launches since the last collect."""
    ms = (ctypes.c_float * max_entries)()
    names = (ctypes.c_char_p * max_entries)()
    cnt = lib().attn_timing_collect(ms, names, max_entries)
    return [(names[i].decode(), float(ms[i])) for i in range(cnt)]


def attn_noalloc_scratch_bytes() -> int:
    return int(lib().attn_noalloc_scratch_bytes())


def attn_noalloc_status() -> int:
    """Synchronises the current stream; status word of the last ``attn_bwd_noalloc`` on this device."""
    return int(lib().attn_noalloc_status(_stream()))


def attn_selftest_wait_timeout(workspace, limit_us: int = 2000) -> None:
    """Enqueues the bounded-wait self-test: afterwards ``attn_workspace_status(workspace)`` is
    ``ATTN_ERR_DEVICE_TIMEOUT``.  ``workspace``: CUDA uint8 tensor of at least 256 bytes."""
    st = lib().attn_selftest_wait_timeout(workspace.data_ptr(), workspace.numel(), limit_us, _stream())
    if st != ATTN_OK:
        raise AttnError(st, "attn_selftest_wait_timeout")


def attn_bwd_noalloc(Q, K, V, O, dO, LSE, dQ, dK, dV, *, mask: Mask | None = None, scale: float = 0.0,
                     cfg: Cfg | None = None):
    """``attn_bwd`` without a workspace, for callers that cannot allocate device memory.

    The caller passes every tensor, outputs included (this wrapper allocates nothing
    either); the scratch is an 8 MiB array inside the library, shared by all calls on a
    device, so calls must not overlap on the GPU.  Problems whose workspace would exceed
    it raise ``AttnError(ATTN_ERR_WORKSPACE)``.
    """
    _check_tensors(Q, K, V, O, dO, LSE, dQ, dK, dV)
    b, h, n, d = Q.shape
    cm, cc = (mask.c() if mask else None), (cfg.c() if cfg else None)
    st = lib().attn_bwd_noalloc(Q.data_ptr(), K.data_ptr(), V.data_ptr(), O.data_ptr(), dO.data_ptr(),
                                LSE.data_ptr(), dQ.data_ptr(), dK.data_ptr(), dV.data_ptr(), n, d, h, b, _ref(cm),
                                _dtype_code(Q), scale, _ref(cc), _stream())
    if st != ATTN_OK:
        raise AttnError(st, "attn_bwd_noalloc")
    return dQ, dK, dV

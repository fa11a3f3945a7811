"""Host-side checks of the C-ABI library that need no GPU: it loads, exports every
symbol the header declares, rejects bad arguments before any launch, and its bound
calculators reproduce the paper's closed forms."""
import ctypes
import math
import os
import re

import pytest

from oracle import oracle as orc
from paper_2410_09397_b200 import binding as B

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))


@pytest.fixture(scope="module")
def lib():
    if not os.path.exists(B.LIB_PATH):
        from paper_2410_09397_b200 import build
        build.build()
    return B.lib()


def declared_symbols():
    text = open(os.path.join(ROOT, "include", "attn.h")).read()
    text = re.sub(r"/\*.*?\*/", "", text, flags=re.S)
    return sorted(set(re.findall(r"\b(attn_[a-z_0-9]+)\s*\(", text)))


def test_exports_every_declared_symbol(lib):
    names = declared_symbols()
    assert set(names) == set(B.EXPORTS), (names, B.EXPORTS)
    for name in names:
        assert getattr(lib, name) is not None


def golden_lines(name):
    with open(os.path.join(ROOT, "tests", "golden", name)) as f:
        return [ln.split() for ln in f if ln.strip() and not ln.startswith("#")]


def test_io_bound_golden_and_oracle(lib):
    for n, d, M, backward, want in golden_lines("io_bounds.txt"):
        got = B.attn_io_bound_elems(float(n), float(d), float(M), int(backward))
        assert got == pytest.approx(float(want), rel=1e-12)
    for n, d in ((8192, 128), (4096, 256), (32768, 128), (100, 7)):
        for M in (64.0, 4096.0, d * d, 116000.0, 3e7):
            assert B.attn_io_bound_elems(n, d, M, True) == pytest.approx(orc.io_bound_backward(n, d, M), rel=1e-13)
            assert B.attn_io_bound_elems(n, d, M, False) == pytest.approx(orc.io_bound_forward(n, d, M), rel=1e-13)
            assert B.attn_io_bound_sparse_elems(n * d, 0.1 * n * n, M) == pytest.approx(
                orc.io_bound_sparse(n * d, 0.1 * n * n, M), rel=1e-13)
    # dividing point of the sparse bound (Section 4.1): both branches equal at M = Z_input^2 / Z_QK
    z_in, z_qk = 4194304.0, 111149056.0
    Ms = z_in ** 2 / z_qk
    assert B.attn_io_bound_sparse_elems(z_in, z_qk, Ms) == pytest.approx(z_in ** 2 / Ms, rel=1e-12)
    assert B.attn_io_bound_sparse_elems(z_in, z_qk, Ms / 4) == pytest.approx(z_in * math.sqrt(z_qk) / math.sqrt(Ms / 4))
    assert B.attn_io_bound_sparse_elems(z_in, z_qk, Ms * 4) == pytest.approx(z_in ** 2 / (4 * Ms))
    assert B.attn_io_bound_elems(0, 1, 1, 1) == 0.0


def test_argument_errors_come_before_any_launch(lib):
    ws = B.attn_fwd_workspace_bytes(128, 64, 1, 1, None, B.ATTN_F32, None)
    assert ws >= 256
    fake = 0x10000  # never dereferenced: every call below must fail validation first
    args = dict(n=128, d=64, heads=1, batch=1, dt=B.ATTN_F32)

    def fwd(Q=fake, K=fake, V=fake, O=fake, LSE=fake, n=128, d=64, heads=1, batch=1, mask=None, dt=B.ATTN_F32,
            cfg=None, w=fake, wb=1 << 20):
        return lib.attn_fwd(Q, K, V, O, LSE, n, d, heads, batch, mask, dt, 0.0, cfg, w, wb, None)

    assert fwd(Q=None) == B.ATTN_ERR_NULL
    assert fwd(LSE=None) == B.ATTN_ERR_NULL
    assert fwd(dt=7) == B.ATTN_ERR_DTYPE
    assert fwd(n=0) == B.ATTN_ERR_SHAPE
    assert fwd(d=60) == B.ATTN_ERR_SHAPE
    assert fwd(d=512) == B.ATTN_ERR_SHAPE
    assert fwd(heads=0) == B.ATTN_ERR_SHAPE
    assert fwd(w=None) == B.ATTN_ERR_WORKSPACE
    assert fwd(wb=8) == B.ATTN_ERR_WORKSPACE
    assert fwd(w=fake + 16) == B.ATTN_ERR_ALIGN
    assert fwd(Q=fake + 4) == B.ATTN_ERR_ALIGN
    bad_mask = B.CMask(9, 0, None, 1)
    assert fwd(mask=ctypes.byref(bad_mask)) == B.ATTN_ERR_MASK
    sparse_no_ptr = B.CMask(B.ATTN_MASK_BLOCK_SPARSE, 128, None, 1)
    assert fwd(mask=ctypes.byref(sparse_no_ptr)) == B.ATTN_ERR_NULL
    sparse_bad_heads = B.CMask(B.ATTN_MASK_BLOCK_SPARSE, 128, fake, 3)
    assert fwd(mask=ctypes.byref(sparse_bad_heads)) == B.ATTN_ERR_MASK
    bad_tile = B.CCfg(48, 0, 0, B.ATTN_ALGO_SIMT, 0)
    assert fwd(cfg=ctypes.byref(bad_tile)) == B.ATTN_ERR_TILE
    fused_f32 = B.CCfg(0, 0, 0, B.ATTN_ALGO_FUSED, 0)
    assert fwd(cfg=ctypes.byref(fused_f32)) == B.ATTN_ERR_DTYPE
    bad_algo = B.CCfg(0, 0, 0, 17, 0)
    assert fwd(cfg=ctypes.byref(bad_algo)) == B.ATTN_ERR_TILE
    # backward: same order
    r = lib.attn_bwd(fake, fake, fake, fake, fake, fake, fake, fake, None, 128, 64, 1, 1, None, B.ATTN_F32, 0.0, None,
                     fake, 1 << 20, None)
    assert r == B.ATTN_ERR_NULL
    assert lib.attn_bwd_preprocess(None, fake, fake, 10, 64, B.ATTN_BF16, None) == B.ATTN_ERR_NULL
    assert lib.attn_bwd_preprocess(fake, fake, fake, 10, 12, B.ATTN_BF16, None) == B.ATTN_ERR_SHAPE
    assert lib.attn_workspace_status(None, None) == B.ATTN_ERR_NULL
    for s in range(0, 11):
        assert B.status_str(s) != "unknown status"
    assert B.status_str(99) == "unknown status"


def test_workspace_sizes_and_cfgs(lib):
    # backward workspace holds D (float per row) after the status block
    n, d, h, b = 2048, 64, 16, 4
    w = B.attn_bwd_workspace_bytes(n, d, h, b, None, B.ATTN_BF16, B.Cfg(algo=B.ATTN_ALGO_SIMT))
    assert w >= 256 + 4 * n * h * b
    assert B.attn_bwd_workspace_bytes(0, d, h, b, None, B.ATTN_BF16, None) == 0
    cfgs = B.attn_supported_cfgs(64, B.ATTN_F32)
    assert any(c.algo == B.ATTN_ALGO_SIMT and c.tile_q == 64 for c in cfgs)
    for c in cfgs:
        assert B.attn_cfg_onchip_elems(64, B.ATTN_F32, c, True) > 0
    assert B.attn_cfg_onchip_elems(64, B.ATTN_F32, B.Cfg(tile_q=48, algo=B.ATTN_ALGO_SIMT), True) == 0


def test_weight_entry_points_validate_before_any_launch(lib):
    fake = 0x10000  # never dereferenced

    def proj(A=fake, W=fake, out=fake, n=128, d=64, heads=2, batch=3, wu=2, dt=B.ATTN_BF16, w=fake, wb=256):
        return lib.attn_project(A, W, out, n, d, heads, batch, wu, dt, w, wb, None)

    def grad(A=fake, G=fake, g=fake, n=128, d=64, heads=2, batch=3, wu=6, dt=B.ATTN_BF16, w=fake, wb=256):
        return lib.attn_weight_grad(A, G, g, n, d, heads, batch, wu, dt, w, wb, None)

    for f in (proj, grad):
        assert f(A=None) == B.ATTN_ERR_NULL
        assert f(n=0) == B.ATTN_ERR_SHAPE
        assert f(d=12) == B.ATTN_ERR_SHAPE
        assert f(d=264) == B.ATTN_ERR_SHAPE
        assert f(wu=3) == B.ATTN_ERR_SHAPE            # neither 1, heads nor batch * heads
        assert f(wu=0) == B.ATTN_ERR_SHAPE
        assert f(dt=5) == B.ATTN_ERR_DTYPE
        assert f(w=None) == B.ATTN_ERR_WORKSPACE
        assert f(wb=16) == B.ATTN_ERR_WORKSPACE
        assert f(w=fake + 16) == B.ATTN_ERR_ALIGN
        assert f(A=fake + 8) == B.ATTN_ERR_ALIGN
    assert proj(out=None) == B.ATTN_ERR_NULL
    assert grad(g=None) == B.ATTN_ERR_NULL

    def wbwd(gX=fake, gY=fake, A3=fake, wb=1 << 30, wu=2, cfg=None, dt=B.ATTN_BF16):
        return lib.attn_weights_bwd(fake, fake, A3, fake, fake, fake, fake, fake, gX, gY, 128, 64, 2, 3, wu, None, dt,
                                    0.0, cfg, fake, wb, None)

    assert wbwd(gX=None) == B.ATTN_ERR_NULL
    assert wbwd(A3=None) == B.ATTN_ERR_NULL           # gY wanted but no A3
    assert wbwd(wu=5) == B.ATTN_ERR_SHAPE
    assert wbwd(wb=4096) == B.ATTN_ERR_WORKSPACE
    bad_tile = B.CCfg(48, 0, 0, B.ATTN_ALGO_SIMT, 0)
    assert wbwd(cfg=ctypes.byref(bad_tile)) == B.ATTN_ERR_TILE
    need = B.attn_weights_bwd_workspace_bytes(128, 64, 2, 3, None, B.ATTN_BF16, None)
    inner = B.attn_bwd_workspace_bytes(128, 64, 2, 3, None, B.ATTN_BF16, None)
    assert need >= inner + 3 * 128 * 64 * 6 * 2
    assert B.attn_weights_bwd_workspace_bytes(0, 64, 2, 3, None, B.ATTN_BF16, None) == 0

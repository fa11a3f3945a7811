"""The host-side replay of the kernels' tilings (attn_io_replay) against closed forms and against the
paper's lower bound (Theorem 1.1) at the CTA's on-chip size.  No GPU needed: the replay is host arithmetic."""
import pytest

from paper_2410_09397_b200 import binding as B

NONE, CAUSAL = B.ATTN_MASK_NONE, B.ATTN_MASK_CAUSAL


def fused(tile_q=0, det=0):
    return B.Cfg(tile_q=tile_q, algo=B.ATTN_ALGO_FUSED, deterministic=det)


@pytest.mark.parametrize("n,d", [(1024, 128), (4096, 64), (2048, 128)])
def test_forward_replay_equals_the_query_stationary_closed_form(n, d):
    r = B.attn_io_replay(n, d, NONE, B.ATTN_BF16, fused(), False)
    nt = n // 128
    assert r["loads"] == n * d + nt * 2 * n * d          # every query tile streams all of K and V
    assert r["stores"] == n * d + n and r["reductions"] == 0
    rc = B.attn_io_replay(n, d, CAUSAL, B.ATTN_BF16, fused(), False)
    assert rc["loads"] == n * d + 2 * 128 * d * nt * (nt + 1) // 2


@pytest.mark.parametrize("n,d", [(1024, 128), (2048, 64)])
def test_fused_backward_replay_equals_the_key_stationary_closed_form(n, d):
    r = B.attn_io_replay(n, d, NONE, B.ATTN_BF16, fused(), True)
    nt = n // 128
    pre_loads, pre_stores = 2 * n * d + n + n * d, 2 * n + 2 * n * d      # D pre-pass + clear, conversion
    assert r["loads"] == pre_loads + 2 * n * d + nt * (2 * n * d + 2 * n)
    assert r["stores"] == pre_stores + 2 * n * d
    assert r["reductions"] == nt * n * d
    rc = B.attn_io_replay(n, d, CAUSAL, B.ATTN_BF16, fused(), True)
    pairs = nt * (nt + 1) // 2
    assert rc["reductions"] == pairs * 128 * d
    assert rc["loads"] == pre_loads + 2 * n * d + pairs * (2 * 128 * d + 2 * 128)


def test_ragged_sizes_count_rows_not_tiles():
    n, d = 200, 128     # tiles of 128 + 72 rows
    r = B.attn_io_replay(n, d, NONE, B.ATTN_BF16, fused(), False)
    assert r["loads"] == n * d + 2 * (2 * n * d)
    assert r["stores"] == n * d + n


def test_io_falls_as_the_tile_grows_and_never_undercuts_the_bound():
    """Section 3.3 / Theorem 1.1: a larger cache (tile) means less I/O, and no tiling beats the bound."""
    n = 8192
    for d in (128, 256):
        rows = []
        for cfg in B.attn_supported_cfgs(d, B.ATTN_BF16):
            if cfg.algo == B.ATTN_ALGO_SIMT:
                continue
            try:
                r = B.attn_io_replay(n, d, NONE, B.ATTN_BF16, cfg, True)
            except B.AttnError:
                continue                      # forward-only shape
            M = B.attn_cfg_onchip_elems(d, B.ATTN_BF16, cfg, True)
            bound = B.attn_io_bound_elems(n, d, M, True)
            assert r["total"] >= bound, (d, cfg, r, bound)
            rows.append((cfg.algo, cfg.tile_q, cfg.tile_k, M, r["total"]))
        fused_rows = sorted((m, t) for a, _, _, m, t in rows if a == B.ATTN_ALGO_FUSED)
        # key-stationary tilings: the I/O is set by the key tile (the stationary dK, dV, K, V), so the query-tile
        # size changes M but not the count -- more on-chip memory never costs I/O
        for (m0, t0), (m1, t1) in zip(fused_rows, fused_rows[1:]):
            assert m1 > m0 and t1 <= t0, fused_rows
        # blocked tilings of the small-cache algorithm: the I/O falls along either edge of the block
        mat = {(tq, tk): t for a, tq, tk, _, t in rows if a == B.ATTN_ALGO_MATERIALIZED}
        assert set(mat) == {(tq, tk) for tq in (128, 256) for tk in (32, 64, 128)}
        for tq in (128, 256):
            assert mat[tq, 32] > mat[tq, 64] > mat[tq, 128], mat
        for tk in (32, 64, 128):
            assert mat[128, tk] > mat[256, tk], mat
        # at every d the fused (large-cache) tilings move less than the materialised (small-cache) ones
        assert max(t for _, t in fused_rows) < min(mat.values())


def test_materialised_replay_counts_the_n_by_n_round_trips():
    n, d, tk = 1024, 256, 64
    r = B.attn_io_replay(n, d, NONE, B.ATTN_BF16, B.Cfg(tile_k=tk, algo=B.ATTN_ALGO_MATERIALIZED), True)
    tiles = (n // 128) * (n // tk)
    gemm12 = 2 * tiles * (128 + tk) * d           # phases 1, 2: operand rows of every 128 x tk block
    gemm4 = 3 * (n // 256) * (256 + d) * n        # phase 4: three products with contraction n, 256 x d tiles
    assert r["loads"] == (2 * n * d + n) + gemm12 + 2 * n * n + gemm4
    assert r["stores"] == 2 * n + 2 * n * n + n * n + 3 * n * d


def test_materialised_replay_beyond_the_kernels_head_sizes_reaches_the_small_cache_regime():
    """d = 512 and 1024 are replayed although no kernel runs them: there a block of 128 x 32 (65,536 elements) is
    smaller than d^2, the I/O still never undercuts the bound, and the bound's active branch is n^2 d / sqrt(M)."""
    n = 4096
    for d in (512, 1024):
        cfg = B.Cfg(tile_q=128, tile_k=32, algo=B.ATTN_ALGO_MATERIALIZED)
        r = B.attn_io_replay(n, d, NONE, B.ATTN_BF16, cfg, True)
        M = B.attn_cfg_onchip_elems(256, B.ATTN_BF16, cfg, True)
        assert M < d * d
        small, large = (n * n * d + n * d * d) / M ** 0.5, (n * n * d * d + n * d ** 3) / M
        assert small < large and B.attn_io_bound_elems(n, d, M, True) == pytest.approx(small)
        assert r["total"] >= small
        tiles = (n // 128) * (n // 32)
        assert r["loads"] == (2 * n * d + n) + 2 * tiles * (128 + 32) * d + 2 * n * n + 3 * (n // 256) * (256 + d) * n
    with pytest.raises(B.AttnError):
        B.attn_io_replay(n, 512, NONE, B.ATTN_BF16, fused(), True)       # the fused tilings exist for d <= 256 only


def test_replay_rejects_what_it_cannot_replay():
    with pytest.raises(B.AttnError):
        B.attn_io_replay(1024, 128, B.ATTN_MASK_BLOCK_SPARSE, B.ATTN_BF16, fused(), True)
    with pytest.raises(B.AttnError):
        B.attn_io_replay(1024, 128, NONE, B.ATTN_F32, None, True)
    with pytest.raises(B.AttnError):
        B.attn_io_replay(1024, 256, NONE, B.ATTN_BF16, fused(tile_q=128), True)

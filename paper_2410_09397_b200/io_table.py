"""Prints the I/O-versus-cache-size table of the library's tilings (the data behind Figure 1 of the paper).

    python -m paper_2410_09397_b200.io_table [--n 8192] [--causal]

For every head dimension and every tile configuration the backward accepts: the CTA's on-chip size M
(elements), the elements one head moves across the SM boundary when the kernels' loop nests are replayed
(``attn_io_replay``), the two branches of Theorem 1.1 at that M, and the ratio to the bound.  Host arithmetic
only; needs the built library but no GPU.
"""
from __future__ import annotations

import argparse

from . import binding as B


def rows(n: int, causal: bool):
    mk = B.ATTN_MASK_CAUSAL if causal else B.ATTN_MASK_NONE
    half = 0.5 if causal else 1.0
    names = {B.ATTN_ALGO_FUSED: "fused", B.ATTN_ALGO_MATERIALIZED: "materialised"}
    for d in (64, 128, 256, 512, 1024):
        # d = 512, 1024: replay only (no kernel runs them); the materialised blocks are those of d = 256
        for cfg in B.attn_supported_cfgs(min(d, 256), B.ATTN_BF16):
            if d > 256 and cfg.algo != B.ATTN_ALGO_MATERIALIZED:
                continue
            if cfg.algo not in names:
                continue
            for det in ((0, 1) if cfg.algo == B.ATTN_ALGO_FUSED else (0,)):
                c = B.Cfg(cfg.tile_q, cfg.tile_k, cfg.tile_d, cfg.algo, det)
                try:
                    r = B.attn_io_replay(n, d, mk, B.ATTN_BF16, c, True)
                except B.AttnError:
                    continue
                M = B.attn_cfg_onchip_elems(min(d, 256), B.ATTN_BF16, c, True)
                large = (n * n * d * d + n * d ** 3) / M * half
                small = (n * n * d + n * d * d) / M ** 0.5 * half
                yield {"d": d, "algo": names[cfg.algo] + (" (no atomics)" if det else ""), "tile_q": cfg.tile_q,
                       "tile_k": cfg.tile_k, "M": M, "regime": "large (M >= d^2)" if M >= d * d else "small (M < d^2)",
                       "replay": r["total"], "loads": r["loads"], "stores": r["stores"], "reductions": r["reductions"],
                       "bound_large": large, "bound_small": small, "ratio": r["total"] / min(large, small)}


def main():
    ap = argparse.ArgumentParser()
    ap.add_argument("--n", type=int, default=8192)
    ap.add_argument("--causal", action="store_true")
    a = ap.parse_args()
    print(f"backward, one head, n = {a.n}, {'causal' if a.causal else 'no mask'}; elements")
    print("| d | algorithm | tile_q x tile_k | M | regime | replayed I/O | n^2d^2/M branch | n^2d/sqrt(M) branch | I/O / bound |")
    print("|---|---|---|---|---|---|---|---|---|")
    for r in rows(a.n, a.causal):
        print(f"| {r['d']} | {r['algo']} | {r['tile_q']} x {r['tile_k']} | {r['M']} | {r['regime']} | {r['replay']:.3e} | "
              f"{r['bound_large']:.3e} | {r['bound_small']:.3e} | {r['ratio']:.1f} |")


if __name__ == "__main__":
    main()

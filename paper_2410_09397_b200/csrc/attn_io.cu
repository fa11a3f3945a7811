// Host-side replay of the kernels' loop nests: counts the elements every CTA moves across
// the SM boundary (TMA loads, stores, fp32 reductions) for one head.  In the paper's
// two-level model (Section 3.3) the cache is what one CTA holds on chip -- shared memory plus
// tensor memory, attn_cfg_onchip_elems() -- and everything behind it (L2, device memory) is
// "memory", so this count is the I/O of the tiling that Theorem 1.1 bounds from below.  The
// loops below visit exactly the tiles the kernels visit, in the same order; nothing here is a
// closed form (the tests compare the replay with closed forms).
#include "attn_internal.h"

namespace attn {
namespace {

struct Count {
    double loads = 0, stores = 0, reductions = 0;
    void add(const Count &o) { loads += o.loads; stores += o.stores; reductions += o.reductions; }
};

int rows_of(int n, int tile, int idx) { return n - idx * tile < tile ? n - idx * tile : tile; }

// query tiles of `tq` rows that a key tile of 128 keys starting at j0 visits (key-stationary kernels)
template <class F> void for_query_tiles(int n, int tq, int jt, int causal, F f)
{
    const int nt = (n + tq - 1) / tq;
    for (int it = causal ? jt * (128 / tq) : 0; it < nt; ++it) f(it);
}

// key-stationary backward: tile_q in {128, 64}; `split` CTAs per key tile each owning d / split columns of
// dK, dV and dQ^T; with_dq = 0 for the kernel without the dQ product
Count key_stationary(int n, int d, int causal, int tq, int split, int with_dq)
{
    Count c;
    const int nk = (n + 127) / 128, ha = d / split;
    for (int jt = 0; jt < nk; ++jt)
        for (int s = 0; s < split; ++s) {
            const double rk = rows_of(n, 128, jt);
            c.loads += 2 * rk * d;                                   // K_j, V_j
            for_query_tiles(n, tq, jt, causal, [&](int it) {
                const double rq = rows_of(n, tq, it);
                c.loads += 2 * rq * d + 2 * rq;                      // Q_i, dO_i, -LSE log2e, scale D
                if (with_dq) c.reductions += rq * ha;                // dQ^T tile, fp32
            });
            c.stores += 2 * rk * ha;                                 // dK_j, dV_j
        }
    return c;
}

// query-stationary kernels (forward: stores O and LSE; dQ kernel: loads dO and the row statistics too)
Count query_stationary(int n, int d, int causal, int tk, int backward)
{
    Count c;
    const int nq = (n + 127) / 128, nkt = (n + tk - 1) / tk;
    for (int it = 0; it < nq; ++it) {
        const double rq = rows_of(n, 128, it);
        c.loads += (backward ? 2 : 1) * rq * d + (backward ? 2 * rq : 0);
        const int last = causal ? ((it * 128 + (int)rq - 1) / tk) : nkt - 1;
        for (int jt = 0; jt <= last && jt < nkt; ++jt) c.loads += 2.0 * rows_of(n, tk, jt) * d;   // K_j, V_j
        c.stores += rq * d + (backward ? 0 : rq);
    }
    return c;
}

// D pre-pass (+ clearing the fp32 accumulator) and the conversion of the accumulator to dQ
Count prepass(int n, int d, int with_acc)
{
    Count c;
    c.loads = 2.0 * n * d + n;
    c.stores = 2.0 * n + (with_acc ? (double)n * d : 0);
    if (with_acc) { c.loads += (double)n * d; c.stores += (double)n * d; }
    return c;
}

// blocked GEMM of the materialised path: C (m x nn) in bm x bn tiles, contraction of length k
Count gemm(double m, double nn, double k, int bm, int bn)
{
    Count c;
    const int tm = (int)((m + bm - 1) / bm), tn = (int)((nn + bn - 1) / bn);
    for (int i = 0; i < tm; ++i)
        for (int j = 0; j < tn; ++j) {
            const double rm = m - i * bm < bm ? m - i * bm : bm, rn = nn - j * bn < bn ? nn - j * bn : bn;
            c.loads += (rm + rn) * k;
            c.stores += rm * rn;
        }
    return c;
}

}  // namespace
}  // namespace attn

using namespace attn;

extern "C" attn_status attn_io_replay(int n, int d, int mask_kind, int dt, const attn_cfg *cfg, int backward,
                                      attn_io_count *out)
{
    if (!out) return ATTN_ERR_NULL;
    if (n < 1 || (dt != ATTN_BF16 && dt != ATTN_F32)) return ATTN_ERR_SHAPE;
    if (mask_kind != ATTN_MASK_NONE && mask_kind != ATTN_MASK_CAUSAL) return ATTN_ERR_MASK;
    attn_cfg c{};
    if (cfg) c = *cfg;
    if (c.algo == ATTN_ALGO_AUTO) c.algo = dt == ATTN_BF16 ? ATTN_ALGO_FUSED : ATTN_ALGO_SIMT;
    if (c.algo == ATTN_ALGO_SIMT) return ATTN_ERR_TILE;      // the fp32 FMA kernels are not tiled for a cache size
    if (c.algo == ATTN_ALGO_MATERIALIZED && !backward) { c.algo = ATTN_ALGO_FUSED; c.tile_q = c.tile_k = c.tile_d = 0; }
    // the blocked loop nest of the materialised backward is the same for every head dimension: it can be replayed for
    // d = 512 or 1024 as well (multiples of 64), where its blocks hold fewer than d^2 elements -- the small-cache side
    // of Theorem 1.1 -- although no kernel of the library runs those sizes
    const bool replay_only = c.algo == ATTN_ALGO_MATERIALIZED && backward && d > 256 && d <= 1024 && d % 64 == 0 &&
                             mat_cfg_supported(256, c);
    if (!replay_only && !tc_cfg_supported(d, c, backward)) {
        if (!(c.algo == ATTN_ALGO_FUSED && !backward && tc_cfg_supported(d, c, 1))) return ATTN_ERR_TILE;
        c.tile_q = c.tile_k = c.tile_d = 0;
    }
    const int causal = mask_kind == ATTN_MASK_CAUSAL;
    Count r;
    if (!backward) {
        r = query_stationary(n, d, causal, d == 256 ? 64 : 128, 0);
    } else if (c.algo == ATTN_ALGO_MATERIALIZED) {
        const int tk = c.tile_k ? c.tile_k : 128, tq = c.tile_q ? c.tile_q : 128;
        r = prepass(n, d, 0);
        r.add(gemm(n, n, d, tq, tk));                                // phase 1: P
        r.add(gemm(n, n, d, tq, tk));                                // phase 2: dP
        r.loads += 2.0 * n * n; r.stores += (double)n * n;           // phase 3: dS from P, dP
        for (int i = 0; i < 3; ++i) r.add(gemm(n, d, n, 256, d));    // phase 4: dV, dK, dQ in 256 x d tiles
    } else if (c.deterministic) {
        r = prepass(n, d, 0);
        r.add(key_stationary(n, d, causal, 128, 1, 0));
        r.add(query_stationary(n, d, causal, 128, 1));
    } else {
        const int tq = (c.tile_q == 64 || d == 256) ? 64 : 128;
        r = prepass(n, d, 1);
        r.add(key_stationary(n, d, causal, tq, d == 256 ? 2 : 1, 1));
    }
    out->loads = r.loads; out->stores = r.stores; out->reductions = r.reductions;
    return ATTN_OK;
}

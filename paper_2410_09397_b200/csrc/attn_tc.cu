// Which tile configurations the tensor-core algorithms accept, and how much on-chip
// memory (shared memory + tensor memory) a CTA of each holds.
#include "attn_internal.h"

namespace attn {

// Fused forward: 128 queries x (128 keys for d <= 128, 64 keys for d = 256).
// Fused backward (key tiles of 128): 128 queries per step for d = 64, 128 (the default there), or 64
// queries per step for d = 128 and 256.  At d = 256 the dK and dV accumulators of a key tile would fill
// tensor memory, so two CTAs share a key tile, each owning 128 columns of the head dimension; that shape
// has no variant without atomics.
bool tc_cfg_supported(int d, const attn_cfg &c, int backward)
{
    if (d != 64 && d != 128 && d != 256) return false;
    if (c.algo == ATTN_ALGO_FUSED) {
        if (c.tile_d != 0 && c.tile_d != d) return false;
        if (backward) {
            if (c.tile_k != 0 && c.tile_k != 128) return false;
            if (c.tile_q == 64) return d != 64 && !c.deterministic;
            if (c.tile_q == 0 && d == 256) return !c.deterministic;
            return d != 256 && (c.tile_q == 0 || c.tile_q == 128);
        }
        if (c.tile_q != 0 && c.tile_q != 128) return false;
        const int tk = d == 256 ? 64 : 128;
        return c.tile_k == 0 || c.tile_k == tk;
    }
    if (c.algo == ATTN_ALGO_MATERIALIZED) return backward && mat_cfg_supported(d, c);
    return false;
}

size_t tc_cfg_onchip_bytes(int d, const attn_cfg &c, int backward)
{
    if (!tc_cfg_supported(d, c, backward)) return 0;
    if (c.algo == ATTN_ALGO_MATERIALIZED) return mat_onchip_bytes(d, c);
    // tensor memory: 128 lanes x 4 bytes per column
    if (backward && (c.tile_q == 64 || d == 256))   // 64-query tiles: dV, dK (128 columns each), S^T / P^T, dP^T / dQ^T, V_j at d = 256
        return bwd64_smem_bytes(d) + (size_t)(256 + 128 + (d == 256 ? 128 : 0)) * 128 * 4;
    // regions A and B, dK_j and dV_j; d = 64: a second region for dP^T in the columns that would otherwise stay free
    if (backward) return bwd_smem_bytes(d) + (size_t)(256 + 2 * d + (d == 64 ? 128 : 0)) * 128 * 4;
    return fwd_smem_bytes(d) + (size_t)(256 + d) * 128 * 4;
}

}  // namespace attn

// Tensor-core (tcgen05 / TMEM / TMA) path -- placeholder until the kernels land.
#include "attn_internal.h"

namespace attn {
bool tc_cfg_supported(int, const attn_cfg &, int) { return false; }
size_t tc_cfg_onchip_bytes(int, const attn_cfg &, int) { return 0; }
attn_status tc_fwd(const Problem &) { return ATTN_ERR_TILE; }
attn_status tc_bwd(const Problem &) { return ATTN_ERR_TILE; }
attn_status mat_bwd(const Problem &) { return ATTN_ERR_TILE; }
}  // namespace attn

// Materialised (small-cache) backward -- placeholder until the kernels land.
#include "attn_internal.h"

namespace attn {
bool mat_cfg_supported(int, const attn_cfg &) { return false; }
size_t mat_onchip_bytes(int, const attn_cfg &) { return 0; }
attn_status mat_bwd(const Problem &) { return ATTN_ERR_TILE; }
}  // namespace attn

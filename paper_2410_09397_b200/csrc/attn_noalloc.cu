// attn_bwd_noalloc: the backward pass for callers that cannot allocate device memory.
//
// attn_bwd needs scratch memory (the status word, D = rowsum(dO o O) and, for the fused
// algorithm, the fp32 dQ accumulator) and asks its caller to pass it in.  Some callers
// have no way to get such a buffer at the moment of the call: code running inside a
// region where cudaMalloc is forbidden (a memory pool that has been frozen, a real-time
// loop, a plug-in that was handed tensors but no allocator).  For them the scratch
// lives here, in a fixed array that is part of the library image.
#include "attn_internal.h"

namespace {

constexpr size_t kScratchBytes = size_t(8) << 20;   // ATTN_NOALLOC_SCRATCH_BYTES

// One copy per GPU that loads the library, held until the process exits.
static __device__ __align__(256) unsigned char g_scratch[kScratchBytes];

constexpr int kMaxDevices = 64;
void *g_scratch_addr[kMaxDevices] = {};

// The array's name is only a host-side handle; kernels need its device address, which
// differs per device.  Looked up once per device, with that device current.
attn_status scratch_for_current_device(void **out)
{
    int dev = -1;
    if (cudaGetDevice(&dev) != cudaSuccess || dev < 0 || dev >= kMaxDevices) return ATTN_ERR_ARCH;
    if (!g_scratch_addr[dev]) {
        void *p = nullptr;
        if (cudaGetSymbolAddress(&p, g_scratch) != cudaSuccess || !p) return ATTN_ERR_LAUNCH;
        g_scratch_addr[dev] = p;
    }
    *out = g_scratch_addr[dev];
    return ATTN_OK;
}

}  // namespace

extern "C" {

size_t attn_noalloc_scratch_bytes(void) { return kScratchBytes; }

// The status word of the last attn_bwd_noalloc call on the current device is the first word of the
// array: copied out with a plain device-to-host copy (no allocation), after `cuda_stream` has drained.
attn_status attn_noalloc_status(void *cuda_stream)
{
    void *scratch = nullptr;
    const attn_status st = scratch_for_current_device(&scratch);
    if (st != ATTN_OK) return st;
    return attn_workspace_status(scratch, cuda_stream);
}

attn_status attn_bwd_noalloc(const void *Q, const void *K, const void *V, const void *O, const void *dO,
                             const float *LSE, void *dQ, void *dK, void *dV, int n, int d, int heads, int batch,
                             const attn_mask *mask, int dt, float scale, const attn_cfg *cfg, void *cuda_stream)
{
    const size_t need = attn_bwd_workspace_bytes(n, d, heads, batch, mask, dt, cfg);
    if (need > kScratchBytes) return ATTN_ERR_WORKSPACE;   // problem too large for the built-in scratch
    void *scratch = nullptr;
    // need == 0 means invalid arguments: let attn_bwd name the error (it checks them before touching memory)
    const attn_status st = scratch_for_current_device(&scratch);
    if (st != ATTN_OK) return st;
    return attn_bwd(Q, K, V, O, dO, LSE, dQ, dK, dV, n, d, heads, batch, mask, dt, scale, cfg, scratch, kScratchBytes,
                    cuda_stream);
}

}  // extern "C"

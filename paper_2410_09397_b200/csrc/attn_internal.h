// Internal declarations shared by the translation units of libattn_b200.
#pragma once
#include <cuda_runtime.h>
#include <stddef.h>
#include <stdint.h>

#include "attn.h"

namespace attn {

// A block mask whose blocks are finer than the 128 x 128 tiles of the tensor-core kernels (block edge 32 or
// 64): the kernels then walk lists of 128 x 128 super-blocks that keep at least one fine block, and drop the
// entries of the fine blocks that are not kept inside every visited tile.  block == 0: not in use.
struct FineMask {
    const uint8_t *bits;   // the caller's mask [mask_heads][nb][nb]
    int block, nb;
};
#ifdef __CUDACC__
// (i, j) < n; which of the caller's masks: head bh unless one mask serves all
__device__ __forceinline__ bool fine_keep(const FineMask &f, int mask_heads, long bh, int i, int j)
{
    const uint8_t *m = f.bits + (mask_heads == 1 ? 0 : (size_t)bh * f.nb * f.nb);
    return m[(size_t)(i / f.block) * f.nb + j / f.block] != 0;
}
#endif

// One fully validated problem, as handed from the C ABI to the kernel launchers.
struct Problem {
    const void *Q, *K, *V, *O, *dO;   // inputs (O, dO only for the backward)
    const float *LSE;                 // backward input
    void *Oout;                       // forward outputs
    float *LSEout;
    void *dQ, *dK, *dV;               // backward outputs
    int n, d, heads, batch;
    long BH;                          // batch * heads
    int mask_kind, block, mask_heads, nb;
    const uint8_t *block_mask;
    FineMask fine;                    // tensor-core algorithms with a block edge below 128: block / nb then describe the super-blocks
    int dt;
    float scale;
    attn_cfg cfg;                     // resolved: algo and tiles are final
    // workspace sections (device)
    uint32_t *status;                 // 4-byte status word
    float *D;                         // [BH * n]
    float *nLSE2;                     // [BH * n]: -LSE * log2(e), fused backward only
    int *row_ptr, *col_idx;           // block-CSR of the mask: [mask_heads][nb+1], [mask_heads][nb*nb]
    int *col_ptr, *row_idx;           // block-CSC
    float *dQ_acc;                    // fp32 dQ accumulator [BH * n * d] (fused backward with atomics)
    void *matP, *matdP, *matdS;       // materialised n x n buffers (per head chunk)
    int mat_heads;                    // heads materialised at once
    cudaStream_t stream;
};

struct WorkspaceLayout {
    size_t status, D, nLSE2, row_ptr, col_idx, col_ptr, row_idx, dQ_acc, matP, matdP, matdS, total;
    int mat_heads;
};

// Every kernel launch goes between these two calls (launch counter + optional event timing).
void launch_begin(const char *name, cudaStream_t s);
void launch_end(cudaStream_t s);

inline size_t align_up(size_t x, size_t a) { return (x + a - 1) / a * a; }

// mask kinds: "block" = described by a block mask, "causal" = entries with j > i are dropped
__host__ __device__ inline bool mask_is_block(int kind) { return kind == ATTN_MASK_BLOCK_SPARSE || kind == ATTN_MASK_BLOCK_SPARSE_CAUSAL; }
__host__ __device__ inline bool mask_is_causal(int kind) { return kind == ATTN_MASK_CAUSAL || kind == ATTN_MASK_BLOCK_SPARSE_CAUSAL; }

// Streaming multiprocessors of the current device (grid sizing of the grid-stride and persistent kernels).
int sm_count();

// SIMT fp32 path (attn_simt.cu)
attn_status simt_fwd(const Problem &p);
attn_status simt_bwd(const Problem &p);
attn_status preprocess_D(const void *O, const void *dO, float *D, size_t rows, int d, int dt, cudaStream_t s);
attn_status build_block_index(const Problem &p);

// Tensor-core path (attn_tc_*.cu)
attn_status tc_fwd(const Problem &p);
attn_status tc_bwd(const Problem &p);
attn_status tc_bwd_dq(const Problem &p);   // query-stationary dQ without atomics (needs p.D = scale*D, p.nLSE2)
attn_status mat_bwd(const Problem &p);
bool tc_cfg_supported(int d, const attn_cfg &cfg, int backward);
size_t tc_cfg_onchip_bytes(int d, const attn_cfg &cfg, int backward);
size_t fwd_smem_bytes(int d);
size_t bwd_smem_bytes(int d);
size_t bwd64_smem_bytes(int d);            // fused backward with 64-query tiles
attn_status tc_bwd64(const Problem &p);
bool mat_cfg_supported(int d, const attn_cfg &cfg);
size_t mat_onchip_bytes(int d, const attn_cfg &cfg);

}  // namespace attn

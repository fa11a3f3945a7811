// Internal declarations shared by the translation units of libattn_b200.
#pragma once
#include <cuda_runtime.h>
#include <stddef.h>
#include <stdint.h>

#include "attn.h"

namespace attn {

// Masks finer than the 128 x 128 tiles of the tensor-core kernels.  The kernels walk lists of the tiles that keep
// anything and drop the other entries inside every visited tile:
//   mode 1: a block mask with a block edge of 32 or 64 (`bits`, the caller's mask [mask_heads][nb][nb]);
//   mode 2: an element mask, one bit per score entry: `rowbits` [mask_heads][n][words] has bit j % 32 of word
//           j / 32 of row i set iff (i, j) is kept (the caller's bitmap), `colbits` is its transpose (row j, bit i),
//           built in the workspace for the key-stationary kernels.
struct FineMask {
    int mode;              // 0: not in use
    const uint8_t *bits;   // mode 1
    int block, nb;
    const uint32_t *rowbits, *colbits;   // mode 2
    int n, words;
};
#ifdef __CUDACC__
// Keep bits of the 32 entries (r, c0 .. c0 + 31), c0 a multiple of 32, r < n, c0 < n.  by_query: r is a query
// row and the columns are keys; otherwise r is a key row and the columns are queries.
__device__ __forceinline__ uint32_t fine_word(const FineMask &f, int mask_heads, long bh, bool by_query, int r, int c0)
{
    const size_t mh = mask_heads == 1 ? 0 : (size_t)bh;
    if (f.mode == 2) return (by_query ? f.rowbits : f.colbits)[(mh * f.n + r) * f.words + c0 / 32];
    // mode 1: 32 aligned columns lie in one block (block edge 32 or 64)
    const int i = by_query ? r : c0, j = by_query ? c0 : r;
    return f.bits[mh * f.nb * f.nb + (size_t)(i / f.block) * f.nb + j / f.block] != 0 ? 0xffffffffu : 0u;
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
    FineMask fine;                    // tensor-core algorithms with a mask finer than their tiles: block / nb / block_mask then describe the 128 x 128 tiles
    int dt;
    float scale;
    attn_cfg cfg;                     // resolved: algo and tiles are final
    // workspace sections (device)
    uint32_t *status;                 // 4-byte status word
    float *D;                         // [BH * n]
    float *nLSE2;                     // [BH * n]: -LSE * log2(e), fused backward only
    int *row_ptr, *col_idx;           // block-CSR of the mask: [mask_heads][nb+1], [mask_heads][nb*nb]
    int *col_ptr, *row_idx;           // block-CSC
    uint8_t *tilemask;                // element mask: which 128 x 128 tiles keep anything [mask_heads][nb][nb]
    uint32_t *colbits;                // element mask: the transposed bitmap
    float *dQ_acc;                    // fp32 dQ accumulator [BH * n * d] (fused backward with atomics)
    void *matP, *matdP, *matdS;       // materialised n x n buffers (per head chunk)
    int mat_heads;                    // heads materialised at once
    cudaStream_t stream;
};

struct WorkspaceLayout {
    size_t status, D, nLSE2, row_ptr, col_idx, col_ptr, row_idx, tilemask, colbits, dQ_acc, matP, matdP, matdS, total;
    int mat_heads;
};

// Every kernel launch goes between these two calls (launch counter + optional event timing).
void launch_begin(const char *name, cudaStream_t s);
void launch_end(cudaStream_t s);

inline size_t align_up(size_t x, size_t a) { return (x + a - 1) / a * a; }

// mask kinds: "block" = described by a block mask, "causal" = entries with j > i are dropped
__host__ __device__ inline bool mask_is_block(int kind) { return kind == ATTN_MASK_BLOCK_SPARSE || kind == ATTN_MASK_BLOCK_SPARSE_CAUSAL; }
__host__ __device__ inline bool mask_is_element(int kind) { return kind == ATTN_MASK_ELEMENT; }
__host__ __device__ inline bool mask_is_causal(int kind) { return kind == ATTN_MASK_CAUSAL || kind == ATTN_MASK_BLOCK_SPARSE_CAUSAL; }

// Streaming multiprocessors of the current device (grid sizing of the grid-stride and persistent kernels).
int sm_count();

// SIMT fp32 path (attn_simt.cu)
attn_status simt_fwd(const Problem &p);
attn_status simt_bwd(const Problem &p);
attn_status preprocess_D(const void *O, const void *dO, float *D, size_t rows, int d, int dt, cudaStream_t s);
attn_status build_block_index(const Problem &p);

// attn_bwd for a caller inside the library that consumes dQ itself (the weight gradients).  With `keep_acc` set and an
// algorithm that accumulates dQ in fp32 in the workspace, the conversion to the storage type is skipped, dQ is left
// untouched and *dQ_acc receives the accumulator's address ([batch * heads][n][d], final values); in every other case
// dQ is written as attn_bwd writes it and *dQ_acc is nullptr.
attn_status bwd_internal(const void *Q, const void *K, const void *V, const void *O, const void *dO, const float *LSE,
                         void *dQ, void *dK, void *dV, int n, int d, int heads, int batch, const attn_mask *mask, int dt,
                         float scale, const attn_cfg *cfg, void *workspace, size_t workspace_bytes, void *cuda_stream,
                         bool keep_acc, const float **dQ_acc);

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

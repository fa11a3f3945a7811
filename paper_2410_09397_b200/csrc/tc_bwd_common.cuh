// Device helpers shared by the key-stationary backward kernels (128-query and 64-query tiles):
// kernel arguments, the enumeration of the query tiles a key tile visits, small PTX wrappers,
// the D pre-pass and the fp32 -> bf16 conversion of the dQ accumulator.
#pragma once
#include "attn_internal.h"
#include "tc_common.cuh"

namespace attn {
namespace bwdk {

using namespace tc;

constexpr int TK = 128;                 // keys per CTA
constexpr uint32_t SLAB = 128 * 128;   // bytes of one [128 rows][64 bf16] slab
struct BwdArgs {
    const float *nLSE2, *Ds;   // -LSE log2(e) and scale * D per row (workspace)
    float *dQ_acc;
    __nv_bfloat16 *dK, *dV;
    int n, BH;
    int mask_kind, block, nb, mask_heads;
    const int *col_ptr, *row_idx;   // block-CSC of the mask
    float scale;
    int group;                 // heads per launch group (divides BH)
    FineMask fine;             // a mask finer than the tiles: dropped entries are masked inside the visited tiles
    uint32_t *status;
};


// Enumerates the query tiles (of TQT queries) a key tile jt (128 keys) has to visit.
template <int TQT>
struct TileIterT {
    int kind, n, jt, sub, raw;
    const int *rows;   // block rows kept in this block column
    __device__ TileIterT(const BwdArgs &a, int jt_, long bh) : kind(a.mask_kind), n(a.n), jt(jt_), sub(1), raw(0), rows(nullptr)
    {
        constexpr int R = TK / TQT;   // query tiles per key tile's worth of rows
        const int nt = (n + TQT - 1) / TQT;
        if (kind == ATTN_MASK_NONE) raw = nt;
        else if (kind == ATTN_MASK_CAUSAL) raw = nt > jt * R ? nt - jt * R : 0;
        else {
            sub = a.block / TQT;
            const int J = jt / (a.block / TK);
            const long mh = a.mask_heads == 1 ? 0 : bh;
            const int *cp = a.col_ptr + mh * 2 * a.nb + 2 * J;
            rows = a.row_idx + mh * (long)a.nb * a.nb + cp[0];
            raw = (cp[1] - cp[0]) * sub;
        }
    }
    // query tile of raw index idx, or -1 if that tile lies beyond n
    __device__ int tile(int idx) const
    {
        int it;
        if (kind == ATTN_MASK_NONE) it = idx;
        else if (kind == ATTN_MASK_CAUSAL) it = jt * (TK / TQT) + idx;
        else {
            it = rows[idx / sub] * sub + idx % sub;
            // block mask AND causal: a query tile that ends before the key tile begins keeps nothing
            if (kind == ATTN_MASK_BLOCK_SPARSE_CAUSAL && (it + 1) * TQT <= jt * TK) return -1;
        }
        return it * TQT < n ? it : -1;
    }
};

__device__ __forceinline__ void bulk_load_1d(void *dst, const void *src, uint32_t bytes, uint64_t *bar)
{
    asm volatile("cp.async.bulk.shared::cluster.global.mbarrier::complete_tx::bytes [%0], [%1], %2, [%3];"
                 ::"r"(smem_u32(dst)), "l"(reinterpret_cast<uint64_t>(src)), "r"(bytes), "r"(smem_u32(bar))
                 : "memory");
}
__device__ __forceinline__ void red_add_f32(float *p, float v)
{
    asm volatile("red.global.add.f32 [%0], %1;" ::"l"(p), "f"(v) : "memory");
}

__device__ __forceinline__ float ex2_approx(float x)
{
    float y;
    asm("ex2.approx.ftz.f32 %0, %1;" : "=f"(y) : "f"(x));
    return y;
}

// D pre-pass of the fused backward: Ds_i = scale * sum_c dO_ic O_ic and
// nlse2_i = -LSE_i * log2(e) (minus infinity for a row with no kept entry, so that its
// probabilities come out as exactly zero).  16-byte loads, HD/8 lanes share a row.  The same
// pass clears the fp32 dQ accumulator of the fused backward (`acc`, `acc16` 16-byte words; null =
// nothing to clear), so that its writes overlap the reads of O and dO.
template <int HD>
__global__ void __launch_bounds__(256) tc_preprocess_kernel(const __nv_bfloat16 *__restrict__ O,
                                                            const __nv_bfloat16 *__restrict__ dO,
                                                            const float *__restrict__ LSE, float *__restrict__ Ds,
                                                            float *__restrict__ nlse2, size_t rows, float scale,
                                                            uint4 *__restrict__ acc, size_t acc16)
{
    constexpr int LPR = HD / 8;   // lanes per row
    constexpr int RPW = 32 / LPR; // rows per warp
    constexpr int U = 4;          // row groups per step: eight 16-byte loads in flight per lane
    const int lane = threadIdx.x % 32, sub = lane / LPR, lr = lane % LPR;
    const size_t warp = ((size_t)blockIdx.x * blockDim.x + threadIdx.x) / 32;
    const size_t nwarps = (size_t)gridDim.x * blockDim.x / 32;
    if (acc != nullptr) {
        for (size_t i = (size_t)blockIdx.x * blockDim.x + threadIdx.x; i < acc16; i += (size_t)gridDim.x * blockDim.x)
            __stcs(acc + i, make_uint4(0u, 0u, 0u, 0u));
    }
    for (size_t base = warp * RPW * U; base < rows; base += nwarps * RPW * U) {
        uint4 xo[U], xg[U];
#pragma unroll
        for (int u = 0; u < U; ++u) {
            const size_t row = base + (size_t)u * RPW + sub;
            xo[u] = xg[u] = make_uint4(0u, 0u, 0u, 0u);
            if (row < rows) {
                xo[u] = __ldcs(reinterpret_cast<const uint4 *>(O + row * HD) + lr);
                xg[u] = __ldcs(reinterpret_cast<const uint4 *>(dO + row * HD) + lr);
            }
        }
#pragma unroll
        for (int u = 0; u < U; ++u) {
            const size_t row = base + (size_t)u * RPW + sub;
            const __nv_bfloat162 *eo = reinterpret_cast<const __nv_bfloat162 *>(&xo[u]);
            const __nv_bfloat162 *eg = reinterpret_cast<const __nv_bfloat162 *>(&xg[u]);
            float acc = 0.f;
#pragma unroll
            for (int e = 0; e < 4; ++e) {
                const float2 fo = __bfloat1622float2(eo[e]), fg = __bfloat1622float2(eg[e]);
                acc = fmaf(fo.x, fg.x, acc);
                acc = fmaf(fo.y, fg.y, acc);
            }
#pragma unroll
            for (int o = LPR / 2; o > 0; o >>= 1) acc += __shfl_xor_sync(0xffffffffu, acc, o);
            if (row < rows && lr == 0) {
                Ds[row] = acc * scale;
                const float l = LSE[row];
                nlse2[row] = l == -INFINITY ? -INFINITY : -l * 1.4426950408889634f;
            }
        }
    }
}


// one arrival per warp: every lane has finished (and fenced) its part, lane 0 tells the barrier
__device__ __forceinline__ void warp_arrive(uint64_t *bar, int lane)
{
    __syncwarp();
    if (lane == 0) mbar_arrive(bar);
}

}  // namespace bwdk

// Launchers of the D pre-pass (optionally clearing the fp32 dQ accumulator in the same pass) and of the
// conversion of that accumulator to bf16 dQ; both live in attn_tc_bwd.cu.
attn_status bwd_preprocess_launch(const Problem &p, bool clear_acc);
attn_status bwd_dq_convert_launch(const Problem &p);
int bwd_head_group(const Problem &p);   // heads launched together: their fp32 dQ accumulators stay in L2

}  // namespace attn

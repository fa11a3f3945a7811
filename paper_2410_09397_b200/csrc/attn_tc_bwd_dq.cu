// dQ without atomics (the deterministic half of the fused backward), bf16, d = 64 / 128.
//
// This is the loop order the paper prints for its large-cache phase 2: the outer loop is
// over query row blocks i (here: one CTA per block of 128 queries, whose dQ_i tile stays
// in tensor memory), the inner loop over the kept key blocks j.  Per (i, j):
//
//   S  = Q_i K_j^T                       tcgen05.mma, K-major smem operands, two S buffers
//   dP = dO_i V_j^T                      same, one buffer
//   dS = scale * exp2(S scale log2e - LSE_i log2e) o (dP - D_i)     256 threads, lane = query
//        -> bf16, written over S in tensor memory
//   dQ_i += dS K_j                       A = dS from tensor memory, B = K_j MN-major smem
//
// S and dP are recomputed here (the key-stationary kernel computes them too), which is
// the price of summing dQ in a fixed order: 7 products instead of 5 per tile pair.
// Roles: warps 0-15 = four warpgroups, warpgroup g owning key columns 32 g .. 32 g + 31 of every
// tile (no barrier couples them, so their exp, dS and tensor-memory phases interleave freely);
// warp 16 lane 0 issues S and dP, warp 17 lane 0 issues dQ, warp 18 lane 0 runs TMA.  Tensor memory: S0 128, S1 128, dP 128, dQ d columns.
#include "attn_internal.h"
#include "tc_common.cuh"

namespace attn {
namespace {

using namespace tc;

constexpr int TQ = 128, TKD = 128;
constexpr int kSoftmaxThreads = 512;
constexpr int kThreads = kSoftmaxThreads + 96;   // + two MMA-issuing warps and the TMA warp
constexpr uint32_t SLAB = 128 * 128;

struct DqArgs {
    __nv_bfloat16 *dQ;
    const float *nLSE2, *Ds;
    int n, BH;
    int mask_kind, block, nb, mask_heads;
    const int *row_ptr, *col_idx;
    FineMask fine;
    float scale;
    uint32_t *status;
};

template <int HD>
struct DqSmem {
    static constexpr int NSTK = 3, NSTV = 2;   // K_j is needed first (S) and released last (dQ): three stages; V_j: two
    static constexpr uint32_t kSlabs = HD / 64;
    static constexpr uint32_t kTile = kSlabs * SLAB;     // one [128][HD] bf16 tile
    static constexpr uint32_t oQ = 0;
    static constexpr uint32_t odO = oQ + kTile;
    static constexpr uint32_t oK = odO + kTile;          // NSTK stages
    static constexpr uint32_t oV = oK + NSTK * kTile;    // NSTV stages
    static constexpr uint32_t oBar = oV + NSTV * kTile;
    static constexpr uint32_t oMisc = oBar + 24 * 8;
    static constexpr uint32_t kUsed = oMisc + 64;
    static constexpr uint32_t kBytes = kUsed < 117 * 1024 ? 117 * 1024 : kUsed;   // one CTA per SM (512 TMEM columns)
    static_assert(kUsed <= 227 * 1024, "shared memory budget");
};

enum { DB_Q = 0, DB_KFULL = 1, DB_KEMPTY = 4, DB_VFULL = 7, DB_VEMPTY = 9, DB_S = 11, DB_DP = 13, DB_DPFREE = 14, DB_DS = 15,
       DB_DQ = 17 };

struct KeyIterD {
    int kind, n, sub, raw, last_i;
    const int *cols;
    __device__ KeyIterD(const DqArgs &a, int it, long bh) : kind(a.mask_kind), n(a.n), sub(1), raw(0), cols(nullptr)
    {
        last_i = min(it * TQ + TQ, n) - 1;
        const int ntk = (n + TKD - 1) / TKD;
        if (kind == ATTN_MASK_NONE) raw = ntk;
        else if (kind == ATTN_MASK_CAUSAL) raw = (min(it * TQ + TQ, n) - 1) / TKD + 1;
        else {
            sub = a.block / TKD;
            const int I = it * TQ / a.block;
            const long mh = a.mask_heads == 1 ? 0 : bh;
            const int *rp = a.row_ptr + mh * 2 * a.nb + 2 * I;
            cols = a.col_idx + mh * (long)a.nb * a.nb + rp[0];
            raw = (rp[1] - rp[0]) * sub;
        }
    }
    __device__ int tile(int idx) const
    {
        const int jt = mask_is_block(kind) ? cols[idx / sub] * sub + idx % sub : idx;
        // block mask AND causal: a key tile that begins after the last query of the tile keeps nothing
        if (kind == ATTN_MASK_BLOCK_SPARSE_CAUSAL && jt * TKD > last_i) return -1;
        return jt * TKD < n ? jt : -1;
    }
};

__device__ __forceinline__ float ex2_fast(float x)
{
    float y;
    asm("ex2.approx.ftz.f32 %0, %1;" : "=f"(y) : "f"(x));
    return y;
}

template <int HD>
__global__ void __launch_bounds__(kThreads, 1)
tc_bwd_dq_kernel(const __grid_constant__ CUtensorMap mQ, const __grid_constant__ CUtensorMap mK,
                 const __grid_constant__ CUtensorMap mV, const __grid_constant__ CUtensorMap mdO, const DqArgs a)
{
    using L = DqSmem<HD>;
    constexpr int NSTK = L::NSTK, NSTV = L::NSTV;
    extern __shared__ __align__(1024) uint8_t smem[];
    uint64_t *bars = reinterpret_cast<uint64_t *>(smem + L::oBar);
    uint32_t *tmem_base_s = reinterpret_cast<uint32_t *>(smem + L::oMisc);
    volatile uint32_t *abort_flag = reinterpret_cast<volatile uint32_t *>(smem + L::oMisc + 4);
    const Abort ab{abort_flag, a.status};

    const int tid = threadIdx.x, warp = tid / 32, lane = tid % 32;
    const int nt = (a.n + TQ - 1) / TQ;
    const int it = nt - 1 - (int)blockIdx.x;    // heaviest causal tiles first
    const long bh = blockIdx.y;
    const int i0 = it * TQ, n = a.n;

    if ((smem_u32(smem) & 1023u) != 0) {
        if (tid == 0) atomicExch(a.status, 9u);
        return;
    }
    if (tid == 0) {
        *abort_flag = 0;
        mbar_init(&bars[DB_Q], 1);
        for (int s = 0; s < NSTK; ++s) { mbar_init(&bars[DB_KFULL + s], 1); mbar_init(&bars[DB_KEMPTY + s], 1); }
        for (int s = 0; s < NSTV; ++s) { mbar_init(&bars[DB_VFULL + s], 1); mbar_init(&bars[DB_VEMPTY + s], 1); }
        for (int b = 0; b < 2; ++b) { mbar_init(&bars[DB_S + b], 1); mbar_init(&bars[DB_DS + b], kSoftmaxThreads / 32); }   // one arrival per warp
        mbar_init(&bars[DB_DP], 1);
        mbar_init(&bars[DB_DPFREE], kSoftmaxThreads / 32);
        mbar_init(&bars[DB_DQ], 1);
        fence_barrier_init();
        prefetch_tensormap(&mQ); prefetch_tensormap(&mK); prefetch_tensormap(&mV); prefetch_tensormap(&mdO);
    }
    if (warp == 0) tmem_alloc(tmem_base_s, 512);
    tcgen05_fence_before();
    __syncthreads();
    tcgen05_fence_after();
    const uint32_t tm = *tmem_base_s;
    const uint32_t T_dP = tm + 256, T_dQ = tm + 384;
    const KeyIterD iter(a, it, bh);
    int niter = 0;
    for (int idx = 0; idx < iter.raw; ++idx) niter += iter.tile(idx) >= 0;

    if (warp == 18) {
        // ------------------------------------------------------------ TMA producer
        if (lane == 0) {
            mbar_expect_tx(&bars[DB_Q], 2 * L::kTile);
#pragma unroll
            for (uint32_t sl = 0; sl < L::kSlabs; ++sl) {
                tma_load_3d(smem + L::oQ + sl * SLAB, &mQ, &bars[DB_Q], sl * 64, i0, (int)bh);
                tma_load_3d(smem + L::odO + sl * SLAB, &mdO, &bars[DB_Q], sl * 64, i0, (int)bh);
            }
            int k = 0;
            for (int idx = 0; idx < iter.raw; ++idx) {
                const int jt = iter.tile(idx);
                if (jt < 0) continue;
                const int sk = k % NSTK, sv = k % NSTV;
                if (k >= NSTK) mbar_wait(&bars[DB_KEMPTY + sk], ((k / NSTK) - 1) & 1, ab);
                mbar_expect_tx(&bars[DB_KFULL + sk], L::kTile);
#pragma unroll
                for (uint32_t sl = 0; sl < L::kSlabs; ++sl)
                    tma_load_3d(smem + L::oK + sk * L::kTile + sl * SLAB, &mK, &bars[DB_KFULL + sk], sl * 64, jt * TKD, (int)bh);
                if (k >= NSTV) mbar_wait(&bars[DB_VEMPTY + sv], ((k / NSTV) - 1) & 1, ab);
                mbar_expect_tx(&bars[DB_VFULL + sv], L::kTile);
#pragma unroll
                for (uint32_t sl = 0; sl < L::kSlabs; ++sl)
                    tma_load_3d(smem + L::oV + sv * L::kTile + sl * SLAB, &mV, &bars[DB_VFULL + sv], sl * 64, jt * TKD, (int)bh);
                ++k;
            }
            if (niter == 0) mbar_wait(&bars[DB_Q], 0, ab);   // let the Q / dO load land before exit
        }
    } else if (warp == 16) {
        // ------------------------------------------------------------ MMA issuer A: the products the warps wait for, S and dP,
        // one tile ahead.  (Two issuing threads: a thread that waits on a barrier or commits cannot keep the short
        // queue of the tensor pipe filled; B's dQ products are ordered against A's through barriers only.)
        if (lane == 0 && niter > 0) {
            constexpr uint32_t idesc_s = idesc_bf16(128, 128, 0, 0);
            constexpr uint32_t kSlab = SLAB >> 4;
            const uint32_t kQ = desc_lo_kmajor(smem_u32(smem + L::oQ)), kdO = desc_lo_kmajor(smem_u32(smem + L::odO));
            auto issue_S = [&](int k) {
                const int s = k % NSTK;
                mbar_wait(&bars[DB_KFULL + s], (k / NSTK) & 1, ab);
                // the buffer of S(k) held dS(k-2): the dQ product of tile k-2 (other thread) must have consumed it
                if (k >= 2) mbar_wait(&bars[DB_KEMPTY + (k - 2) % NSTK], ((k - 2) / NSTK) & 1, ab);
                tcgen05_fence_after();
                const uint32_t kK = desc_lo_kmajor(smem_u32(smem + L::oK + s * L::kTile));
#pragma unroll
                for (int kk = 0; kk < HD / 16; ++kk) {
                    const uint32_t off = (kk / 4) * kSlab + (kk % 4) * 2;
                    mma_ss_lo(tm + (k & 1) * 128, kQ + off, kK + off, idesc_s, kk > 0);
                }
                mma_commit(&bars[DB_S + (k & 1)]);
            };
            auto issue_dP = [&](int k) {
                mbar_wait(&bars[DB_VFULL + k % NSTV], (k / NSTV) & 1, ab);
                tcgen05_fence_after();
                const uint32_t kV = desc_lo_kmajor(smem_u32(smem + L::oV + (k % NSTV) * L::kTile));
#pragma unroll
                for (int kk = 0; kk < HD / 16; ++kk) {
                    const uint32_t off = (kk / 4) * kSlab + (kk % 4) * 2;
                    mma_ss_lo(T_dP, kdO + off, kV + off, idesc_s, kk > 0);
                }
                mma_commit(&bars[DB_DP]);
                mma_commit(&bars[DB_VEMPTY + k % NSTV]);
            };
            mbar_wait(&bars[DB_Q], 0, ab);
            issue_S(0);
            issue_dP(0);
            for (int k = 0; k + 1 < niter; ++k) {
                issue_S(k + 1);
                // dP(k+1) once every thread has read dP(k) out of tensor memory
                mbar_wait(&bars[DB_DPFREE], k & 1, ab);
                tcgen05_fence_after();
                issue_dP(k + 1);
            }
        }
    } else if (warp == 17) {
        // ------------------------------------------------------------ MMA issuer B: dQ_i += dS K_j
        if (lane == 0 && niter > 0) {
            constexpr uint32_t idesc_dq = idesc_bf16(128, HD, 0, 1);
            for (int k = 0; k < niter; ++k) {
                const int s = k % NSTK, b = k & 1;
                mbar_wait(&bars[DB_KFULL + s], (k / NSTK) & 1, ab);
                mbar_wait(&bars[DB_DS + b], (k >> 1) & 1, ab);
                tcgen05_fence_after();
                const uint32_t mK_ = desc_lo_mnmajor(smem_u32(smem + L::oK + s * L::kTile), SLAB);
#pragma unroll
                for (int kk = 0; kk < TKD / 16; ++kk)
                    mma_ts_lo(T_dQ, tm + b * 128 + (kk / 2) * 32 + (kk % 2) * 8, mK_ + kk * 128, idesc_dq,
                              (k > 0) || (kk > 0));
                mma_commit(&bars[DB_KEMPTY + s]);
                if (k == niter - 1) mma_commit(&bars[DB_DQ]);
            }
        }
    } else {
        // ------------------------------------------------------------ dS warpgroups: wg splits the key columns
        const int wg = warp / 4;
        const int row = (warp % 4) * 32 + lane;           // tensor-memory lane = query row of the tile
        const uint32_t lane_addr = (uint32_t)((warp % 4) * 32) << 16;
        const int ig = i0 + row;
        const float sl2 = a.scale * 1.4426950408889634f;
        const float nl = ig < n ? a.nLSE2[(size_t)bh * n + ig] : -INFINITY;   // -inf: every probability of the row is 0
        const float dsi = ig < n ? a.Ds[(size_t)bh * n + ig] : 0.f;
        int k = 0;
        for (int idx = 0; idx < iter.raw; ++idx) {
            const int jt = iter.tile(idx);
            if (jt < 0) continue;
            const int b = k & 1, j0 = jt * TKD + wg * 32;
            const uint32_t T_S = tm + b * 128;
            // a mask finer than the tile: the keep bits of this thread's query row and its 32 key columns
            uint32_t kw = 0xffffffffu;
            if (a.fine.mode) kw = (ig < n && j0 < n) ? fine_word(a.fine, a.mask_heads, bh, true, ig, j0) : 0u;
            const bool masked = (mask_is_causal(a.mask_kind) && jt * TKD + TKD - 1 > i0) || jt * TKD + TKD > n || a.fine.mode != 0;
            mbar_wait(&bars[DB_S + b], (k >> 1) & 1, ab);
            tcgen05_fence_after();
            float p[32];
            {
                uint32_t sv0[32];
                tmem_ld32(T_S + lane_addr + wg * 32, sv0);
                tmem_wait_ld();
#pragma unroll
                for (int e = 0; e < 32; ++e) p[e] = ex2_fast(fmaf(__uint_as_float(sv0[e]), sl2, nl));
            }
            if (masked) {
                const bool causal = mask_is_causal(a.mask_kind);
#pragma unroll
                for (int e = 0; e < 32; ++e) {
                    const int jg = j0 + e;
                    if (jg >= n || (causal && jg > ig) || !((kw >> e) & 1u)) p[e] = 0.f;
                }
            }
            mbar_wait(&bars[DB_DP], k & 1, ab);
            tcgen05_fence_after();
            uint32_t dpack[16];
            {
                uint32_t dv0[32];
                tmem_ld32(T_dP + lane_addr + wg * 32, dv0);
                tmem_wait_ld();
                tcgen05_fence_before();
                __syncwarp();
                if (lane == 0) mbar_arrive(&bars[DB_DPFREE]);
#pragma unroll
                for (int e = 0; e < 32; e += 2)
                    dpack[e / 2] = pack_bf16(p[e] * fmaf(__uint_as_float(dv0[e]), a.scale, -dsi),
                                             p[e + 1] * fmaf(__uint_as_float(dv0[e + 1]), a.scale, -dsi));
            }
            // dS (bf16 pairs) over the first 16 of the 32 S columns this thread has read itself
            tmem_st16(T_S + lane_addr + wg * 32, dpack);
            tmem_wait_st();
            tcgen05_fence_before();
            __syncwarp();
            if (lane == 0) mbar_arrive(&bars[DB_DS + b]);
            ++k;
        }
        // ------------------------------------------------------------ epilogue: dQ_i (dS carried the scale)
        if (k > 0) {
            mbar_wait(&bars[DB_DQ], 0, ab);
            tcgen05_fence_after();
        }
        constexpr int OW = HD / 4;   // dQ columns per warpgroup: 32 or 16
        const int ic = ig < n ? ig : 0;
        __nv_bfloat16 *pq = a.dQ + ((size_t)bh * n + ic) * HD + wg * OW;
        {
            constexpr int c = 0;
            uint32_t v[32];
            if (k > 0) {
                if (OW == 32) tmem_ld32(T_dQ + lane_addr + wg * OW, v);
                else tmem_ld16(T_dQ + lane_addr + wg * OW, *reinterpret_cast<uint32_t(*)[16]>(v));
                tmem_wait_ld();
            } else {
#pragma unroll
                for (int e = 0; e < 32; ++e) v[e] = 0u;
            }
            if (ig < n) {
#pragma unroll
                for (int e = 0; e < OW; e += 8)
                    *reinterpret_cast<uint4 *>(pq + c + e) =
                        make_uint4(pack_bf16(__uint_as_float(v[e]), __uint_as_float(v[e + 1])),
                                   pack_bf16(__uint_as_float(v[e + 2]), __uint_as_float(v[e + 3])),
                                   pack_bf16(__uint_as_float(v[e + 4]), __uint_as_float(v[e + 5])),
                                   pack_bf16(__uint_as_float(v[e + 6]), __uint_as_float(v[e + 7])));
            }
        }
    }
    tcgen05_fence_before();
    __syncthreads();
    if (warp == 0) tmem_dealloc(tm, 512);
}

template <int HD>
attn_status launch_dq(const Problem &p)
{
    using L = DqSmem<HD>;
    CUtensorMap mQ, mK, mV, mdO;
    const uint64_t BH = (uint64_t)p.BH;
    if (!make_tmap_bf16_3d(&mQ, p.Q, HD, p.n, BH, 128) || !make_tmap_bf16_3d(&mK, p.K, HD, p.n, BH, 128) ||
        !make_tmap_bf16_3d(&mV, p.V, HD, p.n, BH, 128) || !make_tmap_bf16_3d(&mdO, p.dO, HD, p.n, BH, 128))
        return ATTN_ERR_LAUNCH;
    DqArgs a{};
    a.dQ = (__nv_bfloat16 *)p.dQ;
    a.nLSE2 = p.nLSE2; a.Ds = p.D;
    a.n = p.n; a.BH = (int)p.BH;
    a.mask_kind = p.mask_kind; a.block = p.block; a.nb = p.nb; a.mask_heads = p.mask_heads; a.fine = p.fine;
    a.row_ptr = p.row_ptr; a.col_idx = p.col_idx;
    a.scale = p.scale;
    a.status = p.status;
    auto kernel = tc_bwd_dq_kernel<HD>;
    if (cudaFuncSetAttribute(kernel, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)L::kBytes) != cudaSuccess)
        return ATTN_ERR_LAUNCH;
    const dim3 grid((p.n + TQ - 1) / TQ, (unsigned)p.BH);
    launch_begin("tc_bwd_dq", p.stream);
    kernel<<<grid, kThreads, L::kBytes, p.stream>>>(mQ, mK, mV, mdO, a);
    launch_end(p.stream);
    return cudaGetLastError() == cudaSuccess ? ATTN_OK : ATTN_ERR_LAUNCH;
}

}  // namespace

// Requires p.D = scale * rowsum(dO o O) and p.nLSE2 = -LSE log2(e), as the key-stationary launch leaves them.
attn_status tc_bwd_dq(const Problem &p)
{
    if (p.d == 64) return launch_dq<64>(p);
    if (p.d == 128) return launch_dq<128>(p);
    return ATTN_ERR_TILE;
}

}  // namespace attn

// Fused backward for bf16 on the 5th-generation tensor cores (large-cache regime of
// Appendix D: no n x n matrix ever leaves the SM).
//
// The loops of the paper's phase-2 algorithm are swapped: a CTA owns one tile of 128
// KEYS j (K_j, V_j stay in shared memory, dK_j and dV_j stay in tensor memory) and walks
// the kept QUERY tiles i.  Per (i, j) pair, with everything transposed so that the
// tensor-memory lane is the key index:
//
//   S^T  = K_j Q_i^T                         (tcgen05.mma, both operands K-major smem)
//   dP^T = V_j dO_i^T                        (same)
//   P^T  = exp2(S^T * scale*log2e - LSE_i*log2e)        (256 threads, fp32)
//   dS^T = scale * P^T o (dP^T - D_i)                   (Definition B.9, p = f o q - diag(v) f;
//                                                        the scale of dQ and dK is folded in here)
//   dV_j += P^T  dO_i      A = P^T  in tensor memory (bf16), B = dO_i MN-major smem
//   dK_j += dS^T Q_i       A = dS^T K-major smem,            B = Q_i  MN-major smem
//   dQ_i += dS K_j         computed as dQ^T = K_j^T dS^T (lane = head-dimension index), so that
//                          the fp32 reductions into global memory are coalesced; at d = 64 the
//                          product is padded to M = 128 with an all-zero slab
//
// dQ partial tiles are added into an fp32 accumulator in the workspace with
// red.global.add (the one place where summation order is not fixed); a small kernel
// converts it to bf16 at the end.  Tensor memory (512 columns): 128 shared by S^T and
// dP^T (fused kernel; S^T / P^T in the dK/dV kernel), 128 by P^T and dQ^T (dP^T / dS^T
// in the dK/dV kernel), dV d, dK d.
//
// Two kernels: tc_bwd_fused_kernel (all five products, the default) and tc_bwd_dkdv_kernel
// (without the dQ product; `deterministic = 1` pairs it with the query-stationary dQ kernel of
// attn_tc_bwd_dq.cu).  Warp roles are described at each kernel.  All waits are bounded
// (tc_common.cuh).
#include "tc_bwd_common.cuh"

namespace attn {
namespace {

using namespace tc;
using namespace bwdk;

constexpr int TQ = 128;
template <int HD>
struct BwdSmem {
    static constexpr uint32_t kSlabs = HD / 64;
    static constexpr uint32_t kTile = kSlabs * SLAB;      // one [128][HD] bf16 tile
    static constexpr uint32_t oK = 0;
    static constexpr uint32_t oV = oK + kTile;
    static constexpr uint32_t oQ = oV + kTile;            // 2 stages
    static constexpr uint32_t odO = oQ + 2 * kTile;       // 2 stages
    static constexpr uint32_t odS = odO + 2 * kTile;      // [128 keys][128 queries] bf16, 2 slabs
    static constexpr uint32_t oLSE = odS + 2 * SLAB;      // 2 stages x 128 floats
    static constexpr uint32_t oD = oLSE + 2 * 128 * 4;
    static constexpr uint32_t oBar = oD + 2 * 128 * 4;    // mbarriers (8 bytes each)
    static constexpr uint32_t oMisc = oBar + 24 * 8;      // tmem base, abort flag
    static constexpr uint32_t kBytes = oMisc + 64;
    static_assert(kBytes <= 227 * 1024, "shared memory budget");
};


using TileIter = TileIterT<TQ>;

// barrier indices of the fused kernel: every barrier exists once per 64-query half of a tile
enum { V2_KV = 0, V2_QFULL = 1, V2_QEMPTY = 3, V2_S = 5, V2_DP = 7, V2_P = 9, V2_DS = 11, V2_DQ = 13, V2_DQDONE = 15, V2_SLD = 17,
       V2_DPLD = 19, V2_DQREL = 21 };


// ---------------------------------------------------------------------------------------
// dK and dV only: the key-stationary half of the path without atomics (dQ comes from the
// query-stationary kernel).  Without the dQ product dS^T never has to be in shared memory.
// Tensor memory: region A (128 columns) receives S^T and dP^T in turn; an exp / dS thread copies its
// 32 columns into registers with one load and releases the region at once.  Region B (128 columns)
// holds P^T and dS^T as bf16 pairs (per 64-query half: P^T in columns 64 h .. 64 h + 31, dS^T in
// 64 h + 32 .. 64 h + 63), from where dV += P^T dO and dK += dS^T Q take them as their A operand.
// Two MMA-issuing threads: A issues dP^T(k) (once S^T(k) has been copied out and dK(k-1) has left
// dS^T(k-1)) and S^T(k+1) (once dP^T(k) has been copied out); B issues dV(k) and dK(k).  The 32 KB that
// dS^T does not take in shared memory hold a third Q stage; Q, dO and the row statistics are released
// separately (dO after dV, Q after dK, LSE / D after the dS phase).
template <int HD> struct DkdvSmem {
    static constexpr uint32_t kSlabs = HD / 64;
    static constexpr uint32_t kTile = kSlabs * SLAB;        // one [128][HD] bf16 tile
    static constexpr uint32_t oK = 0;
    static constexpr uint32_t oV = oK + kTile;
    static constexpr uint32_t oQ = oV + kTile;              // 3 stages
    static constexpr uint32_t odO = oQ + 3 * kTile;         // 2 stages
    static constexpr uint32_t oLSE = odO + 2 * kTile;       // 2 stages x 128 floats
    static constexpr uint32_t oD = oLSE + 2 * 128 * 4;
    static constexpr uint32_t oBar = oD + 2 * 128 * 4;
    static constexpr uint32_t oMisc = oBar + 24 * 8;
    static constexpr uint32_t kBytes = oMisc + 64;
    static_assert(kBytes <= 227 * 1024, "shared memory budget");
};
enum { KD_KV = 0, KD_QFULL = 1, KD_QEMPTY = 4, KD_OFULL = 7, KD_OEMPTY = 9, KD_LFULL = 11, KD_LEMPTY = 13,
       KD_S = 15, KD_DP = 16, KD_SLD = 17, KD_DPLD = 18, KD_P = 19, KD_DS = 21, KD_DONE = 22 };
constexpr int kThreadsDkdv = 512 + 128;   // 16 exp/dS warps, issuer A, TMA producer, issuer B, one idle warp

template <int HD>
__global__ void __launch_bounds__(kThreadsDkdv, 1)
tc_bwd_dkdv_kernel(const __grid_constant__ CUtensorMap mQ, const __grid_constant__ CUtensorMap mK_,
                   const __grid_constant__ CUtensorMap mV, const __grid_constant__ CUtensorMap mdO, const BwdArgs a)
{
    constexpr int kExpWarps = 16, kHalfWarps = 8;
    using L = DkdvSmem<HD>;
    extern __shared__ __align__(1024) uint8_t smem[];
    uint64_t *bars = reinterpret_cast<uint64_t *>(smem + L::oBar);
    uint32_t *tmem_base_s = reinterpret_cast<uint32_t *>(smem + L::oMisc);
    volatile uint32_t *abort_flag = reinterpret_cast<volatile uint32_t *>(smem + L::oMisc + 4);
    const Abort ab{abort_flag, a.status};

    const int tid = threadIdx.x, warp = tid / 32, lane = tid % 32;
    const int jt = blockIdx.x / a.group;
    const long bh = (long)blockIdx.y * a.group + blockIdx.x % a.group;
    const int j0 = jt * TK, n = a.n;

    if ((smem_u32(smem) & 1023u) != 0) {
        if (tid == 0) atomicExch(a.status, 9u);
        return;
    }
    if (tid == 0) {
        *abort_flag = 0;
        mbar_init(&bars[KD_KV], 1);
        for (int s = 0; s < 3; ++s) { mbar_init(&bars[KD_QFULL + s], 1); mbar_init(&bars[KD_QEMPTY + s], 1); }
        for (int s = 0; s < 2; ++s) {
            mbar_init(&bars[KD_OFULL + s], 1);
            mbar_init(&bars[KD_OEMPTY + s], 1);
            mbar_init(&bars[KD_LFULL + s], 1);
            mbar_init(&bars[KD_LEMPTY + s], kExpWarps);
            mbar_init(&bars[KD_P + s], kHalfWarps);
        }
        mbar_init(&bars[KD_S], 1);
        mbar_init(&bars[KD_DP], 1);
        mbar_init(&bars[KD_SLD], kExpWarps);
        mbar_init(&bars[KD_DPLD], kExpWarps);
        mbar_init(&bars[KD_DS], kExpWarps);
        mbar_init(&bars[KD_DONE], 1);
        fence_barrier_init();
        prefetch_tensormap(&mQ); prefetch_tensormap(&mK_); prefetch_tensormap(&mV); prefetch_tensormap(&mdO);
    }
    if (warp == 0) tmem_alloc(tmem_base_s, 512);
    tcgen05_fence_before();
    __syncthreads();
    tcgen05_fence_after();
    const uint32_t tm = *tmem_base_s;
    const uint32_t T_A = tm, T_B = tm + 128, T_dV = tm + 256, T_dK = tm + 256 + HD;
    constexpr uint32_t HALF_ROWS = 64 * 128;   // byte offset of rows 64.. inside a [128][64] slab

    const TileIter iter(a, jt, bh);

    if (warp == 17) {
        // ------------------------------------------------------------ TMA producer
        if (lane == 0) {
            mbar_expect_tx(&bars[KD_KV], 2 * L::kTile);
#pragma unroll
            for (uint32_t sl = 0; sl < L::kSlabs; ++sl) {
                tma_load_3d(smem + L::oK + sl * SLAB, &mK_, &bars[KD_KV], sl * 64, j0, (int)bh);
                tma_load_3d(smem + L::oV + sl * SLAB, &mV, &bars[KD_KV], sl * 64, j0, (int)bh);
            }
            int k = 0;
            for (int idx = 0; idx < iter.raw; ++idx) {
                const int it = iter.tile(idx);
                if (it < 0) continue;
                const int i0 = it * TQ, sq = k % 3, s2 = k & 1;
                const uint32_t rows = min(TQ, n - i0);
                if (k >= 3) mbar_wait(&bars[KD_QEMPTY + sq], ((k / 3) - 1) & 1, ab);
                mbar_expect_tx(&bars[KD_QFULL + sq], L::kTile);
#pragma unroll
                for (uint32_t sl = 0; sl < L::kSlabs; ++sl)
                    tma_load_3d(smem + L::oQ + sq * L::kTile + sl * SLAB, &mQ, &bars[KD_QFULL + sq], sl * 64, i0, (int)bh);
                if (k >= 2) mbar_wait(&bars[KD_LEMPTY + s2], ((k >> 1) - 1) & 1, ab);
                mbar_expect_tx(&bars[KD_LFULL + s2], 2 * rows * 4);
                bulk_load_1d(smem + L::oLSE + s2 * 512, a.nLSE2 + bh * n + i0, rows * 4, &bars[KD_LFULL + s2]);
                bulk_load_1d(smem + L::oD + s2 * 512, a.Ds + bh * n + i0, rows * 4, &bars[KD_LFULL + s2]);
                if (k >= 2) mbar_wait(&bars[KD_OEMPTY + s2], ((k >> 1) - 1) & 1, ab);
                mbar_expect_tx(&bars[KD_OFULL + s2], L::kTile);
#pragma unroll
                for (uint32_t sl = 0; sl < L::kSlabs; ++sl)
                    tma_load_3d(smem + L::odO + s2 * L::kTile + sl * SLAB, &mdO, &bars[KD_OFULL + s2], sl * 64, i0, (int)bh);
                ++k;
            }
            // a key tile without a single query tile (an empty block column): nobody else waits for K_j and V_j, and
            // the CTA must not exit with their bulk loads still in flight into its shared memory
            if (k == 0) mbar_wait(&bars[KD_KV], 0, ab);
        }
    } else if (warp == 16) {
        // ------------------------------------------------------------ MMA issuer A: the products into region A
        if (lane == 0) {
            constexpr uint32_t idesc_s = idesc_bf16(128, 128, 0, 0);       // S^T, dP^T
            const uint32_t kK = desc_lo_kmajor(smem_u32(smem + L::oK)), kV = desc_lo_kmajor(smem_u32(smem + L::oV));
            constexpr uint32_t kSlab = SLAB >> 4;
            auto issue_S = [&](int k) {
                const uint32_t kQ = desc_lo_kmajor(smem_u32(smem + L::oQ + (k % 3) * L::kTile));
#pragma unroll
                for (int kk = 0; kk < HD / 16; ++kk) {
                    const uint32_t off = (kk / 4) * kSlab + (kk % 4) * 2;
                    mma_ss_lo(T_A, kK + off, kQ + off, idesc_s, kk > 0);
                }
                mma_commit(&bars[KD_S]);
            };
            int idx = 0, it = -1;
            while (idx < iter.raw && (it = iter.tile(idx)) < 0) ++idx;
            if (it >= 0) {
                mbar_wait(&bars[KD_KV], 0, ab);
                mbar_wait(&bars[KD_QFULL], 0, ab);
                tcgen05_fence_after();
                issue_S(0);
            }
            int k = 0;
            while (idx < iter.raw) {
                int nidx = idx + 1, nit = -1;
                while (nidx < iter.raw && (nit = iter.tile(nidx)) < 0) ++nidx;
                // dP^T(k) into region A: S^T(k) copied out, dO(k) landed, and -- because the exp / dS warps store
                // dS^T(k) as soon as they have seen dP^T(k) -- the dK product of tile k-1 done with dS^T(k-1)
                mbar_wait(&bars[KD_OFULL + (k & 1)], (k >> 1) & 1, ab);
                if (k > 0) mbar_wait(&bars[KD_QEMPTY + (k - 1) % 3], ((k - 1) / 3) & 1, ab);
                mbar_wait(&bars[KD_SLD], k & 1, ab);
                tcgen05_fence_after();
                {
                    const uint32_t kdO = desc_lo_kmajor(smem_u32(smem + L::odO + (k & 1) * L::kTile));
#pragma unroll
                    for (int kk = 0; kk < HD / 16; ++kk) {
                        const uint32_t off = (kk / 4) * kSlab + (kk % 4) * 2;
                        mma_ss_lo(T_A, kV + off, kdO + off, idesc_s, kk > 0);
                    }
                    mma_commit(&bars[KD_DP]);
                }
                if (nit >= 0) {   // S^T(k+1) as soon as dP^T(k) has been copied out
                    mbar_wait(&bars[KD_QFULL + (k + 1) % 3], ((k + 1) / 3) & 1, ab);
                    mbar_wait(&bars[KD_DPLD], k & 1, ab);
                    tcgen05_fence_after();
                    issue_S(k + 1);
                }
                ++k;
                idx = nidx;
            }
        }
    } else if (warp == 18) {
        // ------------------------------------------------------------ MMA issuer B: dV += P^T dO, dK += dS^T Q
        if (lane == 0) {
            constexpr uint32_t idesc_dv = idesc_bf16(128, HD, 0, 1);       // A in tensor memory, B MN-major
            constexpr uint32_t kHalf = HALF_ROWS >> 4;
            int k = 0;
            for (int idx = 0; idx < iter.raw; ++idx) {
                if (iter.tile(idx) < 0) continue;
                const uint32_t mdO_ = desc_lo_mnmajor(smem_u32(smem + L::odO + (k & 1) * L::kTile), SLAB);
                const uint32_t mQ_ = desc_lo_mnmajor(smem_u32(smem + L::oQ + (k % 3) * L::kTile), SLAB);
                mbar_wait(&bars[KD_OFULL + (k & 1)], (k >> 1) & 1, ab);
#pragma unroll
                for (int h = 0; h < 2; ++h) {
                    mbar_wait(&bars[KD_P + h], k & 1, ab);
                    tcgen05_fence_after();
#pragma unroll
                    for (int kk = 0; kk < 4; ++kk)
                        mma_ts_lo(T_dV, T_B + 64 * h + kk * 8, mdO_ + h * kHalf + kk * 128, idesc_dv, (k > 0) || (h > 0) || (kk > 0));
                }
                mma_commit(&bars[KD_OEMPTY + (k & 1)]);
                mbar_wait(&bars[KD_QFULL + k % 3], (k / 3) & 1, ab);
                mbar_wait(&bars[KD_DS], k & 1, ab);
                tcgen05_fence_after();
#pragma unroll
                for (int h = 0; h < 2; ++h)
#pragma unroll
                    for (int kk = 0; kk < 4; ++kk)
                        mma_ts_lo(T_dK, T_B + 64 * h + 32 + kk * 8, mQ_ + h * kHalf + kk * 128, idesc_dv, (k > 0) || (h > 0) || (kk > 0));
                mma_commit(&bars[KD_QEMPTY + k % 3]);
                ++k;
            }
            mma_commit(&bars[KD_DONE]);
        }
    } else if (warp < 16) {
        // ------------------------------------------------------------ warpgroup 2h + qq owns queries 64 h + 32 qq .. + 31
        const int h = warp / 8, qq = (warp / 4) & 1;
        const int row = (warp % 4) * 32 + lane;        // tensor-memory lane = key row inside the tile
        const uint32_t lane_addr = (uint32_t)((warp % 4) * 32) << 16;
        const int jg = j0 + row;
        const float sl2 = a.scale * 1.4426950408889634f;
        const uint32_t c0 = h * 64 + qq * 32;          // this thread's first column of S^T / dP^T in region A
        const uint32_t cP = h * 64 + qq * 16;          // of its bf16 pairs of P^T in region B; dS^T 32 columns further
        int k = 0;
        for (int idx = 0; idx < iter.raw; ++idx) {
            const int it = iter.tile(idx);
            if (it < 0) continue;
            const int s2 = k & 1, i0 = it * TQ;
            const float4 *sNL = reinterpret_cast<const float4 *>(smem + L::oLSE + s2 * 512 + h * 256 + qq * 128);
            const float4 *sDs = reinterpret_cast<const float4 *>(smem + L::oD + s2 * 512 + h * 256 + qq * 128);
            const bool diag = mask_is_causal(a.mask_kind) && it == jt;
            const int ig0 = i0 + h * 64 + qq * 32;
            // a mask finer than the tile: the keep bits of this thread's key row and its 32 query columns
            uint32_t kw = 0xffffffffu;
            if (a.fine.mode) kw = (ig0 < n && jg < n) ? fine_word(a.fine, a.mask_heads, bh, false, jg, ig0) : 0u;
            const bool masked = diag || i0 + TQ > n || j0 + TK > n || a.fine.mode != 0;
            mbar_wait(&bars[KD_S], k & 1, ab);
            tcgen05_fence_after();
            uint32_t ppack[16];
            {
                uint32_t sv[32];
                tmem_ld32(T_A + lane_addr + c0, sv);
                tmem_wait_ld();
                tcgen05_fence_before();
                warp_arrive(&bars[KD_SLD], lane);   // region A may take dP^T
                mbar_wait(&bars[KD_LFULL + s2], (k >> 1) & 1, ab);
#pragma unroll
                for (int q = 0; q < 8; ++q) {
                    const float4 nl = sNL[q];
                    float p[4];
                    p[0] = ex2_approx(fmaf(__uint_as_float(sv[q * 4 + 0]), sl2, nl.x));
                    p[1] = ex2_approx(fmaf(__uint_as_float(sv[q * 4 + 1]), sl2, nl.y));
                    p[2] = ex2_approx(fmaf(__uint_as_float(sv[q * 4 + 2]), sl2, nl.z));
                    p[3] = ex2_approx(fmaf(__uint_as_float(sv[q * 4 + 3]), sl2, nl.w));
                    if (masked) {
#pragma unroll
                        for (int e = 0; e < 4; ++e) {
                            const int ig = ig0 + q * 4 + e;
                            const bool ok = ig < n && jg < n && (!diag || jg <= ig) && ((kw >> (q * 4 + e)) & 1u);
                            p[e] = ok ? p[e] : 0.f;
                        }
                    }
                    ppack[q * 2 + 0] = pack_bf16(p[0], p[1]);
                    ppack[q * 2 + 1] = pack_bf16(p[2], p[3]);
                }
            }
            mbar_wait(&bars[KD_DP], k & 1, ab);
            tcgen05_fence_after();
            uint32_t dv[32];
            tmem_ld32(T_A + lane_addr + c0, dv);
            tmem_wait_ld();
            tcgen05_fence_before();
            warp_arrive(&bars[KD_DPLD], lane);   // region A may take the next S^T
            // P^T(k) over P^T(k-1): the dV product of the previous tile must have consumed it
            if (k > 0) {
                mbar_wait(&bars[KD_OEMPTY + ((k - 1) & 1)], ((k - 1) >> 1) & 1, ab);
                tcgen05_fence_after();
            }
            tmem_st16(T_B + lane_addr + cP, ppack);
            tmem_wait_st();
            tcgen05_fence_before();
            warp_arrive(&bars[KD_P + h], lane);
            {
                uint32_t dpack[16];
#pragma unroll
                for (int q = 0; q < 8; ++q) {
                    const float4 dsc = sDs[q];
                    // bf16 -> fp32 is a 16-bit shift; a masked entry has p = 0 and a finite dP, so its dS is an exact zero
                    const float p0 = __uint_as_float(ppack[q * 2] << 16), p1 = __uint_as_float(ppack[q * 2] & 0xffff0000u);
                    const float p2 = __uint_as_float(ppack[q * 2 + 1] << 16), p3 = __uint_as_float(ppack[q * 2 + 1] & 0xffff0000u);
                    float d0 = p0 * fmaf(__uint_as_float(dv[q * 4 + 0]), a.scale, -dsc.x);
                    float d1 = p1 * fmaf(__uint_as_float(dv[q * 4 + 1]), a.scale, -dsc.y);
                    float d2 = p2 * fmaf(__uint_as_float(dv[q * 4 + 2]), a.scale, -dsc.z);
                    float d3 = p3 * fmaf(__uint_as_float(dv[q * 4 + 3]), a.scale, -dsc.w);
                    if (masked) {   // stale tail entries of the row vectors may be anything: select, do not multiply
                        d0 = p0 != 0.f ? d0 : 0.f; d1 = p1 != 0.f ? d1 : 0.f;
                        d2 = p2 != 0.f ? d2 : 0.f; d3 = p3 != 0.f ? d3 : 0.f;
                    }
                    dpack[q * 2 + 0] = pack_bf16(d0, d1);
                    dpack[q * 2 + 1] = pack_bf16(d2, d3);
                }
                // dS^T(k) over dS^T(k-1): the issuer of dP^T(k) has seen the dK product of tile k-1 complete
                tmem_st16(T_B + lane_addr + 32 + cP, dpack);
                tmem_wait_st();
            }
            tcgen05_fence_before();
            warp_arrive(&bars[KD_DS], lane);
            warp_arrive(&bars[KD_LEMPTY + s2], lane);
            ++k;
        }
        // ------------------------------------------------------------ epilogue: dV_j, dK_j (32 columns per warpgroup)
        if (k > 0) {
            mbar_wait(&bars[KD_DONE], 0, ab);
            tcgen05_fence_after();
        }
        {
            const int cq = (warp / 4) * 32;       // d = 64: the upper two warpgroups have no columns
            const int jc = jg < n ? jg : 0;
            if (cq < HD) {
#pragma unroll
                for (int which = 0; which < 2; ++which) {
                    __nv_bfloat16 *po = (which == 0 ? a.dV : a.dK) + ((size_t)bh * n + jc) * HD + cq;
                    uint32_t v[32];
                    if (k > 0) {
                        tmem_ld32((which == 0 ? T_dV : T_dK) + lane_addr + cq, v);
                        tmem_wait_ld();
                    } else {
#pragma unroll
                        for (int e = 0; e < 32; ++e) v[e] = 0u;
                    }
                    if (jg < n) {
#pragma unroll
                        for (int e = 0; e < 32; e += 8)
                            *reinterpret_cast<uint4 *>(po + e) =
                                make_uint4(pack_bf16(__uint_as_float(v[e]), __uint_as_float(v[e + 1])),
                                           pack_bf16(__uint_as_float(v[e + 2]), __uint_as_float(v[e + 3])),
                                           pack_bf16(__uint_as_float(v[e + 4]), __uint_as_float(v[e + 5])),
                                           pack_bf16(__uint_as_float(v[e + 6]), __uint_as_float(v[e + 7])));
                    }
                }
            }
        }
    }
    tcgen05_fence_before();
    __syncthreads();
    if (warp == 0) tmem_dealloc(tm, 512);
}

// ---------------------------------------------------------------------------------------
// The fused kernel.  Every 128-query tile is handled as two halves of 64 queries (every barrier exists
// once per half).  Warps 0-15: exp / dS (warpgroups 2h and 2h+1 own the two 32-query quarters of half
// h, so each scheduler has four such warps to hide tensor-memory and MUFU latency); warps 16-23:
// reducers, which do nothing but move finished dQ^T tiles from tensor memory into the fp32
// accumulator, so that the red.global.add queue stalls them and not the warps on the tile loop;
// warp 24 lane 0 issues the products into region A (S^T, dP^T), warp 26 lane 0 the products that read
// P^T and dS^T (dV, dQ^T, dK), warp 25 lane 0 every TMA load; warp 27 only completes that warpgroup.
//
// Tensor memory: region A (128 columns) receives S^T and dP^T in turn, region B (128 columns) holds
// P^T (bf16 pairs, 32 columns per half) and then dQ^T.  An exp / dS thread copies its 32 columns of
// S^T (and later of dP^T) into registers at once and releases region A right away, so the next
// product into A runs while the exponentials (or the dS arithmetic) are still being computed:
//
//   issuer A:  dP^T(k) -> A  (once S^T(k) has been copied out)  |  S^T(k+1) -> A  (once dP^T(k) has been)
//   issuer B:  dV += P^T(k) dO  (P^T(k) written in B)  |  dK += dS^T(k) Q, dQ^T(k) -> B  (dS^T(k) in shared
//              memory, the reducers done with dQ^T(k-1)); dK goes first because it releases the Q / dO stage
//
// The exp / dS warps keep P only as the bf16 pairs they hand to the dV product, and form dS from
// those.  Registers are traded between the warpgroups after launch (setmaxnreg).
template <int N> __device__ __forceinline__ void setmaxnreg_inc() { asm volatile("setmaxnreg.inc.sync.aligned.u32 %0;" ::"n"(N)); }
template <int N> __device__ __forceinline__ void setmaxnreg_dec() { asm volatile("setmaxnreg.dec.sync.aligned.u32 %0;" ::"n"(N)); }
constexpr int kThreadsFused = 512 + 256 + 128;  // 16 exp/dS warps, 8 reducer warps, two issuer warps, TMA producer warp, 1 idle warp
// 72 registers everywhere at launch (896 x 72 = 64,512).  The reducers give up 24 each and work through their
// 64 columns in two steps, the issuer's warpgroup gives up 16, the exp / dS warps take 16:
// 512 x 88 + 256 x 48 + 128 x 56 = 64,512.
struct FusedRegs {
    static constexpr int kExp = 88, kReduce = 48, kIssue = 56;
};
template <int HD, bool FINE>
__global__ void __launch_bounds__(kThreadsFused, 1)
tc_bwd_fused_kernel(const __grid_constant__ CUtensorMap mQ, const __grid_constant__ CUtensorMap mK_,
                 const __grid_constant__ CUtensorMap mV, const __grid_constant__ CUtensorMap mdO,
                 const __grid_constant__ CUtensorMap mdK, const __grid_constant__ CUtensorMap mdV, const BwdArgs a)
{
    // d = 64: the dQ^T product needs M = 128, so the K tile's second 64-wide slab of M is an all-zero slab
    constexpr uint32_t oZero = (BwdSmem<HD>::kBytes + 1023u) & ~1023u;
    constexpr int kHalfWarps = 8;     // exp / dS warps per half
    constexpr int kReduceWarps = 4;   // reducer warps per half
    using L = BwdSmem<HD>;
    static_assert(L::oMisc - L::oBar >= 23 * 8, "barrier area");
    extern __shared__ __align__(1024) uint8_t smem[];
    uint64_t *bars = reinterpret_cast<uint64_t *>(smem + L::oBar);
    uint32_t *tmem_base_s = reinterpret_cast<uint32_t *>(smem + L::oMisc);
    volatile uint32_t *abort_flag = reinterpret_cast<volatile uint32_t *>(smem + L::oMisc + 4);
    const Abort ab{abort_flag, a.status};

    const int tid = threadIdx.x, warp = tid / 32, lane = tid % 32;
    // launch order: heads in groups of `a.group`, inside a group key tile major -- with a causal
    // mask the CTAs of a group then start longest first, which evens out the tail of the grid
    const int jt = blockIdx.x / a.group;
    const long bh = (long)blockIdx.y * a.group + blockIdx.x % a.group;
    const int j0 = jt * TK, n = a.n;

    if ((smem_u32(smem) & 1023u) != 0) {
        if (tid == 0) atomicExch(a.status, 9u);
        return;
    }
    if (tid == 0) {
        *abort_flag = 0;
        mbar_init(&bars[V2_KV], 1);
        for (int h = 0; h < 2; ++h) {
            mbar_init(&bars[V2_QFULL + h], 1);
            mbar_init(&bars[V2_QEMPTY + h], 1);
            mbar_init(&bars[V2_S + h], 1);
            mbar_init(&bars[V2_DP + h], 1);
            mbar_init(&bars[V2_SLD + h], 2 * kHalfWarps);     // SLD, DPLD, DS, DQDONE, DQREL: index 0 serves both halves
            mbar_init(&bars[V2_DPLD + h], 2 * kHalfWarps);
            mbar_init(&bars[V2_P + h], kHalfWarps);
            mbar_init(&bars[V2_DS + h], 2 * kHalfWarps);
            mbar_init(&bars[V2_DQ + h], 1);
            mbar_init(&bars[V2_DQDONE + h], 2 * kReduceWarps);
            mbar_init(&bars[V2_DQREL + h], 2 * kReduceWarps);
        }
        fence_barrier_init();
        prefetch_tensormap(&mQ); prefetch_tensormap(&mK_); prefetch_tensormap(&mV); prefetch_tensormap(&mdO);
    }
    if (HD == 64) {
        for (uint32_t i = tid; i < SLAB / 16; i += kThreadsFused) reinterpret_cast<uint4 *>(smem + oZero)[i] = make_uint4(0, 0, 0, 0);
        fence_proxy_async_smem();
    }
    if (warp == 0) tmem_alloc(tmem_base_s, 512);
    tcgen05_fence_before();
    __syncthreads();
    tcgen05_fence_after();
    const uint32_t tm = *tmem_base_s;
    const uint32_t T_A = tm, T_B = tm + 128, T_dV = tm + 256, T_dK = tm + 256 + HD;
    // d = 64 leaves 128 columns free: dP^T gets a region of its own there, so that S^T(k+1) does not wait for dP^T(k)
    // to be copied out of region A and dP^T(k+1) does not wait for S^T(k+1)
    constexpr bool kSplitA = HD == 64;
    const uint32_t T_A2 = kSplitA ? tm + 384 : T_A;
    constexpr uint32_t HALF_ROWS = 64 * 128;   // byte offset of rows 64.. inside a [128][64] slab

    const TileIter iter(a, jt, bh);

    if (warp >= 24) {
        setmaxnreg_dec<FusedRegs::kIssue>();
        if (warp == 25 && lane == 0) {
            // ------------------------------------------------------------ TMA producer: every load, as soon as its stage is free
            auto issue_load = [&](int it, int s) {
                const int i0 = it * TQ;
                const uint32_t rows = min(TQ, n - i0);
                uint64_t *bar = &bars[V2_QFULL + s];
                mbar_expect_tx(bar, 2 * L::kTile + 2 * rows * 4);
#pragma unroll
                for (uint32_t sl = 0; sl < L::kSlabs; ++sl) {
                    tma_load_3d(smem + L::oQ + s * L::kTile + sl * SLAB, &mQ, bar, sl * 64, i0, (int)bh);
                    tma_load_3d(smem + L::odO + s * L::kTile + sl * SLAB, &mdO, bar, sl * 64, i0, (int)bh);
                }
                bulk_load_1d(smem + L::oLSE + s * 512, a.nLSE2 + bh * n + i0, rows * 4, bar);
                bulk_load_1d(smem + L::oD + s * 512, a.Ds + bh * n + i0, rows * 4, bar);
            };
            mbar_expect_tx(&bars[V2_KV], 2 * L::kTile);
#pragma unroll
            for (uint32_t sl = 0; sl < L::kSlabs; ++sl) {
                tma_load_3d(smem + L::oK + sl * SLAB, &mK_, &bars[V2_KV], sl * 64, j0, (int)bh);
                tma_load_3d(smem + L::oV + sl * SLAB, &mV, &bars[V2_KV], sl * 64, j0, (int)bh);
            }
            int k = 0;
            for (int idx = 0; idx < iter.raw; ++idx) {
                const int it = iter.tile(idx);
                if (it < 0) continue;
                const int s = k & 1;
                if (k >= 2) mbar_wait(&bars[V2_QEMPTY + s], ((k - 2) >> 1) & 1, ab);   // last read by dK of tile k-2
                issue_load(it, s);
                ++k;
            }
            // a key tile without a single query tile (an empty block column): nobody else waits for K_j and V_j, and
            // the CTA must not exit with their bulk loads still in flight into its shared memory
            if (k == 0) mbar_wait(&bars[V2_KV], 0, ab);
        } else if (warp == 24 && lane == 0) {
            // ------------------------------------------------------------ MMA issuer A: the products into region A (S^T, dP^T)
            constexpr uint32_t idesc_s = idesc_bf16(128, 128, 0, 0);
            // low descriptor words (tc_common.cuh): per-step offsets are added as (bytes >> 4)
            const uint32_t kK = desc_lo_kmajor(smem_u32(smem + L::oK)), kV = desc_lo_kmajor(smem_u32(smem + L::oV));
            constexpr uint32_t kSlab = SLAB >> 4;
            // S^T = K_j Q_i^T for the whole tile in stage s
            auto issue_S = [&](int s) {
                const uint32_t kQ = desc_lo_kmajor(smem_u32(smem + L::oQ + s * L::kTile));
#pragma unroll
                for (int kk = 0; kk < HD / 16; ++kk) {
                    const uint32_t off = (kk / 4) * kSlab + (kk % 4) * 2;
                    mma_ss_lo(T_A, kK + off, kQ + off, idesc_s, kk > 0);
                }
                mma_commit(&bars[V2_S]);
            };
            // dP^T = V_j dO_i^T for the whole tile in stage s
            auto issue_dP = [&](int s) {
                const uint32_t kdO = desc_lo_kmajor(smem_u32(smem + L::odO + s * L::kTile));
#pragma unroll
                for (int kk = 0; kk < HD / 16; ++kk) {
                    const uint32_t off = (kk / 4) * kSlab + (kk % 4) * 2;
                    mma_ss_lo(T_A2, kV + off, kdO + off, idesc_s, kk > 0);
                }
                mma_commit(&bars[V2_DP]);
            };
            int idx = 0, it = -1;
            while (idx < iter.raw && (it = iter.tile(idx)) < 0) ++idx;
            if (it >= 0) {
                mbar_wait(&bars[V2_QFULL], 0, ab);
                mbar_wait(&bars[V2_KV], 0, ab);
                tcgen05_fence_after();
                issue_S(0);
                if (kSplitA) issue_dP(0);
            }
            int k = 0;
            while (idx < iter.raw) {
                const int s = k & 1;
                int nidx = idx + 1, nit = -1;
                while (nidx < iter.raw && (nit = iter.tile(nidx)) < 0) ++nidx;
                if constexpr (kSplitA) {
                    // two regions: S^T(k+1) as soon as S^T(k) has been copied out, dP^T(k+1) as soon as dP^T(k) has been
                    if (nit >= 0) {
                        mbar_wait(&bars[V2_SLD], k & 1, ab);
                        mbar_wait(&bars[V2_QFULL + (s ^ 1)], ((k + 1) >> 1) & 1, ab);
                        tcgen05_fence_after();
                        issue_S(s ^ 1);
                        mbar_wait(&bars[V2_DPLD], k & 1, ab);
                        tcgen05_fence_after();
                        issue_dP(s ^ 1);
                    }
                } else {
                    // dP^T = V_j dO_i^T into region A once every exp / dS warp holds its part of S^T in registers
                    mbar_wait(&bars[V2_SLD], k & 1, ab);
                    tcgen05_fence_after();
                    issue_dP(s);
                    // S^T of the next tile into region A as soon as dP^T has been read out of it
                    if (nit >= 0) {
                        mbar_wait(&bars[V2_DPLD], k & 1, ab);
                        mbar_wait(&bars[V2_QFULL + (s ^ 1)], ((k + 1) >> 1) & 1, ab);
                        tcgen05_fence_after();
                        issue_S(s ^ 1);
                    }
                }
                ++k;
                idx = nidx;
            }
        } else if (warp == 26 && lane == 0) {
            // ------------------------------------------------------------ MMA issuer B: the products that read P^T and dS^T
            // (dV, dQ^T into region B, dK).  Two issuing threads, because a thread that waits on a barrier or commits
            // cannot keep the short queue of the tensor pipe filled; everything that orders A's products against B's
            // goes through the exp / dS warps' barriers.
            constexpr uint32_t idesc_dv = idesc_bf16(128, HD, 0, 1);       // dV (A tmem), dK (A K-major smem)
            constexpr uint32_t idesc_dq = idesc_bf16(128, 128, 1, 1);      // dQ^T
            const uint32_t mK = desc_lo_mnmajor(smem_u32(smem + L::oK), HD == 64 ? oZero - L::oK : SLAB);
            const uint32_t kdS = desc_lo_kmajor(smem_u32(smem + L::odS)), mdS = desc_lo_mnmajor(smem_u32(smem + L::odS), SLAB);
            constexpr uint32_t kHalf = HALF_ROWS >> 4, kSlab = SLAB >> 4;
            int k = 0;
            for (int idx = 0; idx < iter.raw; ++idx) {
                if (iter.tile(idx) < 0) continue;
                const int s = k & 1;
                const uint32_t mdO_ = desc_lo_mnmajor(smem_u32(smem + L::odO + s * L::kTile), SLAB);
                const uint32_t mQ_ = desc_lo_mnmajor(smem_u32(smem + L::oQ + s * L::kTile), SLAB);
                if (k == 0) mbar_wait(&bars[V2_KV], 0, ab);
                mbar_wait(&bars[V2_QFULL + s], (k >> 1) & 1, ab);
                // dV += P_h^T dO_h, P_h^T in columns 64 h .. 64 h + 31 of region B
#pragma unroll
                for (int h = 0; h < 2; ++h) {
                    mbar_wait(&bars[V2_P + h], k & 1, ab);
                    tcgen05_fence_after();
#pragma unroll
                    for (int kk = 0; kk < 4; ++kk)
                        mma_ts_lo(T_dV, T_B + 64 * h + kk * 8, mdO_ + h * kHalf + kk * 128, idesc_dv, (k > 0) || (h > 0) || (kk > 0));
                }
                // dK += dS^T Q_i first: its completion releases the Q / dO stage, and the load of the tile after next --
                // two stages only -- is what the next S^T product ends up waiting for.  Then dQ^T = K_j^T dS^T into
                // region B (this thread's products execute in issue order, so dV has consumed P^T by then)
                mbar_wait(&bars[V2_DS], k & 1, ab);
                if (k > 0) {   // the reducers have read all of the previous dQ^T
                    mbar_wait(&bars[V2_DQDONE], (k - 1) & 1, ab);
                }
                tcgen05_fence_after();
#pragma unroll
                for (int kk = 0; kk < TQ / 16; ++kk)
                    mma_ss_lo(T_dK, kdS + (kk / 4) * kSlab + (kk % 4) * 2, mQ_ + kk * 128, idesc_dv, (k > 0) || (kk > 0));
                mma_commit(&bars[V2_QEMPTY + s]);
#pragma unroll
                for (int kk = 0; kk < TK / 16; ++kk)
                    mma_ss_lo(T_B, mK + kk * 128, mdS + kk * 128, idesc_dq, kk > 0);
                mma_commit(&bars[V2_DQ]);
                ++k;
            }
        }
    } else if (warp >= 16) {
        setmaxnreg_dec<FusedRegs::kReduce>();
        // ------------------------------------------------------------ reducers: dQ_h^T tile -> fp32 accumulator
        // lanes = head-dimension index c, columns = queries: one warp instruction adds 128 contiguous bytes.
        // 32 columns at a time (the reducers run on 48 registers); the half is released after the second load
        const int h = (warp - 16) / 4;
        const int row = (warp % 4) * 32 + lane;
        const uint32_t lane_addr = (uint32_t)((warp % 4) * 32) << 16;
        const bool live = (warp % 4) * 32 < HD;   // d = 64: lanes 64..127 of the padded product hold zeros
        int k = 0;
        for (int idx = 0; idx < iter.raw; ++idx) {
            const int it = iter.tile(idx);
            if (it < 0) continue;
            const int ig0 = it * TQ + h * 64;
            float *base = a.dQ_acc + ((size_t)bh * n + ig0) * HD + row;
            mbar_wait(&bars[V2_DQ], k & 1, ab);
            tcgen05_fence_after();
#pragma unroll
            for (int part = 0; part < 2; ++part) {
                uint32_t v0[32];
                if (live) {
                    tmem_ld32(T_B + lane_addr + h * 64 + part * 32, v0);
                    tmem_wait_ld();
                }
                tcgen05_fence_before();
                // part 0: the 32 columns that take P^T of the next tile are free; part 1: the whole half is
                warp_arrive(&bars[part == 0 ? V2_DQREL : V2_DQDONE], lane);
                if (live) {
                    if (ig0 + 64 <= n) {
#pragma unroll
                        for (int e = 0; e < 32; ++e) red_add_f32(base + (size_t)(part * 32 + e) * HD, __uint_as_float(v0[e]));
                    } else {
#pragma unroll
                        for (int e = 0; e < 32; ++e)
                            if (ig0 + part * 32 + e < n) red_add_f32(base + (size_t)(part * 32 + e) * HD, __uint_as_float(v0[e]));
                    }
                }
            }
            ++k;
        }
    } else {
        // ------------------------------------------------------------ warps 0-15: exp / dS; warpgroup 2h + qq owns queries 64 h + 32 qq .. + 31
        setmaxnreg_inc<FusedRegs::kExp>();
        const int h = warp / 8, qq = (warp / 4) & 1;
        const int row = (warp % 4) * 32 + lane;        // tensor-memory lane = key row inside the tile
        const uint32_t lane_addr = (uint32_t)((warp % 4) * 32) << 16;
        const int jg = j0 + row;
        const float sl2 = a.scale * 1.4426950408889634f;
        const uint32_t c0 = h * 64 + qq * 32;          // this thread's first column of S^T / dP^T in region A
        const uint32_t cP = h * 64 + qq * 16;          // and of its bf16 pairs of P^T in region B
        int k = 0;
        for (int idx = 0; idx < iter.raw; ++idx) {
            const int it = iter.tile(idx);
            if (it < 0) continue;
            const int s = k & 1, i0 = it * TQ;
            const float4 *sNL = reinterpret_cast<const float4 *>(smem + L::oLSE + s * 512 + h * 256 + qq * 128);
            const float4 *sDs = reinterpret_cast<const float4 *>(smem + L::oD + s * 512 + h * 256 + qq * 128);
            const bool diag = mask_is_causal(a.mask_kind) && it == jt;
            const int ig0 = i0 + h * 64 + qq * 32;
            // a mask finer than the tile: the keep bits of this thread's key row and its 32 query columns
            uint32_t kw = 0xffffffffu;
            if constexpr (FINE) kw = (ig0 < n && jg < n) ? fine_word(a.fine, a.mask_heads, bh, false, jg, ig0) : 0u;
            const bool masked = diag || i0 + TQ > n || j0 + TK > n || FINE;
            mbar_wait(&bars[V2_QFULL + s], (k >> 1) & 1, ab);
            // the 32 row statistics of this thread's query columns go into registers before the wait for S^T: while the
            // products stream their operands, a shared-memory load inside the arithmetic below waits a few hundred cycles
            float4 nlr[8];
#pragma unroll
            for (int q = 0; q < 8; ++q) nlr[q] = sNL[q];
            mbar_wait(&bars[V2_S], k & 1, ab);
            tcgen05_fence_after();
            uint32_t ppack[16];   // P as bf16 pairs: what dV uses, and what dS is formed from
            {
                uint32_t sv[32];
                tmem_ld32(T_A + lane_addr + c0, sv);
                tmem_wait_ld();
                tcgen05_fence_before();
                warp_arrive(&bars[V2_SLD], lane);   // region A may take dP^T
#pragma unroll
                for (int q = 0; q < 8; ++q) {
                    const float4 nl = nlr[q];
                    float p[4];
                    p[0] = ex2_approx(fmaf(__uint_as_float(sv[q * 4 + 0]), sl2, nl.x));
                    p[1] = ex2_approx(fmaf(__uint_as_float(sv[q * 4 + 1]), sl2, nl.y));
                    p[2] = ex2_approx(fmaf(__uint_as_float(sv[q * 4 + 2]), sl2, nl.z));
                    p[3] = ex2_approx(fmaf(__uint_as_float(sv[q * 4 + 3]), sl2, nl.w));
                    if (masked) {
#pragma unroll
                        for (int e = 0; e < 4; ++e) {
                            const int ig = ig0 + q * 4 + e;
                            const bool ok = ig < n && jg < n && (!diag || jg <= ig) && ((kw >> (q * 4 + e)) & 1u);
                            p[e] = ok ? p[e] : 0.f;
                        }
                    }
                    ppack[q * 2 + 0] = pack_bf16(p[0], p[1]);
                    ppack[q * 2 + 1] = pack_bf16(p[2], p[3]);
                }
            }
            float4 dsr[8];   // scale * D of the same columns, again ahead of the wait
#pragma unroll
            for (int q = 0; q < 8; ++q) dsr[q] = sDs[q];
            // P^T goes into region B before dP^T is awaited: a tensor-memory store issued while products run takes
            // several hundred cycles, which now pass during that wait.  Its first 32 columns per half held dQ^T of the
            // previous tile; the reducers release them after their first load
            if (k > 0) {
                mbar_wait(&bars[V2_DQREL], (k - 1) & 1, ab);
                tcgen05_fence_after();
            }
            tmem_st16(T_B + lane_addr + cP, ppack);
            mbar_wait(&bars[V2_DP], k & 1, ab);
            tcgen05_fence_after();
            {
                uint8_t *slab = smem + L::odS + h * SLAB;
                uint32_t dv[32];
                tmem_ld32(T_A2 + lane_addr + c0, dv);
                tmem_wait_ld();
                tcgen05_fence_before();
                warp_arrive(&bars[V2_DPLD], lane);   // region A may take the next S^T
                tmem_wait_st();
                tcgen05_fence_before();
                warp_arrive(&bars[V2_P + h], lane);
                // dS^T(k) goes over dS^T(k-1), which the dK and dQ^T products of tile k-1 read from shared memory.  Both
                // have completed: the reducers release their columns (awaited above) only after dQ^T(k-1), the later of
                // the two in the other thread's issue order, has landed
#pragma unroll
                for (int g = 0; g < 4; ++g) {    // 8 query columns = one 16-byte chunk
                    float ds[8], p[8];
#pragma unroll
                    for (int e = 0; e < 4; ++e) {
                        const uint32_t pk = ppack[g * 4 + e];   // bf16 -> fp32 is a 16-bit shift
                        p[2 * e] = __uint_as_float(pk << 16);
                        p[2 * e + 1] = __uint_as_float(pk & 0xffff0000u);
                    }
#pragma unroll
                    for (int u = 0; u < 2; ++u) {
                        const float4 dsc = dsr[g * 2 + u];
                        const uint32_t *d4 = &dv[g * 8 + u * 4];
                        ds[u * 4 + 0] = p[u * 4 + 0] * fmaf(__uint_as_float(d4[0]), a.scale, -dsc.x);
                        ds[u * 4 + 1] = p[u * 4 + 1] * fmaf(__uint_as_float(d4[1]), a.scale, -dsc.y);
                        ds[u * 4 + 2] = p[u * 4 + 2] * fmaf(__uint_as_float(d4[2]), a.scale, -dsc.z);
                        ds[u * 4 + 3] = p[u * 4 + 3] * fmaf(__uint_as_float(d4[3]), a.scale, -dsc.w);
                    }
                    if (masked) {   // stale tail entries of the row vectors may be anything: select, do not multiply
#pragma unroll
                        for (int e = 0; e < 8; ++e) ds[e] = p[e] != 0.f ? ds[e] : 0.f;
                    }
                    *reinterpret_cast<uint4 *>(slab + sw128_offset(row, qq * 32 + g * 8)) =
                        make_uint4(pack_bf16(ds[0], ds[1]), pack_bf16(ds[2], ds[3]), pack_bf16(ds[4], ds[5]),
                                   pack_bf16(ds[6], ds[7]));
                }
            }
            fence_proxy_async_smem();
            warp_arrive(&bars[V2_DS], lane);
            ++k;
        }
        // ------------------------------------------------------------ epilogue: dV_j, dK_j (32 columns per warpgroup)
        if (k > 0) {
            // dV and dK of the last tile have completed when its stage is released (dQ^T, queued after them, is the
            // reducers' business and reads neither accumulator nor the stages reused below)
            mbar_wait(&bars[V2_QEMPTY + ((k - 1) & 1)], ((k - 1) >> 1) & 1, ab);
            tcgen05_fence_after();
        }
        {
            // dV_j and dK_j go out through shared memory and TMA stores (coalesced; rows beyond n are clipped): the
            // first Q and dO stages are free by now -- every product that read them has completed.  Each thread packs
            // 32 columns of its key row into the swizzled slab layout the store expects.
            const int cq = (warp / 4) * 32;        // d = 64: the upper two warpgroups have no columns
            if (cq < HD) {
#pragma unroll
                for (int which = 0; which < 2; ++which) {
                    uint32_t v[32];
                    if (k > 0) {
                        tmem_ld32((which == 0 ? T_dV : T_dK) + lane_addr + cq, v);
                        tmem_wait_ld();
                    } else {
#pragma unroll
                        for (int e = 0; e < 32; ++e) v[e] = 0u;
                    }
                    uint8_t *slab = smem + (which == 0 ? L::oQ : L::odO) + (cq / 64) * SLAB;
#pragma unroll
                    for (int e = 0; e < 32; e += 8)
                        *reinterpret_cast<uint4 *>(slab + sw128_offset(row, (cq % 64) + e)) =
                            make_uint4(pack_bf16(__uint_as_float(v[e]), __uint_as_float(v[e + 1])),
                                       pack_bf16(__uint_as_float(v[e + 2]), __uint_as_float(v[e + 3])),
                                       pack_bf16(__uint_as_float(v[e + 4]), __uint_as_float(v[e + 5])),
                                       pack_bf16(__uint_as_float(v[e + 6]), __uint_as_float(v[e + 7])));
                }
            }
            fence_proxy_async_smem();
            asm volatile("bar.sync 1, 512;" ::: "memory");   // the sixteen exp / dS warps
            if (tid == 0) {
#pragma unroll
                for (uint32_t sl = 0; sl < L::kSlabs; ++sl) {
                    tma_store_3d(&mdV, smem + L::oQ + sl * SLAB, sl * 64, j0, (int)bh);
                    tma_store_3d(&mdK, smem + L::odO + sl * SLAB, sl * 64, j0, (int)bh);
                }
                tma_store_commit();
                tma_store_wait_read();   // the slabs have been read; the writes complete with the grid
            }
        }
    }
    tcgen05_fence_before();
    __syncthreads();
    if (warp == 0) tmem_dealloc(tm, 512);
}

// fp32 accumulator -> bf16 dQ
__global__ void __launch_bounds__(256) dq_convert_kernel(const float4 *__restrict__ acc, uint2 *__restrict__ out, size_t n4)
{
    for (size_t i = (size_t)blockIdx.x * blockDim.x + threadIdx.x; i < n4; i += (size_t)gridDim.x * blockDim.x) {
        const float4 v = acc[i];
        out[i] = make_uint2(pack_bf16(v.x, v.y), pack_bf16(v.z, v.w));
    }
}

template <int HD, bool WITH_DQ>
attn_status launch_bwd(const Problem &p)
{
    using L = BwdSmem<HD>;
    CUtensorMap mQ, mK, mV, mdO;
    const uint64_t BH = (uint64_t)p.BH;
    if (!make_tmap_bf16_3d(&mQ, p.Q, HD, p.n, BH, 128) || !make_tmap_bf16_3d(&mK, p.K, HD, p.n, BH, 128) ||
        !make_tmap_bf16_3d(&mV, p.V, HD, p.n, BH, 128) || !make_tmap_bf16_3d(&mdO, p.dO, HD, p.n, BH, 128))
        return ATTN_ERR_LAUNCH;
    BwdArgs a{};
    a.nLSE2 = p.nLSE2; a.Ds = p.D; a.dQ_acc = p.dQ_acc;
    a.dK = (__nv_bfloat16 *)p.dK; a.dV = (__nv_bfloat16 *)p.dV;
    a.n = p.n; a.BH = (int)p.BH;
    a.mask_kind = p.mask_kind; a.block = p.block; a.nb = p.nb; a.mask_heads = p.mask_heads; a.fine = p.fine;
    a.col_ptr = p.col_ptr; a.row_idx = p.row_idx;
    a.scale = p.scale;
    a.status = p.status;
    a.group = bwd_head_group(p);
    if (bwd_preprocess_launch(p, WITH_DQ) != ATTN_OK) return ATTN_ERR_LAUNCH;
    const dim3 grid((unsigned)((p.n + TK - 1) / TK * a.group), (unsigned)(p.BH / a.group));
    launch_begin(WITH_DQ ? "tc_bwd_fused" : "tc_bwd_dkdv", p.stream);
    if (WITH_DQ) {
        constexpr uint32_t bytes = HD == 64 ? ((L::kBytes + 1023u) & ~1023u) + SLAB : L::kBytes;
        auto kernel = p.fine.mode ? tc_bwd_fused_kernel<HD, true> : tc_bwd_fused_kernel<HD, false>;
        if (cudaFuncSetAttribute(kernel, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)bytes) != cudaSuccess)
            return ATTN_ERR_LAUNCH;
        CUtensorMap mdK, mdV;
        if (!make_tmap_bf16_3d(&mdK, p.dK, HD, p.n, BH, 128) || !make_tmap_bf16_3d(&mdV, p.dV, HD, p.n, BH, 128)) return ATTN_ERR_LAUNCH;
        kernel<<<grid, kThreadsFused, bytes, p.stream>>>(mQ, mK, mV, mdO, mdK, mdV, a);
    } else {
        if (cudaFuncSetAttribute(tc_bwd_dkdv_kernel<HD>, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)DkdvSmem<HD>::kBytes) != cudaSuccess)
            return ATTN_ERR_LAUNCH;
        tc_bwd_dkdv_kernel<HD><<<grid, kThreadsDkdv, DkdvSmem<HD>::kBytes, p.stream>>>(mQ, mK, mV, mdO, a);
    }
    launch_end(p.stream);
    if (cudaGetLastError() != cudaSuccess) return ATTN_ERR_LAUNCH;
    if (!WITH_DQ) return tc_bwd_dq(p);   // deterministic path: dQ without atomics, from its own kernel
    return bwd_dq_convert_launch(p);
}

}  // namespace

// Heads are launched in groups (key tile major inside a group).  The fp32 dQ accumulators of the heads that run
// at the same time should stay in L2 between the reductions of one key tile and the next: otherwise every reduced
// sector is fetched from and written back to device memory (measured on the block-sparse workload with n = 32768:
// 13 times the compulsory traffic with 8 heads in flight).  So the group is the largest of 8, 4, 2, 1 that divides
// the head count and whose accumulators take at most kAccBudget bytes.
int bwd_head_group(const Problem &p)
{
    constexpr size_t kAccBudget = 40u << 20;
    for (int g = 8; g > 1; g >>= 1)
        if (p.BH % g == 0 && (size_t)g * p.n * p.d * sizeof(float) <= kAccBudget) return g;
    return 1;
}

namespace {
template <int HD>
attn_status preprocess_launch_t(const Problem &p, bool clear_acc)
{
    const size_t rows = (size_t)p.BH * p.n, acc_elems = rows * HD;
    constexpr size_t rpw = 32 / (HD / 8);
    size_t blocks = ((rows + rpw - 1) / rpw + 7) / 8;
    if (blocks > (size_t)sm_count() * 8) blocks = (size_t)sm_count() * 8;
    launch_begin("tc_bwd_preprocess", p.stream);
    tc_preprocess_kernel<HD><<<(unsigned)blocks, 256, 0, p.stream>>>((const __nv_bfloat16 *)p.O, (const __nv_bfloat16 *)p.dO,
                                                                     p.LSE, p.D, p.nLSE2, rows, p.scale,
                                                                     clear_acc ? (uint4 *)p.dQ_acc : nullptr, acc_elems / 4);
    launch_end(p.stream);
    return cudaGetLastError() == cudaSuccess ? ATTN_OK : ATTN_ERR_LAUNCH;
}
}  // namespace

attn_status bwd_preprocess_launch(const Problem &p, bool clear_acc)
{
    if (p.d == 64) return preprocess_launch_t<64>(p, clear_acc);
    if (p.d == 128) return preprocess_launch_t<128>(p, clear_acc);
    if (p.d == 256) return preprocess_launch_t<256>(p, clear_acc);
    return ATTN_ERR_TILE;
}

attn_status bwd_dq_convert_launch(const Problem &p)
{
    if (!p.dQ) return ATTN_OK;   // the caller reads the fp32 accumulator itself
    const size_t n4 = (size_t)p.BH * p.n * p.d / 4;
    const size_t cap = (size_t)sm_count() * 16;
    const unsigned blocks = (unsigned)((n4 + 255) / 256 < cap ? (n4 + 255) / 256 : cap);
    launch_begin("bwd_dq_convert", p.stream);
    dq_convert_kernel<<<blocks, 256, 0, p.stream>>>((const float4 *)p.dQ_acc, (uint2 *)p.dQ, n4);
    launch_end(p.stream);
    return cudaGetLastError() == cudaSuccess ? ATTN_OK : ATTN_ERR_LAUNCH;
}

size_t bwd_smem_bytes(int d) { return d == 64 ? BwdSmem<64>::kBytes : d == 128 ? BwdSmem<128>::kBytes : 0; }

attn_status tc_bwd(const Problem &p)
{
    if (p.cfg.tile_q == 64 || p.d == 256) return tc_bwd64(p);
    if (p.d == 64) return p.cfg.deterministic ? launch_bwd<64, false>(p) : launch_bwd<64, true>(p);
    if (p.d == 128) return p.cfg.deterministic ? launch_bwd<128, false>(p) : launch_bwd<128, true>(p);
    return ATTN_ERR_TILE;
}

}  // namespace attn

// Fused backward with 64-query tiles (large-cache regime of Appendix D at a smaller on-chip
// size M): the second tile shape of the key-stationary algorithm, and the only fused shape
// that fits a head dimension of 256.
//
// A CTA owns one tile of 128 KEYS j and, at d = 256, one HALF c of the head dimension of the
// results: dK_j[:, 128 c .. 128 c + 127] and dV_j[:, ...] stay in tensor memory (2 x 128 columns),
// and the CTA produces the same column half of the dQ tiles.  It walks the kept tiles of 64
// QUERIES i.  Per (i, j), everything transposed so that the tensor-memory lane is the key index:
//
//   S^T  = K_j Q_i^T                 contraction over the WHOLE head dimension (both CTAs of a
//   dP^T = V_j dO_i^T                key tile at d = 256 form them: 7 product units for 5)
//   P^T  = exp2(S^T scale log2e - LSE_i log2e),  dS^T = scale P^T o (dP^T - D_i)   (Definition B.9)
//   dV_j[:, c] += P^T  dO_i[:, c]    A = P^T from tensor memory (bf16, written over S^T)
//   dK_j[:, c] += dS^T Q_i[:, c]     A = dS^T from shared memory
//   dQ_i[:, c] += dS K_j[:, c]       as dQ^T (lane = head-dimension index) = K_j[:, c]^T dS^T, added to
//                                    the fp32 accumulator with coalesced red.global.add
//
// Shared memory: K_j; V_j (d = 128) -- at d = 256 V_j lives in tensor memory instead (128 columns
// of bf16 pairs, copied there once; it is only ever the A operand of dP^T), which is what leaves
// room for two Q / dO stages; Q_i and dO_i stages of 64 rows; dS^T (128 x 64).
// Tensor memory (512 columns): dV 128 | dK 128 | RS 64 (S^T, then P^T in place) | RD 64 (dP^T, then
// dQ^T) | V_j 128 (d = 256 only).
//
// Roles: warps 0-7 exp / dS (lane quarter = warp % 4, 32 query columns each), warps 8-11 reducers
// (dQ^T tile -> registers -> fp32 accumulator), warp 12 lane 0 issues every product in a fixed
// order, warp 13 lane 0 every TMA load.  All waits are bounded (tc_common.cuh).
#include "tc_bwd_common.cuh"

namespace attn {
namespace {

using namespace tc;
using namespace bwdk;

constexpr int TQ64 = 64;
constexpr uint32_t SLAB = 128 * 128;     // [128 rows][64 bf16]
constexpr uint32_t SLAB64 = 64 * 128;    // [64 rows][64 bf16]
constexpr int kThreads64 = 8 * 32 + 4 * 32 + 2 * 32;

template <int HD>
struct B64 {
    static constexpr bool kVinTmem = HD == 256;
    static constexpr int HA = HD < 128 ? HD : 128;            // accumulator columns per CTA
    static constexpr int kSplit = HD / HA;                    // CTAs per key tile
    static constexpr int NS = HD == 256 ? 2 : 4;              // Q / dO stages
    static constexpr uint32_t kSlabs = HD / 64;
    static constexpr uint32_t kKTile = kSlabs * SLAB;         // [128][HD]
    static constexpr uint32_t kQTile = kSlabs * SLAB64;       // [64][HD]
    static constexpr uint32_t oK = 0;
    static constexpr uint32_t oV = oK + kKTile;               // absent when V_j lives in tensor memory
    static constexpr uint32_t oQ = oV + (kVinTmem ? 0 : kKTile);
    static constexpr uint32_t odO = oQ + NS * kQTile;
    static constexpr uint32_t odS = odO + NS * kQTile;        // [128 keys][64 queries]
    static constexpr uint32_t oLSE = odS + SLAB;              // NS x 64 floats
    static constexpr uint32_t oD = oLSE + NS * 256;
    static constexpr uint32_t oBar = oD + NS * 256;
    static constexpr uint32_t oMisc = oBar + 32 * 8;
    static constexpr uint32_t kUsed = oMisc + 64;
    static_assert(!kVinTmem || NS * kQTile == kKTile, "V_j is staged in the Q stages before it moves to tensor memory");
    static_assert(kUsed <= 227 * 1024, "shared memory budget");
    static constexpr uint32_t kBytes = kUsed < 117 * 1024 ? 117 * 1024 : kUsed;   // one CTA per SM
};

enum { B_KV = 0, B_VDONE = 1, B_S = 2, B_DP = 3, B_P = 4, B_DS = 5, B_DQ = 6, B_DQDONE = 7, B_DONE = 8,
       B_QFULL = 9, B_QEMPTY = 13 };

template <int HD>
__global__ void __launch_bounds__(kThreads64, 1)
tc_bwd_fused64_kernel(const __grid_constant__ CUtensorMap mQ, const __grid_constant__ CUtensorMap mK_,
                      const __grid_constant__ CUtensorMap mV, const __grid_constant__ CUtensorMap mdO, const BwdArgs a)
{
    using L = B64<HD>;
    constexpr int HA = L::HA, NS = L::NS;
    constexpr int kExpWarps = 8, kReduceWarps = 4;
    extern __shared__ __align__(1024) uint8_t smem[];
    uint64_t *bars = reinterpret_cast<uint64_t *>(smem + L::oBar);
    uint32_t *tmem_base_s = reinterpret_cast<uint32_t *>(smem + L::oMisc);
    volatile uint32_t *abort_flag = reinterpret_cast<volatile uint32_t *>(smem + L::oMisc + 4);
    const Abort ab{abort_flag, a.status};

    const int tid = threadIdx.x, warp = tid / 32, lane = tid % 32;
    // launch order as in the 128-query kernel: heads in groups, key tile major inside a group
    const int jt = blockIdx.x / a.group;
    const long bh = (long)blockIdx.y * a.group + blockIdx.x % a.group;
    const int c = blockIdx.z;                    // which 128 columns of the head dimension this CTA owns
    const int j0 = jt * TK, n = a.n;

    if ((smem_u32(smem) & 1023u) != 0) {
        if (tid == 0) atomicExch(a.status, 9u);
        return;
    }
    if (tid == 0) {
        *abort_flag = 0;
        mbar_init(&bars[B_KV], 1);
        mbar_init(&bars[B_VDONE], kExpWarps);
        mbar_init(&bars[B_S], 1);
        mbar_init(&bars[B_DP], 1);
        mbar_init(&bars[B_P], kExpWarps);
        mbar_init(&bars[B_DS], kExpWarps);
        mbar_init(&bars[B_DQ], 1);
        mbar_init(&bars[B_DQDONE], kReduceWarps);
        mbar_init(&bars[B_DONE], 1);
        for (int s = 0; s < NS; ++s) { mbar_init(&bars[B_QFULL + s], 1); mbar_init(&bars[B_QEMPTY + s], 1); }
        fence_barrier_init();
        prefetch_tensormap(&mQ); prefetch_tensormap(&mK_); prefetch_tensormap(&mV); prefetch_tensormap(&mdO);
    }
    if (warp == 0) tmem_alloc(tmem_base_s, 512);
    tcgen05_fence_before();
    __syncthreads();
    tcgen05_fence_after();
    const uint32_t tm = *tmem_base_s;
    const uint32_t T_dV = tm, T_dK = tm + HA, T_RS = tm + 2 * HA, T_RD = tm + 2 * HA + 64, T_V = tm + 2 * HA + 128;

    const TileIterT<TQ64> iter(a, jt, bh);
    int T = 0;   // number of query tiles this CTA visits (same in every role)
    for (int idx = 0; idx < iter.raw; ++idx) T += iter.tile(idx) >= 0;

    if (warp == 13) {
        // ------------------------------------------------------------ TMA producer
        if (lane == 0) {
            mbar_expect_tx(&bars[B_KV], 2 * L::kKTile);
#pragma unroll
            for (uint32_t sl = 0; sl < L::kSlabs; ++sl) {
                tma_load_3d(smem + L::oK + sl * SLAB, &mK_, &bars[B_KV], sl * 64, j0, (int)bh);
                tma_load_3d(smem + (L::kVinTmem ? L::oQ : L::oV) + sl * SLAB, &mV, &bars[B_KV], sl * 64, j0, (int)bh);
            }
            // V_j was staged where the Q stages are: they are free once the exp / dS warps have moved it
            if (L::kVinTmem && T > 0) mbar_wait(&bars[B_VDONE], 0, ab);
            int t = 0;
            for (int idx = 0; idx < iter.raw; ++idx) {
                const int it = iter.tile(idx);
                if (it < 0) continue;
                const int s = t % NS, i0 = it * TQ64;
                const uint32_t rows = min(TQ64, n - i0);
                if (t >= NS) mbar_wait(&bars[B_QEMPTY + s], ((t / NS) - 1) & 1, ab);
                uint64_t *bar = &bars[B_QFULL + s];
                mbar_expect_tx(bar, 2 * L::kQTile + 2 * rows * 4);
#pragma unroll
                for (uint32_t sl = 0; sl < L::kSlabs; ++sl)
                    tma_load_3d(smem + L::oQ + s * L::kQTile + sl * SLAB64, &mQ, bar, sl * 64, i0, (int)bh);
#pragma unroll
                for (uint32_t sl = 0; sl < L::kSlabs; ++sl)
                    tma_load_3d(smem + L::odO + s * L::kQTile + sl * SLAB64, &mdO, bar, sl * 64, i0, (int)bh);
                bulk_load_1d(smem + L::oLSE + s * 256, a.nLSE2 + bh * n + i0, rows * 4, bar);
                bulk_load_1d(smem + L::oD + s * 256, a.Ds + bh * n + i0, rows * 4, bar);
                ++t;
            }
            // nobody else waits for K_j / V_j when there is no tile: do not exit with their loads in flight
            if (T == 0) mbar_wait(&bars[B_KV], 0, ab);
        }
    } else if (warp == 12) {
        // ------------------------------------------------------------ MMA issuer: every product, in a fixed order
        if (lane == 0 && T > 0) {
            constexpr uint32_t idesc_s = idesc_bf16(128, 64, 0, 0);        // S^T, dP^T: N = 64 queries
            constexpr uint32_t idesc_acc = idesc_bf16(128, HA, 0, 1);      // dV, dK: B MN-major
            constexpr uint32_t idesc_dq = idesc_bf16(128, 64, 1, 1);       // dQ^T: both MN-major
            constexpr uint32_t kSlab = SLAB >> 4, kSlab64 = SLAB64 >> 4;
            const uint32_t kK = desc_lo_kmajor(smem_u32(smem + L::oK));
            const uint32_t kV = desc_lo_kmajor(smem_u32(smem + L::oV));   // unused when V_j is in tensor memory
            // K_j[:, c]^T: M = 128 head-dimension indices (two 64-wide slabs of the K tile), contraction over the keys
            const uint32_t mK = desc_lo_mnmajor(smem_u32(smem + L::oK + (HA == 128 ? c * 2 : 0) * SLAB), SLAB);
            const uint32_t kdS = desc_lo_kmajor(smem_u32(smem + L::odS)), mdS = desc_lo_mnmajor(smem_u32(smem + L::odS), SLAB);
            auto issue_S = [&](int s) {
                const uint32_t kQ = desc_lo_kmajor(smem_u32(smem + L::oQ + s * L::kQTile));
#pragma unroll
                for (int kk = 0; kk < HD / 16; ++kk)
                    mma_ss_lo(T_RS, kK + (kk / 4) * kSlab + (kk % 4) * 2, kQ + (kk / 4) * kSlab64 + (kk % 4) * 2, idesc_s, kk > 0);
                mma_commit(&bars[B_S]);
            };
            auto issue_dP = [&](int s) {
                const uint32_t kdO = desc_lo_kmajor(smem_u32(smem + L::odO + s * L::kQTile));
#pragma unroll
                for (int kk = 0; kk < HD / 16; ++kk) {
                    const uint32_t boff = (kk / 4) * kSlab64 + (kk % 4) * 2;
                    if (L::kVinTmem) mma_ts_lo(T_RD, T_V + kk * 8, kdO + boff, idesc_s, kk > 0);
                    else mma_ss_lo(T_RD, kV + (kk / 4) * kSlab + (kk % 4) * 2, kdO + boff, idesc_s, kk > 0);
                }
                mma_commit(&bars[B_DP]);
            };
            mbar_wait(&bars[B_KV], 0, ab);
            if (L::kVinTmem) mbar_wait(&bars[B_VDONE], 0, ab);
            mbar_wait(&bars[B_QFULL], 0, ab);
            tcgen05_fence_after();
            issue_S(0);
            issue_dP(0);
            for (int t = 0; t < T; ++t) {
                const int s = t % NS;
                const uint32_t qbase = smem_u32(smem + L::oQ + s * L::kQTile + (HA == 128 ? c * 2 : 0) * SLAB64);
                const uint32_t obase = smem_u32(smem + L::odO + s * L::kQTile + (HA == 128 ? c * 2 : 0) * SLAB64);
                const uint32_t mQ_ = desc_lo_mnmajor(qbase, SLAB64), mdO_ = desc_lo_mnmajor(obase, SLAB64);
                // dV[:, c] += P^T dO[:, c]; P^T sits in the first 16 columns of each 32-column half of RS
                mbar_wait(&bars[B_P], t & 1, ab);
                tcgen05_fence_after();
#pragma unroll
                for (int kk = 0; kk < 4; ++kk)
                    mma_ts_lo(T_dV, T_RS + (kk / 2) * 32 + (kk % 2) * 8, mdO_ + kk * 128, idesc_acc, (t > 0) || (kk > 0));
                // S^T of the next tile over P^T: the products execute in issue order, dV has consumed it by then
                if (t + 1 < T) {
                    mbar_wait(&bars[B_QFULL + (t + 1) % NS], ((t + 1) / NS) & 1, ab);
                    tcgen05_fence_after();
                    issue_S((t + 1) % NS);
                }
                // dK[:, c] += dS^T Q[:, c], then dQ^T[c] = K_j[:, c]^T dS^T into RD (dP^T has been copied out of it)
                mbar_wait(&bars[B_DS], t & 1, ab);
                tcgen05_fence_after();
#pragma unroll
                for (int kk = 0; kk < 4; ++kk)
                    mma_ss_lo(T_dK, kdS + kk * 2, mQ_ + kk * 128, idesc_acc, (t > 0) || (kk > 0));
                mma_commit(&bars[B_QEMPTY + s]);     // stage s: dO was last read by dV, Q by dK
#pragma unroll
                for (int kk = 0; kk < TK / 16; ++kk)
                    mma_ss_lo(T_RD, mK + kk * 128, mdS + kk * 128, idesc_dq, kk > 0);
                mma_commit(&bars[B_DQ]);
                // dP^T of the next tile into RD once the reducers hold dQ^T in registers
                if (t + 1 < T) {
                    mbar_wait(&bars[B_DQDONE], t & 1, ab);
                    tcgen05_fence_after();
                    issue_dP((t + 1) % NS);
                }
            }
            mma_commit(&bars[B_DONE]);
        }
    } else if (warp >= 8) {
        // ------------------------------------------------------------ reducers: dQ^T[c] tile -> fp32 accumulator
        // lanes = head-dimension index, columns = queries: one warp instruction adds 128 contiguous bytes
        const int row = (warp % 4) * 32 + lane;
        const uint32_t lane_addr = (uint32_t)((warp % 4) * 32) << 16;
        const bool live = (warp % 4) * 32 < HA;
        int t = 0;
        for (int idx = 0; idx < iter.raw; ++idx) {
            const int it = iter.tile(idx);
            if (it < 0) continue;
            const int i0 = it * TQ64;
            float *base = a.dQ_acc + ((size_t)bh * n + i0) * HD + c * HA + row;
            mbar_wait(&bars[B_DQ], t & 1, ab);
            tcgen05_fence_after();
            uint32_t v[64];
            if (live) {
                tmem_ld32(T_RD + lane_addr, *reinterpret_cast<uint32_t(*)[32]>(&v[0]));
                tmem_ld32(T_RD + lane_addr + 32, *reinterpret_cast<uint32_t(*)[32]>(&v[32]));
                tmem_wait_ld();
            }
            tcgen05_fence_before();
            warp_arrive(&bars[B_DQDONE], lane);     // RD may take the next dP^T
            if (live) {
                if (i0 + TQ64 <= n) {
#pragma unroll
                    for (int e = 0; e < 64; ++e) red_add_f32(base + (size_t)e * HD, __uint_as_float(v[e]));
                } else {
#pragma unroll
                    for (int e = 0; e < 64; ++e)
                        if (i0 + e < n) red_add_f32(base + (size_t)e * HD, __uint_as_float(v[e]));
                }
            }
            ++t;
        }
    } else {
        // ------------------------------------------------------------ warps 0-7: exp / dS; g = 32-query half of the tile
        const int g = warp / 4;
        const int row = (warp % 4) * 32 + lane;        // tensor-memory lane = key row inside the tile
        const uint32_t lane_addr = (uint32_t)((warp % 4) * 32) << 16;
        const int jg = j0 + row;
        const float sl2 = a.scale * 1.4426950408889634f;
        const uint32_t c0 = g * 32;                    // this thread's columns of S^T / dP^T; its P^T pairs go to c0 .. c0 + 15
        if (L::kVinTmem && T > 0) {
            // V_j -> tensor memory, once: row `row`, bf16 pairs of head-dimension columns 128 g .. 128 g + 127
            mbar_wait(&bars[B_KV], 0, ab);
#pragma unroll
            for (int part = 0; part < 2; ++part) {
                const uint8_t *slab = smem + L::oQ + (g * 2 + part) * SLAB;
                uint32_t w[32];
#pragma unroll
                for (int ch = 0; ch < 8; ++ch) {
                    const uint4 x = *reinterpret_cast<const uint4 *>(slab + sw128_offset(row, ch * 8));
                    w[ch * 4 + 0] = x.x; w[ch * 4 + 1] = x.y; w[ch * 4 + 2] = x.z; w[ch * 4 + 3] = x.w;
                }
                tmem_st32(T_V + lane_addr + g * 64 + part * 32, w);
            }
            tmem_wait_st();
            tcgen05_fence_before();
            warp_arrive(&bars[B_VDONE], lane);
        }
        int t = 0;
        for (int idx = 0; idx < iter.raw; ++idx) {
            const int it = iter.tile(idx);
            if (it < 0) continue;
            const int s = t % NS, i0 = it * TQ64;
            const float4 *sNL = reinterpret_cast<const float4 *>(smem + L::oLSE + s * 256 + g * 128);
            const float4 *sDs = reinterpret_cast<const float4 *>(smem + L::oD + s * 256 + g * 128);
            const bool diag = mask_is_causal(a.mask_kind) && i0 < j0 + TK;   // some (i, j) of the tile pair has j > i
            const int ig0 = i0 + g * 32;
            // a mask finer than the tile: the keep bits of this thread's key row and its 32 query columns
            uint32_t kw = 0xffffffffu;
            if (a.fine.mode) kw = (ig0 < n && jg < n) ? fine_word(a.fine, a.mask_heads, bh, false, jg, ig0) : 0u;
            const bool masked = diag || i0 + TQ64 > n || j0 + TK > n || a.fine.mode != 0;
            mbar_wait(&bars[B_QFULL + s], (t / NS) & 1, ab);
            float4 nlr[8];
#pragma unroll
            for (int q = 0; q < 8; ++q) nlr[q] = sNL[q];
            mbar_wait(&bars[B_S], t & 1, ab);
            tcgen05_fence_after();
            uint32_t ppack[16];   // P as bf16 pairs: what dV uses, and what dS is formed from
            {
                uint32_t sv[32];
                tmem_ld32(T_RS + lane_addr + c0, sv);
                tmem_wait_ld();
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
            float4 dsr[8];
#pragma unroll
            for (int q = 0; q < 8; ++q) dsr[q] = sDs[q];
            // P^T over this thread's own S^T columns (it holds them in registers; no other thread reads them)
            tmem_st16(T_RS + lane_addr + c0, ppack);
            mbar_wait(&bars[B_DP], t & 1, ab);
            tcgen05_fence_after();
            uint32_t dv[32];
            tmem_ld32(T_RD + lane_addr + c0, dv);
            tmem_wait_ld();
            tmem_wait_st();
            tcgen05_fence_before();
            warp_arrive(&bars[B_P], lane);
            // dS^T(t) goes over dS^T(t-1): the dK and dQ^T products of tile t-1 must be done with it
            if (t > 0) mbar_wait(&bars[B_DQ], (t - 1) & 1, ab);
            {
                uint8_t *slab = smem + L::odS;
#pragma unroll
                for (int gg = 0; gg < 4; ++gg) {    // 8 query columns = one 16-byte chunk
                    float ds[8], p[8];
#pragma unroll
                    for (int e = 0; e < 4; ++e) {
                        const uint32_t pk = ppack[gg * 4 + e];   // bf16 -> fp32 is a 16-bit shift
                        p[2 * e] = __uint_as_float(pk << 16);
                        p[2 * e + 1] = __uint_as_float(pk & 0xffff0000u);
                    }
#pragma unroll
                    for (int u = 0; u < 2; ++u) {
                        const float4 dsc = dsr[gg * 2 + u];
                        const uint32_t *d4 = &dv[gg * 8 + u * 4];
                        ds[u * 4 + 0] = p[u * 4 + 0] * fmaf(__uint_as_float(d4[0]), a.scale, -dsc.x);
                        ds[u * 4 + 1] = p[u * 4 + 1] * fmaf(__uint_as_float(d4[1]), a.scale, -dsc.y);
                        ds[u * 4 + 2] = p[u * 4 + 2] * fmaf(__uint_as_float(d4[2]), a.scale, -dsc.z);
                        ds[u * 4 + 3] = p[u * 4 + 3] * fmaf(__uint_as_float(d4[3]), a.scale, -dsc.w);
                    }
                    if (masked) {   // stale tail entries of the row vectors may be anything: select, do not multiply
#pragma unroll
                        for (int e = 0; e < 8; ++e) ds[e] = p[e] != 0.f ? ds[e] : 0.f;
                    }
                    *reinterpret_cast<uint4 *>(slab + sw128_offset(row, g * 32 + gg * 8)) =
                        make_uint4(pack_bf16(ds[0], ds[1]), pack_bf16(ds[2], ds[3]), pack_bf16(ds[4], ds[5]),
                                   pack_bf16(ds[6], ds[7]));
                }
            }
            fence_proxy_async_smem();
            tcgen05_fence_before();
            warp_arrive(&bars[B_DS], lane);
            ++t;
        }
        // ------------------------------------------------------------ epilogue: dV_j[:, c], dK_j[:, c]
        if (T > 0) {
            mbar_wait(&bars[B_DONE], 0, ab);
            tcgen05_fence_after();
        }
        if (g * 64 < HA) {
            const int jc = jg < n ? jg : 0;
#pragma unroll
            for (int which = 0; which < 2; ++which) {
                __nv_bfloat16 *po = (which == 0 ? a.dV : a.dK) + ((size_t)bh * n + jc) * HD + c * HA + g * 64;
#pragma unroll
                for (int half = 0; half < 2; ++half) {
                    if (g * 64 + half * 32 >= HA) continue;
                    uint32_t v[32];
                    if (T > 0) {
                        tmem_ld32((which == 0 ? T_dV : T_dK) + lane_addr + g * 64 + half * 32, v);
                        tmem_wait_ld();
                    } else {
#pragma unroll
                        for (int e = 0; e < 32; ++e) v[e] = 0u;
                    }
                    if (jg < n) {
#pragma unroll
                        for (int e = 0; e < 32; e += 8)
                            *reinterpret_cast<uint4 *>(po + half * 32 + e) =
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

template <int HD>
attn_status launch_bwd64(const Problem &p)
{
    using L = B64<HD>;
    CUtensorMap mQ, mK, mV, mdO;
    const uint64_t BH = (uint64_t)p.BH;
    if (!make_tmap_bf16_3d(&mQ, p.Q, HD, p.n, BH, 64) || !make_tmap_bf16_3d(&mK, p.K, HD, p.n, BH, 128) ||
        !make_tmap_bf16_3d(&mV, p.V, HD, p.n, BH, 128) || !make_tmap_bf16_3d(&mdO, p.dO, HD, p.n, BH, 64))
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
    if (bwd_preprocess_launch(p, true) != ATTN_OK) return ATTN_ERR_LAUNCH;
    if (cudaFuncSetAttribute(tc_bwd_fused64_kernel<HD>, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)L::kBytes) != cudaSuccess)
        return ATTN_ERR_LAUNCH;
    const dim3 grid((unsigned)((p.n + TK - 1) / TK * a.group), (unsigned)(p.BH / a.group), (unsigned)L::kSplit);
    launch_begin("tc_bwd_fused64", p.stream);
    tc_bwd_fused64_kernel<HD><<<grid, kThreads64, L::kBytes, p.stream>>>(mQ, mK, mV, mdO, a);
    launch_end(p.stream);
    if (cudaGetLastError() != cudaSuccess) return ATTN_ERR_LAUNCH;
    return bwd_dq_convert_launch(p);
}

}  // namespace

size_t bwd64_smem_bytes(int d) { return d == 128 ? B64<128>::kUsed : d == 256 ? B64<256>::kUsed : 0; }

attn_status tc_bwd64(const Problem &p)
{
    if (p.d == 128) return launch_bwd64<128>(p);
    if (p.d == 256) return launch_bwd64<256>(p);
    return ATTN_ERR_TILE;
}

}  // namespace attn

// Fused forward for bf16 on the 5th-generation tensor cores: O = softmax(scale Q K^T) V
// and LSE, never writing a score tile to device memory (Definition 3.1; large-cache
// tiling: a row block of 128 queries stays on chip, key/value blocks stream through).
//
// A CTA owns one tile of 128 queries (tensor-memory lane = query row) and walks the kept
// key tiles j:
//
//   S   = Q_i K_j^T                  tcgen05.mma, operands K-major in shared memory
//   m, l running row maximum / row sum in the exp2 domain; the reference maximum is
//       only moved (and O rescaled in tensor memory) when the tile maximum exceeds it
//       by more than 2^8 -- the final LSE does not depend on which reference was used
//   P   = exp2(S * scale*log2e - m)  -> bf16, written over S in tensor memory
//   O  += P V_j                      A = P from tensor memory, B = V_j MN-major
//
// Two kernels.  tc_fwd_rows_kernel (d = 64, 128; key tiles of 128): the two softmax
// warpgroups take alternate key tiles, each with an S buffer and a partial accumulator of
// its own, a thread holds a whole row of scores, and the two partial softmaxes are merged
// in the epilogue.  tc_fwd_kernel (d = 256; key tiles of 64): both warpgroups split the
// columns of every tile and exchange row maxima through shared memory, one accumulator of
// 256 columns.  Each has one MMA-issuing thread and one TMA-producing thread; the roles and
// the tensor-memory layout are described at each kernel.
#include "attn_internal.h"
#include "tc_common.cuh"

namespace attn {
namespace {

using namespace tc;

constexpr int TQ = 128;
constexpr int kSoftmaxThreads = 256;
constexpr int kThreads = kSoftmaxThreads + 64;
constexpr float kLog2e = 1.4426950408889634f;
constexpr float kLn2 = 0.6931471805599453f;
constexpr float kRescaleThreshold = 8.f;   // log2 units

struct FwdArgs {
    __nv_bfloat16 *O;
    float *LSE;
    int n, BH;
    int mask_kind, block, nb, mask_heads;
    const int *row_ptr, *col_idx;   // block-CSR of the mask
    FineMask fine;                  // a mask finer than the tiles (32- / 64-wide blocks, element bitmap)
    float scale;
    uint32_t *status;
};

template <int HD>
struct FwdCfg {
    static constexpr int TKF = HD == 256 ? 64 : 128;
    static constexpr int NST = HD == 256 ? 2 : 3;
    static constexpr uint32_t kQSlab = 128 * 128;              // [128 queries][64 bf16]
    static constexpr uint32_t kKSlab = TKF * 128;              // [TKF keys][64 bf16]
    static constexpr uint32_t kSlabs = HD / 64;
    static constexpr uint32_t kQTile = kSlabs * kQSlab;
    static constexpr uint32_t kKTile = kSlabs * kKSlab;
    static constexpr uint32_t oQ = 0;
    static constexpr uint32_t oK = oQ + kQTile;                // NST stages
    static constexpr uint32_t oV = oK + NST * kKTile;          // NST stages
    static constexpr uint32_t oX = oV + NST * kKTile;          // row-max exchange [2 buffers][2 wg][128]; row sums reuse buffer 0
    static constexpr uint32_t oBar = oX + 4 * 128 * 4;
    static constexpr uint32_t oMisc = oBar + 24 * 8;
    static constexpr uint32_t kUsed = oMisc + 64;
    static_assert(kUsed <= 227 * 1024, "shared memory budget");
    // at least 117 KB so that only one CTA (which allocates all 512 tensor-memory columns) fits per SM
    static constexpr uint32_t kBytes = kUsed < 117 * 1024 ? 117 * 1024 : kUsed;
};

enum { FB_Q = 0, FB_KVFULL = 1, FB_KVEMPTY = 4, FB_S = 7, FB_P = 9, FB_O = 11, FB_OLAST = 12 };

template <int TKF>
struct KeyIter {
    // Enumerates the key tiles (of TKF keys) a query tile `it` (128 queries) has to visit.
    int kind, n, sub, raw, last_i;
    const int *cols;
    __device__ KeyIter(const FwdArgs &a, int it, long bh) : kind(a.mask_kind), n(a.n), sub(1), raw(0), cols(nullptr)
    {
        last_i = min(it * TQ + TQ, n) - 1;
        const int ntk = (n + TKF - 1) / TKF;
        if (kind == ATTN_MASK_NONE) raw = ntk;
        else if (kind == ATTN_MASK_CAUSAL) {
            const int last_i = min(it * TQ + TQ, n) - 1;
            raw = last_i / TKF + 1;
        } else {
            sub = a.block / TKF;
            const int I = it * TQ / a.block;
            const long mh = a.mask_heads == 1 ? 0 : bh;
            const int *rp = a.row_ptr + mh * 2 * a.nb + 2 * I;
            cols = a.col_idx + mh * (long)a.nb * a.nb + rp[0];
            raw = (rp[1] - rp[0]) * sub;
        }
    }
    __device__ int tile(int idx) const
    {
        int jt;
        if (mask_is_block(kind)) jt = cols[idx / sub] * sub + idx % sub;
        else jt = idx;
        // block mask AND causal: a key tile that begins after the last query of the tile keeps nothing
        if (kind == ATTN_MASK_BLOCK_SPARSE_CAUSAL && jt * TKF > last_i) return -1;
        return jt * TKF < n ? jt : -1;
    }
};

__device__ __forceinline__ float ex2_fast_f(float x)
{
    float y;
    asm("ex2.approx.ftz.f32 %0, %1;" : "=f"(y) : "f"(x));
    return y;
}
__device__ __forceinline__ void named_bar_sync_f(int id, int count)
{
    asm volatile("bar.sync %0, %1;" ::"r"(id), "r"(count) : "memory");
}

template <int HD>
__global__ void __launch_bounds__(kThreads, 1)
tc_fwd_kernel(const __grid_constant__ CUtensorMap mQ, const __grid_constant__ CUtensorMap mK,
              const __grid_constant__ CUtensorMap mV, const FwdArgs a)
{
    using C = FwdCfg<HD>;
    constexpr int TKF = C::TKF, NST = C::NST;
    constexpr int CW = TKF / 2;      // key columns per warpgroup
    extern __shared__ __align__(1024) uint8_t smem[];
    uint64_t *bars = reinterpret_cast<uint64_t *>(smem + C::oBar);
    uint32_t *tmem_base_s = reinterpret_cast<uint32_t *>(smem + C::oMisc);
    volatile uint32_t *abort_flag = reinterpret_cast<volatile uint32_t *>(smem + C::oMisc + 4);
    float *xmax = reinterpret_cast<float *>(smem + C::oX);            // [2][2][128]
    float *xsum = xmax;                                               // [2][128], reuses exchange buffer 0 in the epilogue
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
        mbar_init(&bars[FB_Q], 1);
        for (int s = 0; s < NST; ++s) { mbar_init(&bars[FB_KVFULL + s], 1); mbar_init(&bars[FB_KVEMPTY + s], 1); }
        for (int b = 0; b < 2; ++b) { mbar_init(&bars[FB_S + b], 1); mbar_init(&bars[FB_P + b], kSoftmaxThreads); }
        mbar_init(&bars[FB_O], 1);
        mbar_init(&bars[FB_OLAST], 1);
        fence_barrier_init();
        prefetch_tensormap(&mQ); prefetch_tensormap(&mK); prefetch_tensormap(&mV);
    }
    if (warp == 0) tmem_alloc(tmem_base_s, 512);
    tcgen05_fence_before();
    __syncthreads();
    tcgen05_fence_after();
    const uint32_t tm = *tmem_base_s;
    const uint32_t T_O = tm + 256;
    const KeyIter<TKF> iter(a, it, bh);

    // number of valid key tiles (same in every role)
    int niter = 0;
    for (int idx = 0; idx < iter.raw; ++idx) niter += iter.tile(idx) >= 0;

    if (warp == 9) {
        // ------------------------------------------------------------ TMA producer
        if (lane == 0) {
            mbar_expect_tx(&bars[FB_Q], C::kQTile);
#pragma unroll
            for (uint32_t sl = 0; sl < C::kSlabs; ++sl)
                tma_load_3d(smem + C::oQ + sl * C::kQSlab, &mQ, &bars[FB_Q], sl * 64, i0, (int)bh);
            int k = 0;
            for (int idx = 0; idx < iter.raw; ++idx) {
                const int jt = iter.tile(idx);
                if (jt < 0) continue;
                const int s = k % NST;
                if (k >= NST) mbar_wait(&bars[FB_KVEMPTY + s], ((k / NST) - 1) & 1, ab);
                uint64_t *bar = &bars[FB_KVFULL + s];
                mbar_expect_tx(bar, 2 * C::kKTile);
#pragma unroll
                for (uint32_t sl = 0; sl < C::kSlabs; ++sl) {
                    tma_load_3d(smem + C::oK + s * C::kKTile + sl * C::kKSlab, &mK, bar, sl * 64, jt * TKF, (int)bh);
                    tma_load_3d(smem + C::oV + s * C::kKTile + sl * C::kKSlab, &mV, bar, sl * 64, jt * TKF, (int)bh);
                }
                ++k;
            }
        }
    } else if (warp == 8) {
        // ------------------------------------------------------------ MMA issuer
        if (lane == 0 && niter == 0) mbar_wait(&bars[FB_Q], 0, ab);   // let the Q load land before exit
        if (lane == 0 && niter > 0) {
            constexpr uint32_t idesc_s = idesc_bf16(128, TKF, 0, 0);
            constexpr uint32_t idesc_o = idesc_bf16(128, HD, 0, 1);
            const uint32_t kQ = desc_lo_kmajor(smem_u32(smem + C::oQ));
            auto issue_S = [&](int k) {
                const int s = k % NST;
                mbar_wait(&bars[FB_KVFULL + s], (k / NST) & 1, ab);
                tcgen05_fence_after();
                const uint32_t kK = desc_lo_kmajor(smem_u32(smem + C::oK + s * C::kKTile));
#pragma unroll
                for (int kk = 0; kk < HD / 16; ++kk)
                    mma_ss_lo(tm + (k & 1) * 128, kQ + (kk / 4) * (C::kQSlab >> 4) + (kk % 4) * 2,
                              kK + (kk / 4) * (C::kKSlab >> 4) + (kk % 4) * 2, idesc_s, kk > 0);
                mma_commit(&bars[FB_S + (k & 1)]);
            };
            mbar_wait(&bars[FB_Q], 0, ab);
            issue_S(0);
            for (int k = 0; k < niter; ++k) {
                if (k + 1 < niter) issue_S(k + 1);
                const int s = k % NST, b = k & 1;
                mbar_wait(&bars[FB_P + b], (k >> 1) & 1, ab);
                tcgen05_fence_after();
                const uint32_t mV_ = desc_lo_mnmajor(smem_u32(smem + C::oV + s * C::kKTile), C::kKSlab);
#pragma unroll
                for (int kk = 0; kk < TKF / 16; ++kk)
                    mma_ts_lo(T_O, tm + b * 128 + kk * 8, mV_ + kk * 128, idesc_o, (k > 0) || (kk > 0));
                mma_commit(&bars[FB_KVEMPTY + s]);
                mma_commit(&bars[FB_O]);
                if (k + 1 == niter) mma_commit(&bars[FB_OLAST]);
            }
        }
    } else {
        // ------------------------------------------------------------ softmax warpgroups
        const int wg = warp / 4;
        const int row = (warp % 4) * 32 + lane;
        const uint32_t lane_addr = (uint32_t)((warp % 4) * 32) << 16;
        const int ig = i0 + row;
        const float sl2 = a.scale * kLog2e;
        float m_ref = -INFINITY, l_part = 0.f;
        int k = 0;
        for (int idx = 0; idx < iter.raw; ++idx) {
            const int jt = iter.tile(idx);
            if (jt < 0) continue;
            const int b = k & 1, j0 = jt * TKF;
            // a mask finer than the tile: the keep bits of this thread's query row and its 32 key columns, fetched
            // before the wait for S
            uint32_t kw = 0xffffffffu;
            if (a.fine.mode) kw = (ig < n && j0 + wg * CW < n) ? fine_word(a.fine, a.mask_heads, bh, true, ig, j0 + wg * CW) : 0u;
            mbar_wait(&bars[FB_S + b], (k >> 1) & 1, ab);
            tcgen05_fence_after();
            const uint32_t T_S = tm + b * 128;
            float sv[CW];
#pragma unroll
            for (int c = 0; c < CW; c += 32) {
                uint32_t v[32];
                tmem_ld32(T_S + lane_addr + wg * CW + c, v);
                tmem_wait_ld();
#pragma unroll
                for (int e = 0; e < 32; ++e) sv[c + e] = __uint_as_float(v[e]);   // raw scores; scale * log2e enters below
            }
            const bool need_mask = (mask_is_causal(a.mask_kind) && j0 + TKF - 1 > i0) || j0 + TKF > n || a.fine.mode != 0;
            float mx = -INFINITY;
            if (need_mask) {
                const bool causal = mask_is_causal(a.mask_kind);
#pragma unroll
                static_assert(CW == 32, "one keep word per thread and tile");
#pragma unroll
                for (int e = 0; e < CW; ++e) {
                    const int jg = j0 + wg * CW + e;
                    if (jg >= n || (causal && jg > ig) || !((kw >> e) & 1u)) sv[e] = -INFINITY;
                }
            }
#pragma unroll
            for (int e = 0; e < CW; ++e) mx = fmaxf(mx, sv[e]);
            float *xm = xmax + b * 256;
            xm[wg * 128 + row] = mx;
            named_bar_sync_f(1, kSoftmaxThreads);   // also: every S read of this tile is done
            const float m_tile = fmaxf(xm[row], xm[128 + row]) * sl2;   // scale > 0: the maximum commutes with it
            const bool need = m_tile > m_ref + kRescaleThreshold || (m_ref == -INFINITY && m_tile != -INFINITY);
            if (__any_sync(0xffffffffu, need)) {
                const float m_new = need ? fmaxf(m_ref, m_tile) : m_ref;
                const float alpha = (need && m_ref != -INFINITY) ? ex2_fast_f(m_ref - m_new) : 1.f;
                if (k > 0) {
                    mbar_wait(&bars[FB_O], (k - 1) & 1, ab);   // O += P V of the previous tile has landed
                    tcgen05_fence_after();
#pragma unroll
                    for (int c = 0; c < HD / 2; c += 32) {
                        uint32_t v[32];
                        tmem_ld32(T_O + lane_addr + wg * (HD / 2) + c, v);
                        tmem_wait_ld();
#pragma unroll
                        for (int e = 0; e < 32; ++e) v[e] = __float_as_uint(__uint_as_float(v[e]) * alpha);
                        tmem_st32(T_O + lane_addr + wg * (HD / 2) + c, v);
                    }
                }
                l_part *= alpha;
                m_ref = m_new;
            }
            const float noff = m_ref == -INFINITY ? 0.f : -m_ref;
            uint32_t pp[CW / 2];
            float rs = 0.f;
#pragma unroll
            for (int e = 0; e < CW; e += 2) {
                const float p0 = ex2_fast_f(fmaf(sv[e], sl2, noff)), p1 = ex2_fast_f(fmaf(sv[e + 1], sl2, noff));
                rs += p0 + p1;
                pp[e / 2] = pack_bf16(p0, p1);
            }
            l_part += rs;
            if (CW == 64) {
                uint32_t(&pp32)[32] = *reinterpret_cast<uint32_t(*)[32]>(pp);
                tmem_st32(T_S + lane_addr + wg * (CW / 2), pp32);
            } else {
                uint32_t(&pp16)[16] = *reinterpret_cast<uint32_t(*)[16]>(pp);
                tmem_st16(T_S + lane_addr + wg * (CW / 2), pp16);
            }
            tmem_wait_st();
            tcgen05_fence_before();
            mbar_arrive(&bars[FB_P + b]);
            ++k;
        }
        // ------------------------------------------------------------ epilogue
        named_bar_sync_f(1, kSoftmaxThreads);   // everyone is done with the row-max exchange buffers
        xsum[wg * 128 + row] = l_part;
        named_bar_sync_f(1, kSoftmaxThreads);
        const float l_tot = xsum[row] + xsum[128 + row];
        if (k > 0) {
            // FB_O completes once per tile and a parity wait tells two phases apart, not three: the last completion
            // this thread knows of is S(k-1), queued before O += P V of tile k-2, so FB_O may be two completions
            // behind the one needed here and a wait on it could pass at once.  The last product has a barrier of its own.
            mbar_wait(&bars[FB_OLAST], 0, ab);
            tcgen05_fence_after();
        }
        const float inv = l_tot > 0.f ? 1.f / l_tot : 0.f;
        const int ic = ig < n ? ig : 0;
        __nv_bfloat16 *po = a.O + ((size_t)bh * n + ic) * HD + wg * (HD / 2);
#pragma unroll
        for (int c = 0; c < HD / 2; c += 32) {
            uint32_t v[32];
            if (k > 0) {
                tmem_ld32(T_O + lane_addr + wg * (HD / 2) + c, v);
                tmem_wait_ld();
            } else {
#pragma unroll
                for (int e = 0; e < 32; ++e) v[e] = 0u;
            }
            if (ig < n) {
#pragma unroll
                for (int e = 0; e < 32; e += 8) {
                    uint4 o;
                    o.x = pack_bf16(__uint_as_float(v[e]) * inv, __uint_as_float(v[e + 1]) * inv);
                    o.y = pack_bf16(__uint_as_float(v[e + 2]) * inv, __uint_as_float(v[e + 3]) * inv);
                    o.z = pack_bf16(__uint_as_float(v[e + 4]) * inv, __uint_as_float(v[e + 5]) * inv);
                    o.w = pack_bf16(__uint_as_float(v[e + 6]) * inv, __uint_as_float(v[e + 7]) * inv);
                    *reinterpret_cast<uint4 *>(po + c + e) = o;
                }
            }
        }
        if (wg == 0 && ig < n) a.LSE[(size_t)bh * n + ig] = l_tot > 0.f ? m_ref * kLn2 + logf(l_tot) : -INFINITY;
    }
    tcgen05_fence_before();
    __syncthreads();
    if (warp == 0) tmem_dealloc(tm, 512);
}

// ---------------------------------------------------------------------------------------
// d = 64 and 128: the two softmax warpgroups take ALTERNATE key tiles.  Warpgroup w owns the S buffer w and
// an accumulator O_w of its own (tensor memory: S_0 128, S_1 128, O_0 d, O_1 d columns), and a thread owns a
// whole row of its tile: the row maximum needs no exchange, and while one warpgroup is loading, taking the
// maximum or storing P, the other one keeps the MUFU pipe busy with its exponentials.  Each warpgroup runs its
// own online softmax (m_w, l_w, O_w) over its tiles; the two partial results are merged once at the end:
// O = (2^(m_0 - m) O_0 + 2^(m_1 - m) O_1) / (2^(m_0 - m) l_0 + 2^(m_1 - m) l_1), m = max(m_0, m_1).
// Issue order of the single issuing thread: S(0), S(1), then per tile k: O_{k&1} += P(k) V(k), S(k+2).
enum { F2_Q = 0, F2_KFULL = 1, F2_KEMPTY = 4, F2_VFULL = 7, F2_VEMPTY = 10, F2_S = 13, F2_P = 15, F2_O = 17 };

// 384 threads: warps 0-7 softmax, warp 8 MMA issuer, warp 9 TMA producer, warps 10-11 only complete that warpgroup.
// Three warps per scheduler cap the launch at 168 registers; after launch the last warpgroup gives registers up and
// the softmax warpgroups take them (256 x 224 + 128 x 40 = 62,464 of the 384 x 168 = 64,512 the block holds), so
// that a thread can keep its whole row of 128 scores.
constexpr int kThreadsRows = kSoftmaxThreads + 128;
template <int HD, bool FINE>
__global__ void __launch_bounds__(kThreadsRows, 1)
tc_fwd_rows_kernel(const __grid_constant__ CUtensorMap mQ, const __grid_constant__ CUtensorMap mK,
                   const __grid_constant__ CUtensorMap mV, const FwdArgs a)
{
    using C = FwdCfg<HD>;
    static_assert(C::TKF == 128 && C::NST == 3 && 256 + 2 * HD <= 512, "layout of the row-per-thread forward");
    constexpr int TKF = 128, NST = 3;
    extern __shared__ __align__(1024) uint8_t smem[];
    uint64_t *bars = reinterpret_cast<uint64_t *>(smem + C::oBar);
    uint32_t *tmem_base_s = reinterpret_cast<uint32_t *>(smem + C::oMisc);
    volatile uint32_t *abort_flag = reinterpret_cast<volatile uint32_t *>(smem + C::oMisc + 4);
    float *xm = reinterpret_cast<float *>(smem + C::oX);   // [2 warpgroups][128 rows] reference maxima
    float *xl = xm + 256;                                  // [2][128] row sums
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
        mbar_init(&bars[F2_Q], 1);
        for (int s = 0; s < NST; ++s) {
            mbar_init(&bars[F2_KFULL + s], 1); mbar_init(&bars[F2_KEMPTY + s], 1);
            mbar_init(&bars[F2_VFULL + s], 1); mbar_init(&bars[F2_VEMPTY + s], 1);
        }
        for (int b = 0; b < 2; ++b) { mbar_init(&bars[F2_S + b], 1); mbar_init(&bars[F2_P + b], 4); mbar_init(&bars[F2_O + b], 1); }
        fence_barrier_init();
        prefetch_tensormap(&mQ); prefetch_tensormap(&mK); prefetch_tensormap(&mV);
    }
    if (warp == 0) tmem_alloc(tmem_base_s, 512);
    tcgen05_fence_before();
    __syncthreads();
    tcgen05_fence_after();
    const uint32_t tm = *tmem_base_s;
    const KeyIter<TKF> iter(a, it, bh);

    int niter = 0;   // number of valid key tiles (same in every role)
    for (int idx = 0; idx < iter.raw; ++idx) niter += iter.tile(idx) >= 0;

    if (warp >= 8) {
      asm volatile("setmaxnreg.dec.sync.aligned.u32 40;");
      if (warp == 9) {
        // ------------------------------------------------------------ TMA producer
        if (lane == 0) {
            mbar_expect_tx(&bars[F2_Q], C::kQTile);
#pragma unroll
            for (uint32_t sl = 0; sl < C::kSlabs; ++sl)
                tma_load_3d(smem + C::oQ + sl * C::kQSlab, &mQ, &bars[F2_Q], sl * 64, i0, (int)bh);
            int k = 0;
            for (int idx = 0; idx < iter.raw; ++idx) {
                const int jt = iter.tile(idx);
                if (jt < 0) continue;
                const int s = k % NST;
                // K and V of a tile have rings of their own: the K stage is free again as soon as S has been formed,
                // long before the V stage, so K runs further ahead
                if (k >= NST) mbar_wait(&bars[F2_KEMPTY + s], ((k / NST) - 1) & 1, ab);
                mbar_expect_tx(&bars[F2_KFULL + s], C::kKTile);
#pragma unroll
                for (uint32_t sl = 0; sl < C::kSlabs; ++sl)
                    tma_load_3d(smem + C::oK + s * C::kKTile + sl * C::kKSlab, &mK, &bars[F2_KFULL + s], sl * 64, jt * TKF, (int)bh);
                // The release of a V stage has no barrier of its own (a commit costs the issuing thread about a hundred
                // cycles per tile): the V stage of tile k - 3 is free when S(k-1) has completed, which the issuing thread
                // queues right after O += P V of tile k - 3 (products complete in issue order).  S(k-1) is the newest
                // completion its barrier can have here -- S(k+1) needs the K tile that this thread loads next -- so the
                // parity wait cannot be a phase behind
                if (k >= NST) mbar_wait(&bars[F2_S + ((k - 1) & 1)], ((k - 1) >> 1) & 1, ab);
                mbar_expect_tx(&bars[F2_VFULL + s], C::kKTile);
#pragma unroll
                for (uint32_t sl = 0; sl < C::kSlabs; ++sl)
                    tma_load_3d(smem + C::oV + s * C::kKTile + sl * C::kKSlab, &mV, &bars[F2_VFULL + s], sl * 64, jt * TKF, (int)bh);
                ++k;
            }
        }
      } else if (warp == 8) {
        // ------------------------------------------------------------ MMA issuer
        if (lane == 0 && niter == 0) mbar_wait(&bars[F2_Q], 0, ab);   // let the Q load land before exit
        if (lane == 0 && niter > 0) {
            constexpr uint32_t idesc_s = idesc_bf16(128, TKF, 0, 0);
            constexpr uint32_t idesc_o = idesc_bf16(128, HD, 0, 1);
            const uint32_t kQ = desc_lo_kmajor(smem_u32(smem + C::oQ));
            auto issue_S = [&](int k) {   // the caller has waited for K of tile k
                const uint32_t kK = desc_lo_kmajor(smem_u32(smem + C::oK + (k % NST) * C::kKTile));
#pragma unroll
                for (int kk = 0; kk < HD / 16; ++kk)
                    mma_ss_lo(tm + (k & 1) * 128, kQ + (kk / 4) * (C::kQSlab >> 4) + (kk % 4) * 2,
                              kK + (kk / 4) * (C::kKSlab >> 4) + (kk % 4) * 2, idesc_s, kk > 0);
                mma_commit(&bars[F2_S + (k & 1)]);
                mma_commit(&bars[F2_KEMPTY + k % NST]);
            };
            mbar_wait(&bars[F2_Q], 0, ab);
            mbar_wait(&bars[F2_KFULL], 0, ab);
            tcgen05_fence_after();
            issue_S(0);
            if (niter > 1) {
                mbar_wait(&bars[F2_KFULL + 1], 0, ab);
                tcgen05_fence_after();
                issue_S(1);
            }
            for (int k = 0; k < niter; ++k) {
                const int s = k % NST, b = k & 1;
                // everything that can be waited for ahead of P(k) is: the path P(k) -> O += P V -> S(k+2) -> next
                // softmax of that warpgroup is the one that decides the tile period
                mbar_wait(&bars[F2_VFULL + s], (k / NST) & 1, ab);
                if (k + 2 < niter) mbar_wait(&bars[F2_KFULL + (k + 2) % NST], ((k + 2) / NST) & 1, ab);
                mbar_wait(&bars[F2_P + b], (k >> 1) & 1, ab);
                tcgen05_fence_after();
                const uint32_t mV_ = desc_lo_mnmajor(smem_u32(smem + C::oV + s * C::kKTile), C::kKSlab);
#pragma unroll
                for (int kk = 0; kk < TKF / 16; ++kk)
                    mma_ts_lo(tm + 256 + b * HD, tm + b * 128 + kk * 8, mV_ + kk * 128, idesc_o, (k > 1) || (kk > 0));
                // the products execute in issue order: S(k+2) overwrites buffer b after P(k) has been consumed, and
                // its completion tells warpgroup b that O_b holds the product of tile k as well
                if (k + 2 < niter) issue_S(k + 2);
                else mma_commit(&bars[F2_O + b]);   // the last product of each warpgroup, for the epilogue
            }
        }
      }
    } else {
        // ------------------------------------------------------------ softmax warpgroup w: tiles k = w, w + 2, ...
        asm volatile("setmaxnreg.inc.sync.aligned.u32 224;");
        const int w = warp / 4;
        const int row = (warp % 4) * 32 + lane;
        const uint32_t lane_addr = (uint32_t)((warp % 4) * 32) << 16;
        const int ig = i0 + row;
        const float sl2 = a.scale * kLog2e;
        const uint32_t T_S = tm + w * 128, T_O = tm + 256 + w * HD;
        float m_ref = -INFINITY, l_run = 0.f;
        int k = 0, cnt = 0;
        for (int idx = 0; idx < iter.raw; ++idx) {
            const int jt = iter.tile(idx);
            if (jt < 0) continue;
            if ((k++ & 1) != w) continue;
            const int j0 = jt * TKF;
            const bool causal = mask_is_causal(a.mask_kind);
            const bool need_mask = (causal && j0 + TKF - 1 > i0) || j0 + TKF > n || FINE;
            mbar_wait(&bars[F2_S + w], cnt & 1, ab);
            tcgen05_fence_after();
            // the whole row of raw scores in registers: four loads in flight, one wait
            uint32_t v[TKF];
#pragma unroll
            for (int c = 0; c < TKF; c += 32) tmem_ld32(T_S + lane_addr + c, *reinterpret_cast<uint32_t(*)[32]>(&v[c]));
            tmem_wait_ld();
            if (need_mask) {
                const bool edge = (causal && j0 + TKF - 1 > i0) || j0 + TKF > n;   // entries dropped by position as well
#pragma unroll
                for (int q = 0; q < TKF / 32; ++q) {
                    // a mask finer than the tile: the keep bits of this thread's query row and 32 key columns.  A word that
                    // keeps all or nothing (the rule with 32- and 64-wide blocks) needs no test per entry
                    uint32_t kw = 0xffffffffu;
                    if constexpr (FINE) kw = (ig < n && j0 + q * 32 < n) ? fine_word(a.fine, a.mask_heads, bh, true, ig, j0 + q * 32) : 0u;
                    if (FINE && !edge && kw == 0xffffffffu) continue;
                    if (FINE && kw == 0u) {
#pragma unroll
                        for (int e = 0; e < 32; ++e) v[q * 32 + e] = 0xff800000u;   // -inf
                        continue;
                    }
#pragma unroll
                    for (int e = 0; e < 32; ++e) {
                        const int jg = j0 + q * 32 + e;
                        if (jg >= n || (causal && jg > ig) || !((kw >> e) & 1u)) v[q * 32 + e] = 0xff800000u;
                    }
                }
            }
            float mx8[8];   // eight independent chains instead of one of 128 dependent maxima
#pragma unroll
            for (int e = 0; e < 8; ++e) mx8[e] = __uint_as_float(v[e]);
#pragma unroll
            for (int e = 8; e < TKF; ++e) mx8[e & 7] = fmaxf(mx8[e & 7], __uint_as_float(v[e]));
            const float mx = fmaxf(fmaxf(fmaxf(mx8[0], mx8[1]), fmaxf(mx8[2], mx8[3])), fmaxf(fmaxf(mx8[4], mx8[5]), fmaxf(mx8[6], mx8[7])));
            const float m_tile = mx * sl2;   // scale > 0: the maximum commutes with it
            const bool need = m_tile > m_ref + kRescaleThreshold || (m_ref == -INFINITY && m_tile != -INFINITY);
            if (__any_sync(0xffffffffu, need)) {
                const float m_new = need ? fmaxf(m_ref, m_tile) : m_ref;
                const float alpha = (need && m_ref != -INFINITY) ? ex2_fast_f(m_ref - m_new) : 1.f;
                if (cnt > 0) {   // O_w += P V of this warpgroup's previous tile was issued before this tile's S: it has landed
#pragma unroll
                    for (int c = 0; c < HD; c += 16) {
                        uint32_t o[16];
                        tmem_ld16(T_O + lane_addr + c, o);
                        tmem_wait_ld();
#pragma unroll
                        for (int e = 0; e < 16; ++e) o[e] = __float_as_uint(__uint_as_float(o[e]) * alpha);
                        tmem_st16(T_O + lane_addr + c, o);
                    }
                }
                l_run *= alpha;
                m_ref = m_new;
            }
            const float noff = m_ref == -INFINITY ? 0.f : -m_ref;
            // P = exp2(S * scale * log2e - m_ref) as bf16 pairs over the first 64 columns of S (every thread
            // overwrites only its own lane, whose scores it already holds)
            float rs4[4] = {0.f, 0.f, 0.f, 0.f};
#pragma unroll
            for (int c = 0; c < TKF; c += 32) {
                uint32_t pp[16];
#pragma unroll
                for (int e = 0; e < 32; e += 2) {
                    const float p0 = ex2_fast_f(fmaf(__uint_as_float(v[c + e]), sl2, noff));
                    const float p1 = ex2_fast_f(fmaf(__uint_as_float(v[c + e + 1]), sl2, noff));
                    rs4[(e / 2) & 3] += p0 + p1;
                    pp[e / 2] = pack_bf16(p0, p1);
                }
                tmem_st16(T_S + lane_addr + c / 2, pp);
            }
            const float rs = (rs4[0] + rs4[1]) + (rs4[2] + rs4[3]);
            l_run += rs;
            tmem_wait_st();
            tcgen05_fence_before();
            __syncwarp();
            if (lane == 0) mbar_arrive(&bars[F2_P + w]);
            ++cnt;
        }
        // ------------------------------------------------------------ epilogue: merge the two partial softmaxes
        xm[w * 128 + row] = m_ref;
        xl[w * 128 + row] = l_run;
        named_bar_sync_f(1, kSoftmaxThreads);
        const float m0 = xm[row], m1 = xm[128 + row], l0 = xl[row], l1 = xl[128 + row];
        const float m_all = fmaxf(m0, m1);
        const float a0 = m0 == -INFINITY ? 0.f : ex2_fast_f(m0 - m_all), a1 = m1 == -INFINITY ? 0.f : ex2_fast_f(m1 - m_all);
        const float l_tot = a0 * l0 + a1 * l1;
        const float inv = l_tot > 0.f ? 1.f / l_tot : 0.f;
        const float c0 = a0 * inv, c1 = a1 * inv;
        const int cnt0 = (niter + 1) / 2, cnt1 = niter / 2;
        if (cnt0 > 0) mbar_wait(&bars[F2_O], 0, ab);
        if (cnt1 > 0) mbar_wait(&bars[F2_O + 1], 0, ab);
        tcgen05_fence_after();
        const int ic = ig < n ? ig : 0;
        __nv_bfloat16 *po = a.O + ((size_t)bh * n + ic) * HD + w * (HD / 2);
#pragma unroll
        for (int c = 0; c < HD / 2; c += 32) {
            uint32_t v0[32], v1[32];
            if (cnt0 > 0) tmem_ld32(tm + 256 + lane_addr + w * (HD / 2) + c, v0);
            if (cnt1 > 0) tmem_ld32(tm + 256 + HD + lane_addr + w * (HD / 2) + c, v1);
            tmem_wait_ld();
            float o[32];
#pragma unroll
            for (int e = 0; e < 32; ++e) {
                // a partial accumulator that never received a product holds stale bits: select, do not multiply
                const float x0 = cnt0 > 0 ? __uint_as_float(v0[e]) * c0 : 0.f;
                const float x1 = cnt1 > 0 ? __uint_as_float(v1[e]) * c1 : 0.f;
                o[e] = x0 + x1;
            }
            if (ig < n) {
#pragma unroll
                for (int e = 0; e < 32; e += 8)
                    *reinterpret_cast<uint4 *>(po + c + e) = make_uint4(pack_bf16(o[e], o[e + 1]), pack_bf16(o[e + 2], o[e + 3]),
                                                                        pack_bf16(o[e + 4], o[e + 5]), pack_bf16(o[e + 6], o[e + 7]));
            }
        }
        if (w == 0 && ig < n) a.LSE[(size_t)bh * n + ig] = l_tot > 0.f ? m_all * kLn2 + logf(l_tot) : -INFINITY;
    }
    tcgen05_fence_before();
    __syncthreads();
    if (warp == 0) tmem_dealloc(tm, 512);
}

template <int HD>
attn_status launch_fwd(const Problem &p)
{
    using C = FwdCfg<HD>;
    CUtensorMap mQ, mK, mV;
    const uint64_t BH = (uint64_t)p.BH;
    if (!make_tmap_bf16_3d(&mQ, p.Q, HD, p.n, BH, 128) || !make_tmap_bf16_3d(&mK, p.K, HD, p.n, BH, C::TKF) ||
        !make_tmap_bf16_3d(&mV, p.V, HD, p.n, BH, C::TKF))
        return ATTN_ERR_LAUNCH;
    FwdArgs a{};
    a.O = (__nv_bfloat16 *)p.Oout; a.LSE = p.LSEout;
    a.n = p.n; a.BH = (int)p.BH;
    a.mask_kind = p.mask_kind; a.block = p.block; a.nb = p.nb; a.mask_heads = p.mask_heads; a.fine = p.fine;
    a.row_ptr = p.row_ptr; a.col_idx = p.col_idx;
    a.scale = p.scale;
    a.status = p.status;
    void (*kernel)(CUtensorMap, CUtensorMap, CUtensorMap, FwdArgs);
    if constexpr (HD == 256) kernel = tc_fwd_kernel<HD>;
    else kernel = p.fine.mode ? tc_fwd_rows_kernel<HD, true> : tc_fwd_rows_kernel<HD, false>;
    if (cudaFuncSetAttribute(kernel, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)C::kBytes) != cudaSuccess)
        return ATTN_ERR_LAUNCH;
    const dim3 grid((p.n + TQ - 1) / TQ, (unsigned)p.BH);
    launch_begin("tc_fwd", p.stream);
    kernel<<<grid, HD == 256 ? kThreads : kThreadsRows, C::kBytes, p.stream>>>(mQ, mK, mV, a);
    launch_end(p.stream);
    return cudaGetLastError() == cudaSuccess ? ATTN_OK : ATTN_ERR_LAUNCH;
}

}  // namespace

size_t fwd_smem_bytes(int d)
{
    return d == 64 ? FwdCfg<64>::kUsed : d == 128 ? FwdCfg<128>::kUsed : d == 256 ? FwdCfg<256>::kUsed : 0;
}

attn_status tc_fwd(const Problem &p)
{
    if (p.d == 64) return launch_fwd<64>(p);
    if (p.d == 128) return launch_fwd<128>(p);
    if (p.d == 256) return launch_fwd<256>(p);
    return ATTN_ERR_TILE;
}

}  // namespace attn

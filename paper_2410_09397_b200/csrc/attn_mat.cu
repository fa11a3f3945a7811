// Materialised backward for bf16: the small-cache scheme of Appendix C.  The n x n
// matrices f (P), q (dP) and p (dS) are written to and re-read from device memory in
// blocks, and every product is a blocked GEMM whose contraction is walked in chunks of
// 64 -- this is the regime the paper bounds by O((n^2 d + n d^2) / sqrt(M)), used when a
// whole-d tile set does not fit on chip (d = 256).
//
//   phase 1  P  = exp(scale Q K^T - LSE)      blocked GEMM over d, exp in the epilogue,
//                                             P written (LSE comes from the forward, so
//                                             the paper's second sweep for l is not needed)
//   phase 2  dP = dO V^T                      blocked GEMM over d, written
//   phase 3  dS = scale P o (dP - D)          streaming pass: reads P, dP, writes dS
//   phase 4  dV = P^T dO, dK = dS^T Q, dQ = dS K     blocked GEMMs over n reading P / dS
//
// One persistent GEMM kernel serves all products.  A CTA walks a strided list of 128 x BN
// tiles of C (tile t = blockIdx.x + i gridDim.x; the column tile runs fastest, so the CTAs
// that run together share their A rows in L2).  Per tile: a TMA producer thread and an MMA
// issuing thread run a ring of 64-deep operand chunks into one of TWO fp32 accumulators in
// tensor memory; eight epilogue warps turn the other accumulator into bf16 (exp / plain),
// write it into a swizzled staging tile in shared memory and hand it to a TMA store, so
// that the epilogue of tile i and its store run under the products of tile i + 1.  Operands
// are taken K-major or MN-major straight from their row-major arrays (no transposes).
#include "attn_internal.h"
#include "tc_bwd_common.cuh"
#include "tc_common.cuh"

#include <type_traits>

namespace attn {
namespace {

using namespace tc;

enum { EPI_EXP = 0, EPI_PLAIN = 1, EPI_OUT = 2 };
constexpr int kEpiWarps = 8;
constexpr int kGemmThreads = kEpiWarps * 32 + 64;   // epilogue warps, TMA producer warp, MMA issuer warp

struct GemmArgs {
    int heads;               // of this launch
    int m_total, n_total;    // valid rows / cols of C per head
    int k_total;             // contraction length
    const float *nlse2;      // EPI_EXP: -LSE log2e per row [heads][m_total]
    float sl2;               // EPI_EXP: scale * log2e
    int causal;              // EPI_EXP: entries with col > row are zero; tiles wholly above the diagonal skip the product
    uint32_t *status;
};

// BN: columns of a tile; MT: 128-row sub-tiles of a tile (1 or 2).  MT = 2 forms a 256 x BN tile in two accumulators
// that share every B chunk (less operand traffic than two separate 128-row tiles).  Tensor memory holds two sets of
// MT accumulators that alternate between tiles where 2 MT BN <= 512 columns, else one set.
template <int BN, int MT>
struct GemmSmem {
    static constexpr int OUTW = BN < 128 ? BN : 128;     // columns of one staging step
    static constexpr int kOutBufs = MT * BN >= 512 ? 1 : 2;
    static constexpr int NBUF = 2 * MT * BN <= 512 ? 2 : 1;   // accumulator sets
    static constexpr uint32_t kA = MT * 128 * 128;       // MT x 128 x 64 bf16 (either major)
    static constexpr uint32_t kB = BN * 128;             // BN x 64 bf16
    static constexpr uint32_t kStage = kA + kB;
    static constexpr uint32_t kOut = 128 * OUTW * 2;     // staging: [128][64] slabs, 128-byte swizzle (OUTW = 32: [128][32], 64-byte swizzle)
    static constexpr int kStages = (227 * 1024 - 1024 - kOutBufs * (int)kOut) / (int)kStage < 4 ? (227 * 1024 - 1024 - kOutBufs * (int)kOut) / (int)kStage : 4;
    static constexpr uint32_t oOut = kStages * kStage;
    static constexpr uint32_t oBar = oOut + kOutBufs * kOut;
    static constexpr uint32_t oMisc = oBar + 16 * 8;
    static constexpr uint32_t kBytes = oMisc + 64;
    static_assert(kStages >= 3 && kBytes <= 227 * 1024 && kStage % 1024 == 0 && kOut % 1024 == 0, "shared memory layout");
    static_assert(NBUF * MT * BN <= 512, "tensor memory");
};

__device__ __forceinline__ float ex2a(float x)
{
    float y;
    asm("ex2.approx.ftz.f32 %0, %1;" : "=f"(y) : "f"(x));
    return y;
}

// byte offset of (row, col) in a staging tile of W columns, as the TMA store reads it
template <int W>
__device__ __forceinline__ uint32_t stage_offset(uint32_t row, uint32_t col)
{
    if constexpr (W >= 64) return (col / 64) * (128u * 128u) + sw128_offset(row, col % 64);
    else return row * 64u + ((((col >> 3) ^ ((row >> 1) & 3u)) << 4) | ((col & 7u) << 1));   // 64-byte swizzle
}

// A_MN: A is stored [k][m] (m contiguous); otherwise [m][k].  B_MN: B stored [k][n]; otherwise [n][k].
template <int BN, int MT, bool A_MN, bool B_MN, int EPI>
__global__ void __launch_bounds__(kGemmThreads, 1)
mat_gemm_kernel(const __grid_constant__ CUtensorMap mA, const __grid_constant__ CUtensorMap mB,
                const __grid_constant__ CUtensorMap mC, const GemmArgs g)
{
    using L = GemmSmem<BN, MT>;
    constexpr int kStages = L::kStages, kOutBufs = L::kOutBufs, OUTW = L::OUTW;
    constexpr int NBUF = L::NBUF;            // accumulator sets that alternate between tiles
    constexpr int TM = 128 * MT;
    extern __shared__ __align__(1024) uint8_t smem[];
    uint64_t *full = reinterpret_cast<uint64_t *>(smem + L::oBar);
    uint64_t *empty = full + kStages;
    uint64_t *accfull = empty + kStages;
    uint64_t *accempty = accfull + 2;
    uint32_t *tmem_base_s = reinterpret_cast<uint32_t *>(smem + L::oMisc);
    volatile uint32_t *abort_flag = reinterpret_cast<volatile uint32_t *>(smem + L::oMisc + 4);
    const Abort ab{abort_flag, g.status};
    constexpr uint32_t kTmemCols = NBUF * MT * BN < 32 ? 32 : NBUF * MT * BN;

    const int tid = threadIdx.x, warp = tid / 32, lane = tid % 32;
    const int tiles_n = (g.n_total + BN - 1) / BN, tiles_m = (g.m_total + TM - 1) / TM;
    const long total = (long)tiles_n * tiles_m * g.heads;
    const int nk = (g.k_total + 63) / 64;
    // the product of a tile that lies wholly above the diagonal is not formed (its entries are exact zeros)
    auto skipped = [&](int m0, int n0) { return EPI == EPI_EXP && g.causal && n0 > m0 + TM - 1; };

    if ((smem_u32(smem) & 1023u) != 0) {
        if (tid == 0) atomicExch(g.status, 9u);
        return;
    }
    if (tid == 0) {
        *abort_flag = 0;
        for (int s = 0; s < kStages; ++s) { mbar_init(&full[s], 1); mbar_init(&empty[s], 1); }
        for (int b = 0; b < 2; ++b) { mbar_init(&accfull[b], 1); mbar_init(&accempty[b], kEpiWarps); }
        fence_barrier_init();
        prefetch_tensormap(&mA); prefetch_tensormap(&mB); prefetch_tensormap(&mC);
    }
    if (warp == 0) tmem_alloc(tmem_base_s, kTmemCols);
    tcgen05_fence_before();
    __syncthreads();
    tcgen05_fence_after();
    const uint32_t tm = *tmem_base_s;

    if (warp == kEpiWarps) {
        // ------------------------------------------------------------ TMA producer
        if (lane == 0) {
            int kc = 0;   // chunks loaded so far, over all tiles
            for (long t = blockIdx.x; t < total; t += gridDim.x) {
                const int head = (int)(t / ((long)tiles_n * tiles_m));
                const int m0 = (int)(t / tiles_n % tiles_m) * TM, n0 = (int)(t % tiles_n) * BN;
                if (skipped(m0, n0)) continue;
                for (int kt = 0; kt < nk; ++kt, ++kc) {
                    const int s = kc % kStages;
                    if (kc >= kStages) mbar_wait(&empty[s], ((kc / kStages) - 1) & 1, ab);
                    uint8_t *sA = smem + s * L::kStage, *sB = sA + L::kA;
                    mbar_expect_tx(&full[s], L::kStage);
                    if (A_MN) {
#pragma unroll
                        for (int q = 0; q < 2 * MT; ++q) tma_load_3d(sA + q * 8192, &mA, &full[s], m0 + q * 64, kt * 64, head);
                    } else {
#pragma unroll
                        for (int q = 0; q < MT; ++q) tma_load_3d(sA + q * 16384, &mA, &full[s], kt * 64, m0 + q * 128, head);
                    }
                    if (B_MN) {
#pragma unroll
                        for (int sl = 0; sl < BN / 64; ++sl) tma_load_3d(sB + sl * 8192, &mB, &full[s], n0 + sl * 64, kt * 64, head);
                    } else {
                        tma_load_3d(sB, &mB, &full[s], kt * 64, n0, head);
                    }
                }
            }
        }
    } else if (warp == kEpiWarps + 1) {
        // ------------------------------------------------------------ MMA issuer
        if (lane == 0) {
            constexpr uint32_t idesc = idesc_bf16(128, BN, A_MN ? 1 : 0, B_MN ? 1 : 0);
            int kc = 0, ai = 0;   // chunks consumed; accumulator sets filled
            for (long t = blockIdx.x; t < total; t += gridDim.x) {
                const int m0 = (int)(t / tiles_n % tiles_m) * TM, n0 = (int)(t % tiles_n) * BN;
                if (skipped(m0, n0)) continue;
                const int b = ai % NBUF;
                if (ai >= NBUF) {   // the epilogue has read the tile that used this accumulator set before
                    mbar_wait(&accempty[b], ((ai / NBUF) - 1) & 1, ab);
                    tcgen05_fence_after();
                }
                for (int kt = 0; kt < nk; ++kt, ++kc) {
                    const int s = kc % kStages;
                    mbar_wait(&full[s], (kc / kStages) & 1, ab);
                    tcgen05_fence_after();
                    const uint32_t sA = smem_u32(smem + s * L::kStage), sB = sA + L::kA;
                    const uint32_t db = B_MN ? desc_lo_mnmajor(sB, 8192) : desc_lo_kmajor(sB);
#pragma unroll
                    for (int q = 0; q < MT; ++q) {
                        const uint32_t da = A_MN ? desc_lo_mnmajor(sA + q * 16384, 8192) : desc_lo_kmajor(sA + q * 16384);
#pragma unroll
                        for (int ks = 0; ks < 4; ++ks)
                            mma_ss_lo(tm + (b * MT + q) * BN, da + ks * (A_MN ? 128 : 2), db + ks * (B_MN ? 128 : 2), idesc,
                                      (kt > 0) || (ks > 0));
                    }
                    mma_commit(&empty[s]);
                }
                mma_commit(&accfull[b]);
                ++ai;
            }
        }
    } else {
        // ------------------------------------------------------------ epilogue (warps 0-7): a tile leaves in steps of
        // 128 rows x OUTW columns; in every step warp w takes the lane quarter w % 4 (its rows) and the column half w / 4
        constexpr int CW = OUTW / 2, CH = CW < 32 ? CW : 32;
        const int row = (warp % 4) * 32 + lane, c_first = (warp / 4) * CW;
        const uint32_t lane_addr = (uint32_t)((warp % 4) * 32) << 16;
        int ai = 0, oi = 0;   // accumulator sets read; staging tiles written
        for (long t = blockIdx.x; t < total; t += gridDim.x) {
            const int head = (int)(t / ((long)tiles_n * tiles_m));
            const int m0 = (int)(t / tiles_n % tiles_m) * TM, n0 = (int)(t % tiles_n) * BN;
            const bool skip = skipped(m0, n0);
            const int b = ai % NBUF;
            // the row statistics of this thread's rows are fetched before the wait for the products, which hides the load
            float nlq[MT];
#pragma unroll
            for (int q = 0; q < MT; ++q) {
                nlq[q] = 0.f;
                if (EPI == EPI_EXP && m0 + q * 128 + row < g.m_total) nlq[q] = g.nlse2[(size_t)head * g.m_total + m0 + q * 128 + row];
            }
            if (!skip) {
                mbar_wait(&accfull[b], (ai / NBUF) & 1, ab);
                tcgen05_fence_after();
            }
#pragma unroll 1
            for (int step = 0; step < MT * (BN / OUTW); ++step, ++oi) {
                const int q = step / (BN / OUTW), cb = (step % (BN / OUTW)) * OUTW;   // row sub-tile, first column
                const int gi = m0 + q * 128 + row;
                const uint32_t acc = tm + lane_addr + (b * MT + q) * BN + cb + c_first;
                uint8_t *stage = smem + L::oOut + (oi % kOutBufs) * L::kOut;
                const float nl = MT == 1 ? nlq[0] : (q == 0 ? nlq[0] : nlq[MT - 1]);
                // the store that last read this staging tile is done with it
                if (tid == 0) {
                    if (kOutBufs == 1) asm volatile("cp.async.bulk.wait_group.read 0;" ::: "memory");
                    else asm volatile("cp.async.bulk.wait_group.read 1;" ::: "memory");
                }
                asm volatile("bar.sync 1, 256;" ::: "memory");
#pragma unroll
                for (int c = 0; c < CW; c += CH) {
                    uint32_t v[32];
                    if (!skip) {
                        if constexpr (CH == 32) tmem_ld32(acc + c, v);
                        else tmem_ld16(acc + c, *reinterpret_cast<uint32_t(*)[16]>(v));
                        tmem_wait_ld();
                    }
#pragma unroll
                    for (int e = 0; e < CH; e += 8) {
                        const int gj = n0 + cb + c_first + c + e;
                        float x[8];
#pragma unroll
                        for (int u = 0; u < 8; ++u) {
                            x[u] = skip ? 0.f : __uint_as_float(v[e + u]);
                            if (EPI == EPI_EXP) {
                                x[u] = ex2a(fmaf(x[u], g.sl2, nl));
                                if (skip || (g.causal && gj + u > gi)) x[u] = 0.f;
                            }
                        }
                        *reinterpret_cast<uint4 *>(stage + stage_offset<OUTW>(row, c_first + c + e)) =
                            make_uint4(pack_bf16(x[0], x[1]), pack_bf16(x[2], x[3]), pack_bf16(x[4], x[5]), pack_bf16(x[6], x[7]));
                    }
                }
                if (!skip && step + 1 == MT * (BN / OUTW)) {   // the accumulator set may take its next tile
                    tcgen05_fence_before();
                    bwdk::warp_arrive(&accempty[b], lane);
                }
                fence_proxy_async_smem();
                asm volatile("bar.sync 1, 256;" ::: "memory");
                if (tid == 0 && !*abort_flag) {
                    // rows beyond m_total and columns beyond n_total are clipped by the store
                    if constexpr (OUTW >= 64) {
#pragma unroll
                        for (int sl = 0; sl < OUTW / 64; ++sl) tma_store_3d(&mC, stage + sl * 16384, n0 + cb + sl * 64, m0 + q * 128, head);
                    } else {
                        tma_store_3d(&mC, stage, n0 + cb, m0 + q * 128, head);
                    }
                    tma_store_commit();
                }
            }
            if (!skip) ++ai;
        }
        if (tid == 0) tma_store_wait_all();
    }
    tcgen05_fence_before();
    __syncthreads();
    if (warp == 0) tmem_dealloc(tm, kTmemCols);
}

// phase 3: dS = P o (scale dP - scale D), 8 elements per thread per step
__global__ void __launch_bounds__(256) mat_ds_kernel(const uint4 *__restrict__ P, const uint4 *__restrict__ dP,
                                                     uint4 *__restrict__ dS, const float *__restrict__ Ds, size_t nvec,
                                                     int n, float scale)
{
    const int vec_per_row = n / 8;
    for (size_t i = (size_t)blockIdx.x * blockDim.x + threadIdx.x; i < nvec; i += (size_t)gridDim.x * blockDim.x) {
        const float d = Ds[i / vec_per_row];
        const uint4 p = P[i], q = dP[i];
        const __nv_bfloat162 *pp = reinterpret_cast<const __nv_bfloat162 *>(&p);
        const __nv_bfloat162 *qq = reinterpret_cast<const __nv_bfloat162 *>(&q);
        uint32_t o[4];
#pragma unroll
        for (int e = 0; e < 4; ++e) {
            const float2 fp = __bfloat1622float2(pp[e]), fq = __bfloat1622float2(qq[e]);
            o[e] = pack_bf16(fp.x * fmaf(fq.x, scale, -d), fp.y * fmaf(fq.y, scale, -d));
        }
        dS[i] = make_uint4(o[0], o[1], o[2], o[3]);
    }
}

// C: [heads][m_total][n_total] bf16, rows `ldc` elements apart, heads m_total * ldc elements apart
template <int BN, int MT, bool A_MN, bool B_MN, int EPI>
attn_status launch_gemm(const char *name, const CUtensorMap &mA, const CUtensorMap &mB, void *C, int ldc, GemmArgs g, int heads,
                        cudaStream_t s)
{
    using L = GemmSmem<BN, MT>;
    auto kernel = mat_gemm_kernel<BN, MT, A_MN, B_MN, EPI>;
    if (cudaFuncSetAttribute(kernel, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)L::kBytes) != cudaSuccess)
        return ATTN_ERR_LAUNCH;
    CUtensorMap mC;
    if (!make_tmap_bf16_3d_box(&mC, C, (uint64_t)g.n_total, (uint64_t)g.m_total, (uint64_t)heads, (uint64_t)ldc, BN < 64 ? BN : 64, 128,
                               BN < 64 ? 64 : 128))
        return ATTN_ERR_LAUNCH;
    g.heads = heads;
    const long total = (long)((g.n_total + BN - 1) / BN) * ((g.m_total + 128 * MT - 1) / (128 * MT)) * heads;
    // as many CTAs per SM as fit (registers, shared memory; 2 BN tensor-memory columns each): every CTA is resident
    int per_sm = 1;
    if (cudaOccupancyMaxActiveBlocksPerMultiprocessor(&per_sm, kernel, kGemmThreads, L::kBytes) != cudaSuccess || per_sm < 1) per_sm = 1;
    if (per_sm > 512 / (L::NBUF * MT * BN)) per_sm = 512 / (L::NBUF * MT * BN);
    if (per_sm > 2) per_sm = 2;
    const long ctas = (long)sm_count() * per_sm;
    launch_begin(name, s);
    kernel<<<(unsigned)(total < ctas ? total : ctas), kGemmThreads, L::kBytes, s>>>(mA, mB, mC, g);
    launch_end(s);
    return cudaGetLastError() == cudaSuccess ? ATTN_OK : ATTN_ERR_LAUNCH;
}

template <int TK, int MT>
attn_status run_scores(const Problem &p, size_t h0, int mh)
{
    const int n = p.n, d = p.d;
    const __nv_bfloat16 *Q = (const __nv_bfloat16 *)p.Q + h0 * n * d, *K = (const __nv_bfloat16 *)p.K + h0 * n * d,
                        *V = (const __nv_bfloat16 *)p.V + h0 * n * d, *dO = (const __nv_bfloat16 *)p.dO + h0 * n * d;
    CUtensorMap mQ, mK, mV, mdO;
    if (!make_tmap_bf16_3d(&mQ, Q, d, n, mh, 128) || !make_tmap_bf16_3d(&mdO, dO, d, n, mh, 128) ||
        !make_tmap_bf16_3d(&mK, K, d, n, mh, TK) || !make_tmap_bf16_3d(&mV, V, d, n, mh, TK))
        return ATTN_ERR_LAUNCH;
    GemmArgs g{};
    g.m_total = n; g.n_total = n; g.k_total = d;
    g.status = p.status;
    // phase 1: P = exp(scale Q K^T - LSE)
    g.nlse2 = p.nLSE2 + h0 * n; g.sl2 = p.scale * 1.4426950408889634f; g.causal = p.mask_kind == ATTN_MASK_CAUSAL;
    attn_status st = launch_gemm<TK, MT, false, false, EPI_EXP>("mat_phase1_P", mQ, mK, p.matP, n, g, mh, p.stream);
    if (st != ATTN_OK) return st;
    // phase 2: dP = dO V^T
    g.causal = 0;
    return launch_gemm<TK, MT, false, false, EPI_PLAIN>("mat_phase2_dP", mdO, mV, p.matdP, n, g, mh, p.stream);
}

attn_status run_chunk(const Problem &p, size_t h0, int mh)
{
    const int n = p.n, d = p.d;
    attn_status st;
    if (p.cfg.tile_q == 256) {
        if (p.cfg.tile_k == 128) st = run_scores<128, 2>(p, h0, mh);
        else if (p.cfg.tile_k == 64) st = run_scores<64, 2>(p, h0, mh);
        else st = run_scores<32, 2>(p, h0, mh);
    } else {
        if (p.cfg.tile_k == 128) st = run_scores<128, 1>(p, h0, mh);
        else if (p.cfg.tile_k == 64) st = run_scores<64, 1>(p, h0, mh);
        else st = run_scores<32, 1>(p, h0, mh);
    }
    if (st != ATTN_OK) return st;
    // phase 3: dS = scale P o (dP - D)
    {
        const size_t nvec = (size_t)mh * n * n / 8;
        const size_t cap = (size_t)sm_count() * 16;
        const unsigned blocks = (unsigned)((nvec + 255) / 256 < cap ? (nvec + 255) / 256 : cap);
        launch_begin("mat_phase3_dS", p.stream);
        mat_ds_kernel<<<blocks, 256, 0, p.stream>>>((const uint4 *)p.matP, (const uint4 *)p.matdP, (uint4 *)p.matdS,
                                                    p.D + h0 * n, nvec, n, p.scale);
        launch_end(p.stream);
        if (cudaGetLastError() != cudaSuccess) return ATTN_ERR_LAUNCH;
    }
    // phase 4: dV = P^T dO, dK = dS^T Q, dQ = dS K
    const __nv_bfloat16 *Q = (const __nv_bfloat16 *)p.Q + h0 * n * d, *K = (const __nv_bfloat16 *)p.K + h0 * n * d,
                        *dO = (const __nv_bfloat16 *)p.dO + h0 * n * d;
    CUtensorMap mPt, mdSt, mdS, mQ, mK, mdO;
    if (!make_tmap_bf16_3d(&mPt, p.matP, n, n, mh, 64) || !make_tmap_bf16_3d(&mdSt, p.matdS, n, n, mh, 64) ||
        !make_tmap_bf16_3d(&mdS, p.matdS, n, n, mh, 128) || !make_tmap_bf16_3d(&mQ, Q, d, n, mh, 64) ||
        !make_tmap_bf16_3d(&mK, K, d, n, mh, 64) || !make_tmap_bf16_3d(&mdO, dO, d, n, mh, 64))
        return ATTN_ERR_LAUNCH;
    GemmArgs g{};
    g.m_total = n; g.n_total = d; g.k_total = n;
    g.status = p.status;
    __nv_bfloat16 *dV = (__nv_bfloat16 *)p.dV + h0 * n * d, *dK = (__nv_bfloat16 *)p.dK + h0 * n * d,
                  *dQ = (__nv_bfloat16 *)p.dQ + h0 * n * d;
    auto phase4 = [&](auto bn) -> attn_status {
        constexpr int BN = decltype(bn)::value;
        attn_status r;
        if ((r = launch_gemm<BN, 2, true, true, EPI_OUT>("mat_phase4_dV", mPt, mdO, dV, d, g, mh, p.stream)) != ATTN_OK) return r;
        if ((r = launch_gemm<BN, 2, true, true, EPI_OUT>("mat_phase4_dK", mdSt, mQ, dK, d, g, mh, p.stream)) != ATTN_OK) return r;
        return launch_gemm<BN, 2, false, true, EPI_OUT>("mat_phase4_dQ", mdS, mK, dQ, d, g, mh, p.stream);
    };
    if (d == 256) return phase4(std::integral_constant<int, 256>{});
    if (d == 128) return phase4(std::integral_constant<int, 128>{});
    return phase4(std::integral_constant<int, 64>{});
}

}  // namespace

// tile_q in {128, 256} x tile_k in {128, 64, 32} is the block of the n x n matrices in phases 1 and 2;
// tile_d = 64 is the chunk in which every contraction is walked.  Phase 4 always forms 256 x d tiles.
bool mat_cfg_supported(int d, const attn_cfg &c)
{
    if (d != 64 && d != 128 && d != 256) return false;
    if (c.tile_q != 0 && c.tile_q != 128 && c.tile_q != 256) return false;
    if (c.tile_k != 0 && c.tile_k != 128 && c.tile_k != 64 && c.tile_k != 32) return false;
    return c.tile_d == 0 || c.tile_d == 64;
}

// On-chip bytes of a phase-1/2 CTA: operand ring + fp32 accumulator tiles in tensor memory + staging tiles of C.
template <int BN, int MT> constexpr size_t gemm_onchip()
{
    using L = GemmSmem<BN, MT>;
    return (size_t)L::kStages * L::kStage + (size_t)L::kOutBufs * L::kOut + (size_t)L::NBUF * MT * BN * 128 * 4;
}
size_t mat_onchip_bytes(int, const attn_cfg &c)
{
    const int tk = c.tile_k ? c.tile_k : 128;
    if (c.tile_q == 256) return tk == 128 ? gemm_onchip<128, 2>() : tk == 64 ? gemm_onchip<64, 2>() : gemm_onchip<32, 2>();
    return tk == 128 ? gemm_onchip<128, 1>() : tk == 64 ? gemm_onchip<64, 1>() : gemm_onchip<32, 1>();
}

attn_status mat_bwd(const Problem &p)
{
    if (mask_is_block(p.mask_kind)) return ATTN_ERR_MASK;
    if (bwd_preprocess_launch(p, false) != ATTN_OK) return ATTN_ERR_LAUNCH;   // Ds = scale D, -LSE log2e
    for (size_t h0 = 0; h0 < (size_t)p.BH; h0 += p.mat_heads) {
        const int mh = (int)((size_t)p.BH - h0 < (size_t)p.mat_heads ? (size_t)p.BH - h0 : (size_t)p.mat_heads);
        const attn_status st = run_chunk(p, h0, mh);
        if (st != ATTN_OK) return st;
    }
    return ATTN_OK;
}

}  // namespace attn

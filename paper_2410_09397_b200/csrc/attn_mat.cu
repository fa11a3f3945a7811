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
// One GEMM kernel serves all products: a CTA computes a 128 x BN tile of C with fp32
// accumulators in tensor memory; a TMA producer warp and an MMA issuer warp run a
// 4-stage ring of 64-deep operand chunks; four warps run the epilogue.  Operands are
// taken K-major or MN-major straight from their row-major arrays (no transposes).
#include "attn_internal.h"
#include "tc_common.cuh"

namespace attn {
namespace {

using namespace tc;

enum { EPI_EXP = 0, EPI_PLAIN = 1, EPI_OUT = 2 };
constexpr int kStages = 4;
constexpr int kGemmThreads = 192;

struct GemmArgs {
    __nv_bfloat16 *C;        // output base (head 0 of this launch)
    size_t c_head_stride;    // elements between heads of C
    int ldc;                 // row pitch of C in elements
    int m_total, n_total;    // valid rows / cols of C per head
    int k_total;             // contraction length
    const float *nlse2;      // EPI_EXP: -LSE log2e per row [heads][m_total]
    float sl2;               // EPI_EXP: scale * log2e
    int causal;              // EPI_EXP: zero entries with col > row
    uint32_t *status;
};

template <int BN>
struct GemmSmem {
    static constexpr uint32_t kA = 128 * 128;           // 128 x 64 bf16 (either major)
    static constexpr uint32_t kB = BN * 128;            // BN x 64 bf16
    static constexpr uint32_t kStage = kA + kB;
    static constexpr uint32_t oBar = kStages * kStage;
    static constexpr uint32_t oMisc = oBar + 16 * 8;
    static constexpr uint32_t kBytes = oMisc + 64;
};

__device__ __forceinline__ float ex2a(float x)
{
    float y;
    asm("ex2.approx.ftz.f32 %0, %1;" : "=f"(y) : "f"(x));
    return y;
}

// A_MN: A is stored [k][m] (m contiguous); otherwise [m][k].  B_MN: B stored [k][n]; otherwise [n][k].
template <int BN, bool A_MN, bool B_MN, int EPI>
__global__ void __launch_bounds__(kGemmThreads)
mat_gemm_kernel(const __grid_constant__ CUtensorMap mA, const __grid_constant__ CUtensorMap mB, const GemmArgs g)
{
    using L = GemmSmem<BN>;
    extern __shared__ __align__(1024) uint8_t smem[];
    uint64_t *full = reinterpret_cast<uint64_t *>(smem + L::oBar);
    uint64_t *empty = full + kStages;
    uint64_t *done = empty + kStages;
    uint32_t *tmem_base_s = reinterpret_cast<uint32_t *>(smem + L::oMisc);
    volatile uint32_t *abort_flag = reinterpret_cast<volatile uint32_t *>(smem + L::oMisc + 4);
    const Abort ab{abort_flag, g.status};
    constexpr uint32_t kTmemCols = BN < 32 ? 32 : BN;

    const int tid = threadIdx.x, warp = tid / 32, lane = tid % 32;
    const int n0 = blockIdx.x * BN, m0 = blockIdx.y * 128, head = blockIdx.z;
    const int nk = (g.k_total + 63) / 64;

    if ((smem_u32(smem) & 1023u) != 0) {
        if (tid == 0) atomicExch(g.status, 9u);
        return;
    }
    if (tid == 0) {
        *abort_flag = 0;
        for (int s = 0; s < kStages; ++s) { mbar_init(&full[s], 1); mbar_init(&empty[s], 1); }
        mbar_init(done, 1);
        fence_barrier_init();
        prefetch_tensormap(&mA); prefetch_tensormap(&mB);
    }
    if (warp == 0) tmem_alloc(tmem_base_s, kTmemCols);
    tcgen05_fence_before();
    __syncthreads();
    tcgen05_fence_after();
    const uint32_t tm = *tmem_base_s;

    if (warp == 4) {
        if (lane == 0) {
            for (int kt = 0; kt < nk; ++kt) {
                const int s = kt % kStages;
                if (kt >= kStages) mbar_wait(&empty[s], ((kt / kStages) - 1) & 1, ab);
                uint8_t *sA = smem + s * L::kStage, *sB = sA + L::kA;
                mbar_expect_tx(&full[s], L::kStage);
                if (A_MN) {
                    tma_load_3d(sA, &mA, &full[s], m0, kt * 64, head);
                    tma_load_3d(sA + 8192, &mA, &full[s], m0 + 64, kt * 64, head);
                } else {
                    tma_load_3d(sA, &mA, &full[s], kt * 64, m0, head);
                }
                if (B_MN) {
#pragma unroll
                    for (int sl = 0; sl < BN / 64; ++sl) tma_load_3d(sB + sl * 8192, &mB, &full[s], n0 + sl * 64, kt * 64, head);
                } else {
                    tma_load_3d(sB, &mB, &full[s], kt * 64, n0, head);
                }
            }
        }
    } else if (warp == 5) {
        if (lane == 0) {
            constexpr uint32_t idesc = idesc_bf16(128, BN, A_MN ? 1 : 0, B_MN ? 1 : 0);
            for (int kt = 0; kt < nk; ++kt) {
                const int s = kt % kStages;
                mbar_wait(&full[s], (kt / kStages) & 1, ab);
                tcgen05_fence_after();
                const uint32_t sA = smem_u32(smem + s * L::kStage), sB = sA + L::kA;
#pragma unroll
                for (int ks = 0; ks < 4; ++ks) {
                    const uint64_t da = A_MN ? smem_desc_mnmajor(sA + ks * 2048, 8192) : smem_desc_kmajor(sA + ks * 32);
                    const uint64_t db = B_MN ? smem_desc_mnmajor(sB + ks * 2048, 8192) : smem_desc_kmajor(sB + ks * 32);
                    mma_ss(tm, da, db, idesc, (kt > 0) || (ks > 0));
                }
                mma_commit(&empty[s]);
            }
            mma_commit(done);
        }
    } else {
        // ------------------------------------------------------------ epilogue (warps 0-3)
        const int row = warp * 32 + lane, gi = m0 + row;
        const uint32_t lane_addr = (uint32_t)(warp * 32) << 16;
        mbar_wait(done, 0, ab);
        tcgen05_fence_after();
        const bool row_ok = gi < g.m_total;
        __nv_bfloat16 *crow = g.C + (size_t)head * g.c_head_stride + (size_t)(row_ok ? gi : 0) * g.ldc + n0;
        float nl = 0.f;
        if (EPI == EPI_EXP && row_ok) nl = g.nlse2[(size_t)head * g.m_total + gi];
        constexpr int CH = BN < 32 ? BN : 32;
#pragma unroll 1
        for (int c = 0; c < BN; c += CH) {
            uint32_t v[32];
            if (CH == 32) tmem_ld32(tm + lane_addr + c, v);
            else tmem_ld16(tm + lane_addr + c, *reinterpret_cast<uint32_t(*)[16]>(v));
            tmem_wait_ld();
            if (!row_ok) continue;
#pragma unroll
            for (int e = 0; e < CH; e += 8) {
                const int gj = n0 + c + e;
                if (gj >= g.n_total) break;
                float x[8];
#pragma unroll
                for (int u = 0; u < 8; ++u) {
                    x[u] = __uint_as_float(v[e + u]);
                    if (EPI == EPI_EXP) {
                        x[u] = ex2a(fmaf(x[u], g.sl2, nl));
                        if (g.causal && gj + u > gi) x[u] = 0.f;
                    }
                }
                *reinterpret_cast<uint4 *>(crow + c + e) =
                    make_uint4(pack_bf16(x[0], x[1]), pack_bf16(x[2], x[3]), pack_bf16(x[4], x[5]), pack_bf16(x[6], x[7]));
            }
        }
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

// D pre-pass for d = 256: Ds = scale * rowsum(dO o O), nlse2 = -LSE log2e (one warp per row)
__global__ void __launch_bounds__(256) mat_preprocess_kernel(const __nv_bfloat16 *__restrict__ O,
                                                             const __nv_bfloat16 *__restrict__ dO,
                                                             const float *__restrict__ LSE, float *__restrict__ Ds,
                                                             float *__restrict__ nlse2, size_t rows, int d, float scale)
{
    const int lane = threadIdx.x % 32;
    const size_t warp = ((size_t)blockIdx.x * blockDim.x + threadIdx.x) / 32;
    const size_t nwarps = (size_t)gridDim.x * blockDim.x / 32;
    const int vec = d / 8;
    for (size_t row = warp; row < rows; row += nwarps) {
        float acc = 0.f;
        for (int v = lane; v < vec; v += 32) {
            const uint4 xo = __ldg(reinterpret_cast<const uint4 *>(O + row * d) + v);
            const uint4 xg = __ldg(reinterpret_cast<const uint4 *>(dO + row * d) + v);
            const __nv_bfloat162 *eo = reinterpret_cast<const __nv_bfloat162 *>(&xo);
            const __nv_bfloat162 *eg = reinterpret_cast<const __nv_bfloat162 *>(&xg);
#pragma unroll
            for (int e = 0; e < 4; ++e) {
                const float2 fo = __bfloat1622float2(eo[e]), fg = __bfloat1622float2(eg[e]);
                acc = fmaf(fo.x, fg.x, acc);
                acc = fmaf(fo.y, fg.y, acc);
            }
        }
#pragma unroll
        for (int o = 16; o > 0; o >>= 1) acc += __shfl_xor_sync(0xffffffffu, acc, o);
        if (lane == 0) {
            Ds[row] = acc * scale;
            const float l = LSE[row];
            nlse2[row] = l == -INFINITY ? -INFINITY : -l * 1.4426950408889634f;
        }
    }
}

template <int BN, bool A_MN, bool B_MN, int EPI>
attn_status launch_gemm(const char *name, const CUtensorMap &mA, const CUtensorMap &mB, const GemmArgs &g, int heads,
                        cudaStream_t s)
{
    using L = GemmSmem<BN>;
    auto kernel = mat_gemm_kernel<BN, A_MN, B_MN, EPI>;
    if (cudaFuncSetAttribute(kernel, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)L::kBytes) != cudaSuccess)
        return ATTN_ERR_LAUNCH;
    const dim3 grid((g.n_total + BN - 1) / BN, (g.m_total + 127) / 128, heads);
    launch_begin(name, s);
    kernel<<<grid, kGemmThreads, L::kBytes, s>>>(mA, mB, g);
    launch_end(s);
    return cudaGetLastError() == cudaSuccess ? ATTN_OK : ATTN_ERR_LAUNCH;
}

template <int TK>
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
    g.c_head_stride = (size_t)n * n; g.ldc = n; g.m_total = n; g.n_total = n; g.k_total = d;
    g.status = p.status;
    // phase 1: P = exp(scale Q K^T - LSE)
    g.C = (__nv_bfloat16 *)p.matP;
    g.nlse2 = p.nLSE2 + h0 * n; g.sl2 = p.scale * 1.4426950408889634f; g.causal = p.mask_kind == ATTN_MASK_CAUSAL;
    attn_status st = launch_gemm<TK, false, false, EPI_EXP>("mat_phase1_P", mQ, mK, g, mh, p.stream);
    if (st != ATTN_OK) return st;
    // phase 2: dP = dO V^T
    g.C = (__nv_bfloat16 *)p.matdP; g.causal = 0;
    return launch_gemm<TK, false, false, EPI_PLAIN>("mat_phase2_dP", mdO, mV, g, mh, p.stream);
}

attn_status run_chunk(const Problem &p, size_t h0, int mh)
{
    const int n = p.n, d = p.d;
    attn_status st;
    if (p.cfg.tile_k == 128) st = run_scores<128>(p, h0, mh);
    else if (p.cfg.tile_k == 64) st = run_scores<64>(p, h0, mh);
    else st = run_scores<32>(p, h0, mh);
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
    g.c_head_stride = (size_t)n * d; g.ldc = d; g.m_total = n; g.n_total = d; g.k_total = n;
    g.status = p.status;
    g.C = (__nv_bfloat16 *)p.dV + h0 * n * d;
    if (d == 256) {
        if ((st = launch_gemm<256, true, true, EPI_OUT>("mat_phase4_dV", mPt, mdO, g, mh, p.stream)) != ATTN_OK) return st;
        g.C = (__nv_bfloat16 *)p.dK + h0 * n * d;
        if ((st = launch_gemm<256, true, true, EPI_OUT>("mat_phase4_dK", mdSt, mQ, g, mh, p.stream)) != ATTN_OK) return st;
        g.C = (__nv_bfloat16 *)p.dQ + h0 * n * d;
        return launch_gemm<256, false, true, EPI_OUT>("mat_phase4_dQ", mdS, mK, g, mh, p.stream);
    } else if (d == 128) {
        if ((st = launch_gemm<128, true, true, EPI_OUT>("mat_phase4_dV", mPt, mdO, g, mh, p.stream)) != ATTN_OK) return st;
        g.C = (__nv_bfloat16 *)p.dK + h0 * n * d;
        if ((st = launch_gemm<128, true, true, EPI_OUT>("mat_phase4_dK", mdSt, mQ, g, mh, p.stream)) != ATTN_OK) return st;
        g.C = (__nv_bfloat16 *)p.dQ + h0 * n * d;
        return launch_gemm<128, false, true, EPI_OUT>("mat_phase4_dQ", mdS, mK, g, mh, p.stream);
    }
    if ((st = launch_gemm<64, true, true, EPI_OUT>("mat_phase4_dV", mPt, mdO, g, mh, p.stream)) != ATTN_OK) return st;
    g.C = (__nv_bfloat16 *)p.dK + h0 * n * d;
    if ((st = launch_gemm<64, true, true, EPI_OUT>("mat_phase4_dK", mdSt, mQ, g, mh, p.stream)) != ATTN_OK) return st;
    g.C = (__nv_bfloat16 *)p.dQ + h0 * n * d;
    return launch_gemm<64, false, true, EPI_OUT>("mat_phase4_dQ", mdS, mK, g, mh, p.stream);
}

}  // namespace

// tile_q = 128; tile_k in {128, 64, 32} is the block edge of the n x n matrices in phases
// 1 and 2; tile_d = 64 is the chunk in which every contraction is walked.
bool mat_cfg_supported(int d, const attn_cfg &c)
{
    if (d != 64 && d != 128 && d != 256) return false;
    if (c.tile_q != 0 && c.tile_q != 128) return false;
    if (c.tile_k != 0 && c.tile_k != 128 && c.tile_k != 64 && c.tile_k != 32) return false;
    return c.tile_d == 0 || c.tile_d == 64;
}

// On-chip bytes of a phase-1/2 CTA: operand ring + fp32 accumulator tile in tensor memory.
size_t mat_onchip_bytes(int, const attn_cfg &c)
{
    const int tk = c.tile_k ? c.tile_k : 128;
    return (size_t)kStages * (128 * 128 + tk * 128) + (size_t)128 * tk * 4;
}

attn_status mat_bwd(const Problem &p)
{
    if (mask_is_block(p.mask_kind)) return ATTN_ERR_MASK;
    const size_t rows = (size_t)p.BH * p.n;
    size_t blocks = (rows + 7) / 8;
    if (blocks > (size_t)sm_count() * 8) blocks = (size_t)sm_count() * 8;
    launch_begin("mat_preprocess", p.stream);
    mat_preprocess_kernel<<<(unsigned)blocks, 256, 0, p.stream>>>((const __nv_bfloat16 *)p.O, (const __nv_bfloat16 *)p.dO,
                                                                  p.LSE, p.D, p.nLSE2, rows, p.d, p.scale);
    launch_end(p.stream);
    if (cudaGetLastError() != cudaSuccess) return ATTN_ERR_LAUNCH;
    for (size_t h0 = 0; h0 < (size_t)p.BH; h0 += p.mat_heads) {
        const int mh = (int)((size_t)p.BH - h0 < (size_t)p.mat_heads ? (size_t)p.BH - h0 : (size_t)p.mat_heads);
        const attn_status st = run_chunk(p, h0, mh);
        if (st != ATTN_OK) return st;
    }
    return ATTN_OK;
}

}  // namespace attn

// The attention weights X and Y of the paper's own problem statement (Definition 3.1:
// S = A1 X, h = A3 Y; Definition 3.2: dL/dX = A1^T p A2):
//
//   attn_project       out = A W per (batch, head) unit        (Appendix D, phase 1)
//   attn_weight_grad   g  += A^T G over the units of a weight  (closing product of phase 2)
//   attn_weights_bwd   phase 2 as a whole: attn_bwd for p A2 and f^T dO, then the two
//                      weight-gradient products (the first one straight from the fp32
//                      dQ accumulator where the backward has one)
//
// Both products stream n x d operands once and produce (or consume) a d x d matrix, so
// they are bound by HBM bandwidth; the bf16 kernels use tcgen05 only so that the
// arithmetic stays hidden behind the loads.  Any other dtype / head size takes the
// fp32 FMA kernels at the end of the file.
#include "attn_internal.h"
#include "tc_common.cuh"

namespace attn {
namespace {

using namespace tc;

constexpr uint32_t kStatusBytes = 256;

__device__ __forceinline__ void red_add_v4(float *p, float a, float b, float c, float d)
{
    asm volatile("red.global.add.v4.f32 [%0], {%1, %2, %3, %4};" ::"l"(p), "f"(a), "f"(b), "f"(c), "f"(d) : "memory");
}

// ===================================================================== out = A W (bf16), one tile per CTA (d = 256)
// One CTA per 128-row tile of one unit.  A tile K-major (contraction along d), W MN-major
// (rows of W are the contraction index), accumulator [128 rows][HD] in tensor memory.
template <int HD> struct ProjSmem {
    static constexpr uint32_t kASlab = 128 * 128;            // [128 rows][64 bf16]
    static constexpr uint32_t kWSlab = HD * 128;             // [HD rows][64 bf16]
    static constexpr uint32_t oA = 0;
    static constexpr uint32_t oW = oA + (HD / 64) * kASlab;
    static constexpr uint32_t oBar = oW + (HD / 64) * kWSlab;
    static constexpr uint32_t oMisc = oBar + 64;
    static constexpr uint32_t kBytes = oMisc + 64;
    static constexpr uint32_t kTx = (HD / 64) * (kASlab + kWSlab);
    static_assert(kBytes <= 227 * 1024, "shared memory budget");
};

struct ProjArgs {
    __nv_bfloat16 *out;
    uint32_t *status;
    int n;
    long weight_units;
};

constexpr int kProjThreads = 192;   // warps 0-3 epilogue, warp 4 TMA, warp 5 MMA

template <int HD>
__global__ void __launch_bounds__(kProjThreads)
wproj_kernel(const __grid_constant__ CUtensorMap mA, const __grid_constant__ CUtensorMap mW, const ProjArgs g)
{
    using L = ProjSmem<HD>;
    extern __shared__ __align__(1024) uint8_t smem[];
    uint64_t *full = reinterpret_cast<uint64_t *>(smem + L::oBar);
    uint64_t *done = full + 1;
    uint32_t *tmem_base_s = reinterpret_cast<uint32_t *>(smem + L::oMisc);
    volatile uint32_t *abort_flag = reinterpret_cast<volatile uint32_t *>(smem + L::oMisc + 4);
    const Abort ab{abort_flag, g.status};
    constexpr uint32_t kTmemCols = HD;

    const int tid = threadIdx.x, warp = tid / 32, lane = tid % 32;
    const int m0 = blockIdx.x * 128;
    const long unit = blockIdx.y;

    if ((smem_u32(smem) & 1023u) != 0) {
        if (tid == 0) atomicExch(g.status, 9u);
        return;
    }
    if (tid == 0) {
        *abort_flag = 0;
        mbar_init(full, 1);
        mbar_init(done, 1);
        fence_barrier_init();
        prefetch_tensormap(&mA); prefetch_tensormap(&mW);
    }
    if (warp == 0) tmem_alloc(tmem_base_s, kTmemCols);
    tcgen05_fence_before();
    __syncthreads();
    tcgen05_fence_after();
    const uint32_t tm = *tmem_base_s;

    if (warp == 4) {
        if (lane == 0) {
            mbar_expect_tx(full, L::kTx);
#pragma unroll
            for (int sl = 0; sl < HD / 64; ++sl) {
                tma_load_3d(smem + L::oA + sl * L::kASlab, &mA, full, sl * 64, m0, (int)unit);
                tma_load_3d(smem + L::oW + sl * L::kWSlab, &mW, full, sl * 64, 0, (int)(unit % g.weight_units));
            }
        }
    } else if (warp == 5) {
        if (lane == 0) {
            constexpr uint32_t idesc = idesc_bf16(128, HD, 0, 1);
            mbar_wait(full, 0, ab);
            tcgen05_fence_after();
            const uint32_t sA = smem_u32(smem + L::oA);
            const uint32_t bW = desc_lo_mnmajor(smem_u32(smem + L::oW), L::kWSlab);
#pragma unroll
            for (int ks = 0; ks < HD / 16; ++ks) {
                const uint32_t aA = desc_lo_kmajor(sA + (ks / 4) * L::kASlab + (ks % 4) * 32);
                mma_ss_lo(tm, aA, bW + ks * (2048 >> 4), idesc, ks > 0);
            }
            mma_commit(done);
        }
    } else {
        const int gi = m0 + warp * 32 + lane;
        const uint32_t lane_addr = (uint32_t)(warp * 32) << 16;
        mbar_wait(done, 0, ab);
        tcgen05_fence_after();
        const bool row_ok = gi < g.n;
        __nv_bfloat16 *orow = g.out + ((size_t)unit * g.n + (row_ok ? gi : 0)) * HD;
#pragma unroll 1
        for (int c = 0; c < HD; c += 32) {
            uint32_t v[32];
            tmem_ld32(tm + lane_addr + c, v);
            tmem_wait_ld();
            if (!row_ok) continue;
#pragma unroll
            for (int e = 0; e < 32; e += 8)
                *reinterpret_cast<uint4 *>(orow + c + e) = make_uint4(
                    pack_bf16(__uint_as_float(v[e]), __uint_as_float(v[e + 1])),
                    pack_bf16(__uint_as_float(v[e + 2]), __uint_as_float(v[e + 3])),
                    pack_bf16(__uint_as_float(v[e + 4]), __uint_as_float(v[e + 5])),
                    pack_bf16(__uint_as_float(v[e + 6]), __uint_as_float(v[e + 7])));
        }
    }
    tcgen05_fence_before();
    __syncthreads();
    if (warp == 0) tmem_dealloc(tm, kTmemCols);
}

// ===================================================================== out = A W, persistent (d = 64, 128)
// CTA c takes a contiguous range of the (unit, 128-row tile) list.  A tiles arrive through a
// ring of TMA stages, W is loaded when the range starts and again whenever the unit's weight
// index changes, the accumulator is double-buffered in tensor memory, and the bf16 result
// leaves through a double-buffered staging tile and TMA stores, so that loads, products and
// stores of neighbouring tiles overlap.
template <int HD> struct ProjPSmem {
    static constexpr int kStages = HD == 128 ? 3 : 4;
    static constexpr uint32_t kASlab = 128 * 128;
    static constexpr uint32_t kATile = (HD / 64) * kASlab;
    static constexpr uint32_t kWSlab = HD * 128;
    static constexpr uint32_t kW = (HD / 64) * kWSlab;
    static constexpr uint32_t oA = 0;
    static constexpr uint32_t oW = oA + kStages * kATile;
    static constexpr uint32_t oOut = oW + kW;
    static constexpr uint32_t oBar = oOut + 2 * kATile;
    static constexpr uint32_t oMisc = oBar + 256;
    static constexpr uint32_t kBytes = oMisc + 64;
    static_assert(oW % 1024 == 0 && oOut % 1024 == 0, "tile bases are 1024-byte aligned");
    static_assert(kBytes <= 227 * 1024, "shared memory budget");
};

struct ProjPArgs {
    uint32_t *status;
    int tiles_per_unit;
    long total_tiles, weight_units;
};

template <int HD>
__global__ void __launch_bounds__(kProjThreads)
wproj_persistent_kernel(const __grid_constant__ CUtensorMap mA, const __grid_constant__ CUtensorMap mW,
                        const __grid_constant__ CUtensorMap mOut, const ProjPArgs g)
{
    using L = ProjPSmem<HD>;
    constexpr int kStages = L::kStages;
    extern __shared__ __align__(1024) uint8_t smem[];
    uint64_t *afull = reinterpret_cast<uint64_t *>(smem + L::oBar);
    uint64_t *aempty = afull + kStages;
    uint64_t *wfull = aempty + kStages;
    uint64_t *wfree = wfull + 1;
    uint64_t *accfull = wfree + 1;
    uint64_t *accempty = accfull + 2;
    uint32_t *tmem_base_s = reinterpret_cast<uint32_t *>(smem + L::oMisc);
    volatile uint32_t *abort_flag = reinterpret_cast<volatile uint32_t *>(smem + L::oMisc + 4);
    const Abort ab{abort_flag, g.status};
    constexpr uint32_t kTmemCols = 2 * HD;

    const int tid = threadIdx.x, warp = tid / 32, lane = tid % 32;
    const long t0 = g.total_tiles * blockIdx.x / gridDim.x, t1 = g.total_tiles * (blockIdx.x + 1) / gridDim.x;

    if ((smem_u32(smem) & 1023u) != 0) {
        if (tid == 0) atomicExch(g.status, 9u);
        return;
    }
    auto load_W = [&](long wi) {
        mbar_expect_tx(wfull, L::kW);
#pragma unroll
        for (int sl = 0; sl < HD / 64; ++sl) tma_load_3d(smem + L::oW + sl * L::kWSlab, &mW, wfull, sl * 64, 0, (int)wi);
    };
    auto load_A = [&](int kt, long t) {
        const int s = kt % kStages;
        const int unit = (int)(t / g.tiles_per_unit), r0 = (int)(t % g.tiles_per_unit) * 128;
        mbar_expect_tx(&afull[s], L::kATile);
#pragma unroll
        for (int sl = 0; sl < HD / 64; ++sl)
            tma_load_3d(smem + L::oA + s * L::kATile + sl * L::kASlab, &mA, &afull[s], sl * 64, r0, unit);
    };
    // tiles the producer can fetch before anything else is set up: the first ring-full that shares the first weight
    const long w_first = (t0 / g.tiles_per_unit) % g.weight_units;
    int early = 0;
    while (early < kStages && t0 + early < t1 && ((t0 + early) / g.tiles_per_unit) % g.weight_units == w_first) ++early;
    if (tid == 0) {
        *abort_flag = 0;
        for (int b = 0; b < 2; ++b) { mbar_init(&accfull[b], 1); mbar_init(&accempty[b], 128); }
        fence_barrier_init();
        prefetch_tensormap(&mOut);
    }
    if (tid == 4 * 32) {
        for (int s = 0; s < kStages; ++s) { mbar_init(&afull[s], 1); mbar_init(&aempty[s], 1); }
        mbar_init(wfull, 1);
        mbar_init(wfree, 1);
        fence_barrier_init();
        load_W(w_first);
        for (int kt = 0; kt < early; ++kt) load_A(kt, t0 + kt);
    }
    if (warp == 0) tmem_alloc(tmem_base_s, kTmemCols);
    tcgen05_fence_before();
    __syncthreads();
    tcgen05_fence_after();
    const uint32_t tm = *tmem_base_s;

    if (warp == 4) {
        if (lane == 0) {
            int kt = early, wloads = 1;
            long wprev = w_first;
            for (long t = t0 + early; t < t1; ++t, ++kt) {
                const long wi = (t / g.tiles_per_unit) % g.weight_units;
                if (wi != wprev) {
                    mbar_wait(wfree, (wloads - 1) & 1, ab);   // products with the old W are done
                    load_W(wi);
                    ++wloads;
                    wprev = wi;
                }
                if (kt >= kStages) mbar_wait(&aempty[kt % kStages], ((kt / kStages) - 1) & 1, ab);
                load_A(kt, t);
            }
        }
    } else if (warp == 5) {
        if (lane == 0) {
            constexpr uint32_t idesc = idesc_bf16(128, HD, 0, 1);
            const uint32_t bW = desc_lo_mnmajor(smem_u32(smem + L::oW), L::kWSlab);
            int kt = 0, wloads = 0;
            long wprev = -1;
            for (long t = t0; t < t1; ++t, ++kt) {
                const long wi = (t / g.tiles_per_unit) % g.weight_units;
                if (wi != wprev) {
                    mbar_wait(wfull, wloads & 1, ab);
                    ++wloads;
                    wprev = wi;
                }
                const int s = kt % kStages, b = kt & 1;
                if (kt >= 2) mbar_wait(&accempty[b], ((kt / 2) - 1) & 1, ab);
                mbar_wait(&afull[s], (kt / kStages) & 1, ab);
                tcgen05_fence_after();
                const uint32_t sA = smem_u32(smem + L::oA + s * L::kATile);
#pragma unroll
                for (int ks = 0; ks < HD / 16; ++ks)
                    mma_ss_lo(tm + b * HD, desc_lo_kmajor(sA + (ks / 4) * L::kASlab + (ks % 4) * 32), bW + ks * (2048 >> 4),
                              idesc, ks > 0);
                mma_commit(&aempty[s]);
                mma_commit(&accfull[b]);
                if (t + 1 < t1 && ((t + 1) / g.tiles_per_unit) % g.weight_units != wi) mma_commit(wfree);
            }
        }
    } else {
        const int row = warp * 32 + lane;
        const uint32_t lane_addr = (uint32_t)(warp * 32) << 16;
        int kt = 0;
        for (long t = t0; t < t1; ++t, ++kt) {
            const int b = kt & 1;
            const int unit = (int)(t / g.tiles_per_unit), r0 = (int)(t % g.tiles_per_unit) * 128;
            uint8_t *stage = smem + L::oOut + b * L::kATile;
            mbar_wait(&accfull[b], (kt / 2) & 1, ab);
            tcgen05_fence_after();
            if (tid == 0) asm volatile("cp.async.bulk.wait_group.read 1;" ::: "memory");   // the store two tiles back has read `stage`
            asm volatile("bar.sync 1, 128;" ::: "memory");
#pragma unroll 1
            for (int c = 0; c < HD; c += 32) {
                uint32_t v[32];
                tmem_ld32(tm + lane_addr + b * HD + c, v);
                tmem_wait_ld();
                uint8_t *slab = stage + (c / 64) * L::kASlab;
#pragma unroll
                for (int e = 0; e < 32; e += 8)
                    *reinterpret_cast<uint4 *>(slab + sw128_offset(row, (c % 64) + e)) = make_uint4(
                        pack_bf16(__uint_as_float(v[e]), __uint_as_float(v[e + 1])),
                        pack_bf16(__uint_as_float(v[e + 2]), __uint_as_float(v[e + 3])),
                        pack_bf16(__uint_as_float(v[e + 4]), __uint_as_float(v[e + 5])),
                        pack_bf16(__uint_as_float(v[e + 6]), __uint_as_float(v[e + 7])));
            }
            tcgen05_fence_before();
            mbar_arrive(&accempty[b]);
            fence_proxy_async_smem();
            asm volatile("bar.sync 1, 128;" ::: "memory");
            if (tid == 0 && !*abort_flag) {
#pragma unroll
                for (int sl = 0; sl < HD / 64; ++sl) tma_store_3d(&mOut, stage + sl * L::kASlab, sl * 64, r0, unit);
                tma_store_commit();
            }
        }
        if (tid == 0) tma_store_wait_all();
    }
    tcgen05_fence_before();
    __syncthreads();
    if (warp == 0) tmem_dealloc(tm, kTmemCols);
}

// ===================================================================== g += A^T G (bf16 in, fp32 out)
// Persistent: CTA c takes a contiguous range of the (unit, row tile) list, accumulates the
// d x d product of consecutive tiles that belong to the same weight matrix in tensor
// memory, and adds the block to g with fp32 reductions when the weight index changes or
// its range ends.  Both operands are MN-major (the contraction runs along the rows).
template <int HD> struct GradSmem {
    static constexpr int TR = HD == 256 ? 64 : 128;          // rows per stage
    static constexpr int kStages = 3;
    static constexpr uint32_t kSlab = TR * 128;              // [TR rows][64 bf16]
    static constexpr uint32_t kTile = (HD / 64) * kSlab;     // one operand of one stage
    static constexpr uint32_t kStage = 2 * kTile;
    static constexpr uint32_t oZero = kStages * kStage;      // d = 64: an all-zero slab, the upper half of M = 128
    static constexpr uint32_t oBar = oZero + (HD == 64 ? kSlab : 0);
    static constexpr uint32_t oMisc = oBar + 128;
    static constexpr uint32_t kBytes = oMisc + 64;
    static_assert(kBytes <= 227 * 1024, "shared memory budget");
};

struct GradArgs {
    float *g;
    uint32_t *status;
    int n, tiles_per_unit;
    long total_tiles, weight_units;
};

constexpr int kGradThreads = 192;

template <int HD>
__global__ void __launch_bounds__(kGradThreads)
wgrad_kernel(const __grid_constant__ CUtensorMap mA, const __grid_constant__ CUtensorMap mG, const GradArgs g)
{
    using L = GradSmem<HD>;
    constexpr int TR = L::TR, kStages = L::kStages;
    extern __shared__ __align__(1024) uint8_t smem[];
    uint64_t *full = reinterpret_cast<uint64_t *>(smem + L::oBar);
    uint64_t *empty = full + kStages;
    uint64_t *done = empty + kStages;
    uint64_t *tfree = done + 1;
    uint32_t *tmem_base_s = reinterpret_cast<uint32_t *>(smem + L::oMisc);
    volatile uint32_t *abort_flag = reinterpret_cast<volatile uint32_t *>(smem + L::oMisc + 4);
    const Abort ab{abort_flag, g.status};
    constexpr uint32_t kTmemCols = HD == 256 ? 512 : HD;

    const int tid = threadIdx.x, warp = tid / 32, lane = tid % 32;
    const long t0 = g.total_tiles * blockIdx.x / gridDim.x, t1 = g.total_tiles * (blockIdx.x + 1) / gridDim.x;

    if ((smem_u32(smem) & 1023u) != 0) {
        if (tid == 0) atomicExch(g.status, 9u);
        return;
    }
    auto load_stage = [&](int kt, long t) {
        const int s = kt % kStages;
        const int unit = (int)(t / g.tiles_per_unit), r0 = (int)(t % g.tiles_per_unit) * TR;
        uint8_t *sA = smem + s * L::kStage, *sG = sA + L::kTile;
        mbar_expect_tx(&full[s], L::kStage);
#pragma unroll
        for (int sl = 0; sl < HD / 64; ++sl) {
            tma_load_3d(sA + sl * L::kSlab, &mA, &full[s], sl * 64, r0, unit);
            tma_load_3d(sG + sl * L::kSlab, &mG, &full[s], sl * 64, r0, unit);
        }
    };
    const int early = (int)((t1 - t0) < kStages ? (t1 - t0) : kStages);
    if (tid == 0) {
        *abort_flag = 0;
        mbar_init(done, 1);
        mbar_init(tfree, 128);
        fence_barrier_init();
    }
    if (tid == 4 * 32) {
        // the producer sets up its own ring and fills it before the CTA-wide setup is over
        for (int s = 0; s < kStages; ++s) { mbar_init(&full[s], 1); mbar_init(&empty[s], 1); }
        fence_barrier_init();
        for (int kt = 0; kt < early; ++kt) load_stage(kt, t0 + kt);
    }
    if (HD == 64) {
        for (uint32_t i = tid; i < L::kSlab / 16; i += kGradThreads)
            reinterpret_cast<uint4 *>(smem + L::oZero)[i] = make_uint4(0, 0, 0, 0);
        fence_proxy_async_smem();
    }
    if (warp == 0) tmem_alloc(tmem_base_s, kTmemCols);
    tcgen05_fence_before();
    __syncthreads();
    tcgen05_fence_after();
    const uint32_t tm = *tmem_base_s;

    if (warp == 4) {
        if (lane == 0) {
            int kt = early;
            for (long t = t0 + early; t < t1; ++t, ++kt) {
                mbar_wait(&empty[kt % kStages], ((kt / kStages) - 1) & 1, ab);
                load_stage(kt, t);
            }
        }
    } else if (warp == 5) {
        if (lane == 0) {
            constexpr uint32_t idesc = idesc_bf16(128, HD, 1, 1);
            int kt = 0, flushes = 0;
            bool fresh = true;
            for (long t = t0; t < t1; ++t, ++kt) {
                const int s = kt % kStages;
                if (fresh && flushes > 0) {            // the previous block must have left tensor memory
                    mbar_wait(tfree, (flushes - 1) & 1, ab);
                    tcgen05_fence_after();
                }
                mbar_wait(&full[s], (kt / kStages) & 1, ab);
                tcgen05_fence_after();
                const uint32_t sA = smem_u32(smem + s * L::kStage), sG = sA + L::kTile;
                const uint32_t lboA = HD == 64 ? smem_u32(smem + L::oZero) - sA : L::kSlab;
                const uint32_t bG = desc_lo_mnmajor(sG, L::kSlab);
#pragma unroll
                for (int ks = 0; ks < TR / 16; ++ks) {
                    const uint32_t acc = (!fresh || ks > 0) ? 1u : 0u;
                    mma_ss_lo(tm, desc_lo_mnmajor(sA + ks * 2048, lboA), bG + ks * (2048 >> 4), idesc, acc);
                    if (HD == 256)
                        mma_ss_lo(tm + 256, desc_lo_mnmajor(sA + 2 * L::kSlab + ks * 2048, lboA), bG + ks * (2048 >> 4),
                                  idesc, acc);
                }
                mma_commit(&empty[s]);
                fresh = false;
                const long w = (t / g.tiles_per_unit) % g.weight_units;
                if (t + 1 == t1 || ((t + 1) / g.tiles_per_unit) % g.weight_units != w) {
                    mma_commit(done);
                    ++flushes;
                    fresh = true;
                }
            }
        }
    } else {
        int flushes = 0;
        const uint32_t lane_addr = (uint32_t)(warp * 32) << 16;
        const int row = warp * 32 + lane;
        for (long t = t0; t < t1; ++t) {
            const long w = (t / g.tiles_per_unit) % g.weight_units;
            if (!(t + 1 == t1 || ((t + 1) / g.tiles_per_unit) % g.weight_units != w)) continue;
            mbar_wait(done, flushes & 1, ab);
            tcgen05_fence_after();
            float *gw = g.g + (size_t)w * HD * HD;
            if (HD != 64 || warp < 2) {
#pragma unroll 1
                for (int half = 0; half < (HD == 256 ? 2 : 1); ++half) {
                    float *grow = gw + (size_t)(half * 128 + row) * HD;
#pragma unroll 1
                    for (int c = 0; c < HD; c += 32) {
                        uint32_t v[32];
                        tmem_ld32(tm + lane_addr + half * 256 + c, v);
                        tmem_wait_ld();
                        if (*abort_flag) continue;
#pragma unroll
                        for (int e = 0; e < 32; e += 4)
                            red_add_v4(grow + c + e, __uint_as_float(v[e]), __uint_as_float(v[e + 1]),
                                       __uint_as_float(v[e + 2]), __uint_as_float(v[e + 3]));
                    }
                }
            }
            tcgen05_fence_before();
            mbar_arrive(tfree);
            ++flushes;
        }
    }
    tcgen05_fence_before();
    __syncthreads();
    if (warp == 0) tmem_dealloc(tm, kTmemCols);
}

// ===================================================================== g += A^T G with G in fp32
// The same product for a G that sits in device memory as fp32 -- the dQ accumulator of the fused backward, so that
// the closing product of phase 2 (Appendix D) reads it directly: no bf16 copy of dQ is written and read back, and dQ
// is rounded once, on its way into the product.  Per stage the loading thread brings a bf16 tile of A and the fp32
// tile of G; warps 0-3 turn the latter into the bf16 MN-major operand (two buffers) and later add finished d x d
// blocks to g; the issuing thread runs the products.  A stage is free again when its product has completed and all
// four converting warps have read it (five arrivals).
template <int HD> struct GradAccSmem {
    static constexpr int TR = 8192 / HD;                     // rows per stage: 48 KB a stage at every head size
    static constexpr int kStages = 3;
    static constexpr uint32_t kSlab = TR * 128;              // [TR rows][128 bytes]: 64 bf16 or 32 fp32 a row
    static constexpr uint32_t kATile = (HD / 64) * kSlab;    // bf16 tile (A, and G after conversion)
    static constexpr uint32_t kGfTile = (HD / 32) * kSlab;   // fp32 tile of G
    static constexpr uint32_t kStage = kATile + kGfTile;
    static constexpr uint32_t oGb = kStages * kStage;        // two converted tiles
    static constexpr uint32_t oZero = oGb + 2 * kATile;      // d = 64: an all-zero slab, the upper half of M = 128
    static constexpr uint32_t oBar = oZero + (HD == 64 ? kSlab : 0);
    static constexpr uint32_t oMisc = oBar + 128;
    static constexpr uint32_t kBytes = oMisc + 64;
    static_assert(kBytes <= 227 * 1024, "shared memory budget");
};

template <int HD>
__global__ void __launch_bounds__(kGradThreads)
wgrad_acc_kernel(const __grid_constant__ CUtensorMap mA, const __grid_constant__ CUtensorMap mG, const GradArgs g)
{
    using L = GradAccSmem<HD>;
    constexpr int TR = L::TR, kStages = L::kStages;
    extern __shared__ __align__(1024) uint8_t smem[];
    uint64_t *full = reinterpret_cast<uint64_t *>(smem + L::oBar);
    uint64_t *empty = full + kStages;       // 1 (the product) + 4 (the converting warps)
    uint64_t *gbfull = empty + kStages;     // [2] converted tile written, 4 arrivals
    uint64_t *gbfree = gbfull + 2;          // [2] its product has completed
    uint64_t *done = gbfree + 2;
    uint64_t *tfree = done + 1;
    uint32_t *tmem_base_s = reinterpret_cast<uint32_t *>(smem + L::oMisc);
    volatile uint32_t *abort_flag = reinterpret_cast<volatile uint32_t *>(smem + L::oMisc + 4);
    const Abort ab{abort_flag, g.status};
    constexpr uint32_t kTmemCols = HD == 256 ? 512 : HD;   // d = 256: two accumulators of 128 rows x 256 columns

    const int tid = threadIdx.x, warp = tid / 32, lane = tid % 32;
    const long t0 = g.total_tiles * blockIdx.x / gridDim.x, t1 = g.total_tiles * (blockIdx.x + 1) / gridDim.x;

    if ((smem_u32(smem) & 1023u) != 0) {
        if (tid == 0) atomicExch(g.status, 9u);
        return;
    }
    auto load_stage = [&](int kt, long t) {
        const int s = kt % kStages;
        const int unit = (int)(t / g.tiles_per_unit), r0 = (int)(t % g.tiles_per_unit) * TR;
        uint8_t *sA = smem + s * L::kStage, *sGf = sA + L::kATile;
        mbar_expect_tx(&full[s], L::kStage);
#pragma unroll
        for (int sl = 0; sl < HD / 64; ++sl) tma_load_3d(sA + sl * L::kSlab, &mA, &full[s], sl * 64, r0, unit);
#pragma unroll
        for (int sl = 0; sl < HD / 32; ++sl) tma_load_3d(sGf + sl * L::kSlab, &mG, &full[s], sl * 32, r0, unit);
    };
    const int early = (int)((t1 - t0) < kStages ? (t1 - t0) : kStages);
    if (tid == 0) {
        *abort_flag = 0;
        for (int b = 0; b < 2; ++b) { mbar_init(&gbfull[b], 4); mbar_init(&gbfree[b], 1); }
        mbar_init(done, 1);
        mbar_init(tfree, 128);
        fence_barrier_init();
    }
    if (tid == 4 * 32) {
        // the loading thread sets up its own ring and fills it before the CTA-wide setup is over
        for (int s = 0; s < kStages; ++s) { mbar_init(&full[s], 1); mbar_init(&empty[s], 5); }
        fence_barrier_init();
        for (int kt = 0; kt < early; ++kt) load_stage(kt, t0 + kt);
    }
    if (HD == 64) {
        for (uint32_t i = tid; i < L::kSlab / 16; i += kGradThreads)
            reinterpret_cast<uint4 *>(smem + L::oZero)[i] = make_uint4(0, 0, 0, 0);
        fence_proxy_async_smem();
    }
    if (warp == 0) tmem_alloc(tmem_base_s, kTmemCols);
    tcgen05_fence_before();
    __syncthreads();
    tcgen05_fence_after();
    const uint32_t tm = *tmem_base_s;

    if (warp == 4) {
        if (lane == 0) {
            int kt = early;
            for (long t = t0 + early; t < t1; ++t, ++kt) {
                mbar_wait(&empty[kt % kStages], ((kt / kStages) - 1) & 1, ab);
                load_stage(kt, t);
            }
        }
    } else if (warp == 5) {
        if (lane == 0) {
            constexpr uint32_t idesc = idesc_bf16(128, HD, 1, 1);
            int kt = 0, flushes = 0;
            bool fresh = true;
            for (long t = t0; t < t1; ++t, ++kt) {
                const int s = kt % kStages, cb = kt & 1;
                if (fresh && flushes > 0) {            // the previous block must have left tensor memory
                    mbar_wait(tfree, (flushes - 1) & 1, ab);
                    tcgen05_fence_after();
                }
                mbar_wait(&full[s], (kt / kStages) & 1, ab);
                mbar_wait(&gbfull[cb], (kt >> 1) & 1, ab);
                tcgen05_fence_after();
                const uint32_t sA = smem_u32(smem + s * L::kStage), sG = smem_u32(smem + L::oGb + cb * L::kATile);
                const uint32_t lboA = HD == 64 ? smem_u32(smem + L::oZero) - sA : L::kSlab;
                const uint32_t bG = desc_lo_mnmajor(sG, L::kSlab);
#pragma unroll
                for (int ks = 0; ks < TR / 16; ++ks) {
                    const uint32_t acc = (!fresh || ks > 0) ? 1u : 0u;
                    mma_ss_lo(tm, desc_lo_mnmajor(sA + ks * 2048, lboA), bG + ks * (2048 >> 4), idesc, acc);
                    if (HD == 256)
                        mma_ss_lo(tm + 256, desc_lo_mnmajor(sA + 2 * L::kSlab + ks * 2048, lboA), bG + ks * (2048 >> 4),
                                  idesc, acc);
                }
                mma_commit(&empty[s]);
                mma_commit(&gbfree[cb]);
                fresh = false;
                const long w = (t / g.tiles_per_unit) % g.weight_units;
                if (t + 1 == t1 || ((t + 1) / g.tiles_per_unit) % g.weight_units != w) {
                    mma_commit(done);
                    ++flushes;
                    fresh = true;
                }
            }
        }
    } else {
        // converting warps: thread -> (row, column range) of the stage's tile; a 16-byte chunk of the swizzled fp32 slab
        // holds 4 columns, of the bf16 slab 8
        constexpr int kColsPerThread = HD * TR / 128;
        const int row = tid % TR, col0 = (tid / TR) * kColsPerThread;
        const uint32_t lane_addr = (uint32_t)(warp * 32) << 16;
        const int grow = warp * 32 + lane;    // row of the d x d block this thread adds to g
        int flushes = 0, kt = 0;
        for (long t = t0; t < t1; ++t, ++kt) {
            const int s = kt % kStages, cb = kt & 1;
            mbar_wait(&full[s], (kt / kStages) & 1, ab);
            if (kt >= 2) mbar_wait(&gbfree[cb], ((kt >> 1) - 1) & 1, ab);
            const uint8_t *sGf = smem + s * L::kStage + L::kATile;
            uint8_t *sGb = smem + L::oGb + cb * L::kATile;
#pragma unroll
            for (int j = 0; j < kColsPerThread; j += 8) {
                const uint32_t c = col0 + j, cc = c % 32;
                const uint8_t *src = sGf + (c / 32) * L::kSlab + row * 128;
                const float4 lo = *reinterpret_cast<const float4 *>(src + ((((cc >> 2)) ^ (row & 7)) << 4));
                const float4 hi = *reinterpret_cast<const float4 *>(src + ((((cc >> 2) + 1) ^ (row & 7)) << 4));
                *reinterpret_cast<uint4 *>(sGb + (c / 64) * L::kSlab + sw128_offset(row, c % 64)) =
                    make_uint4(pack_bf16(lo.x, lo.y), pack_bf16(lo.z, lo.w), pack_bf16(hi.x, hi.y), pack_bf16(hi.z, hi.w));
            }
            fence_proxy_async_smem();
            __syncwarp();
            if (lane == 0) {
                mbar_arrive(&gbfull[cb]);
                mbar_arrive(&empty[s]);
            }
            const long w = (t / g.tiles_per_unit) % g.weight_units;
            if (!(t + 1 == t1 || ((t + 1) / g.tiles_per_unit) % g.weight_units != w)) continue;
            // the last tile of a weight's block: add the block to g
            mbar_wait(done, flushes & 1, ab);
            tcgen05_fence_after();
            if (HD != 64 || warp < 2) {
#pragma unroll 1
                for (int half = 0; half < (HD == 256 ? 2 : 1); ++half) {
                    float *grow_p = g.g + (size_t)w * HD * HD + (size_t)(half * 128 + grow) * HD;
#pragma unroll 1
                    for (int c = 0; c < HD; c += 32) {
                        uint32_t v[32];
                        tmem_ld32(tm + lane_addr + half * 256 + c, v);
                        tmem_wait_ld();
                        if (*abort_flag) continue;
#pragma unroll
                        for (int e = 0; e < 32; e += 4)
                            red_add_v4(grow_p + c + e, __uint_as_float(v[e]), __uint_as_float(v[e + 1]),
                                       __uint_as_float(v[e + 2]), __uint_as_float(v[e + 3]));
                    }
                }
            }
            tcgen05_fence_before();
            mbar_arrive(tfree);
            ++flushes;
        }
    }
    tcgen05_fence_before();
    __syncthreads();
    if (warp == 0) tmem_dealloc(tm, kTmemCols);
}

// ===================================================================== fp32 FMA kernels (any dtype, d % 8 == 0)
template <typename T> __device__ __forceinline__ float to_f(T v);
template <> __device__ __forceinline__ float to_f<float>(float v) { return v; }
template <> __device__ __forceinline__ float to_f<__nv_bfloat16>(__nv_bfloat16 v) { return __bfloat162float(v); }
template <typename T> __device__ __forceinline__ T from_f(float v);
template <> __device__ __forceinline__ float from_f<float>(float v) { return v; }
template <> __device__ __forceinline__ __nv_bfloat16 from_f<__nv_bfloat16>(float v) { return __float2bfloat16_rn(v); }

template <typename T>
__global__ void __launch_bounds__(256) simt_project_kernel(const T *__restrict__ A, const T *__restrict__ W,
                                                           T *__restrict__ out, size_t total, int n, int d, long weight_units)
{
    for (size_t idx = (size_t)blockIdx.x * blockDim.x + threadIdx.x; idx < total; idx += (size_t)gridDim.x * blockDim.x) {
        const size_t row = idx / d;
        const int c = (int)(idx % d);
        const T *a = A + row * d;
        const T *w = W + (size_t)((row / n) % weight_units) * d * d + c;
        float acc = 0.f;
        for (int k = 0; k < d; ++k) acc = fmaf(to_f(a[k]), to_f(w[(size_t)k * d]), acc);
        out[idx] = from_f<T>(acc);
    }
}

// grid (row chunks, units): every thread owns entries (a, b) of the d x d block and sums its chunk of rows
template <typename T>
__global__ void __launch_bounds__(256) simt_wgrad_kernel(const T *__restrict__ A, const T *__restrict__ G,
                                                         float *__restrict__ g, int n, int d, long weight_units, int rows_per_block)
{
    const long unit = blockIdx.y;
    const int r0 = blockIdx.x * rows_per_block, r1 = min(n, r0 + rows_per_block);
    const T *a = A + (size_t)unit * n * d, *gg = G + (size_t)unit * n * d;
    float *out = g + (size_t)(unit % weight_units) * d * d;
    for (int idx = threadIdx.x; idx < d * d; idx += blockDim.x) {
        const int ia = idx / d, ib = idx % d;
        float acc = 0.f;
        for (int i = r0; i < r1; ++i) acc = fmaf(to_f(a[(size_t)i * d + ia]), to_f(gg[(size_t)i * d + ib]), acc);
        atomicAdd(out + idx, acc);
    }
}

bool aligned16(const void *p) { return ((uintptr_t)p & 15) == 0; }

attn_status check_arch()
{
    int dev = 0, major = 0;
    if (cudaGetDevice(&dev) != cudaSuccess) return ATTN_ERR_ARCH;
    if (cudaDeviceGetAttribute(&major, cudaDevAttrComputeCapabilityMajor, dev) != cudaSuccess) return ATTN_ERR_ARCH;
    return major == 10 ? ATTN_OK : ATTN_ERR_ARCH;
}

attn_status check_common(int n, int d, int heads, int batch, int weight_units, int dt, const void *workspace,
                         size_t workspace_bytes)
{
    if (n <= 0 || heads <= 0 || batch <= 0 || d < 8 || d > 256 || d % 8 != 0) return ATTN_ERR_SHAPE;
    if ((double)n * d * heads * batch > 4.0e12 || (long)heads * batch > 0x7fffffffL) return ATTN_ERR_SHAPE;
    if (weight_units != 1 && weight_units != heads && (long)weight_units != (long)heads * batch) return ATTN_ERR_SHAPE;
    if (dt != ATTN_F32 && dt != ATTN_BF16) return ATTN_ERR_DTYPE;
    if (!workspace || workspace_bytes < kStatusBytes) return ATTN_ERR_WORKSPACE;
    if ((uintptr_t)workspace & 255) return ATTN_ERR_ALIGN;
    return ATTN_OK;
}

bool use_tc(int d, int dt) { return dt == ATTN_BF16 && (d == 64 || d == 128 || d == 256); }

template <int HD>
attn_status launch_project(const void *A, const void *W, void *out, int n, long BH, long wu, uint32_t *status, cudaStream_t s)
{
    using L = ProjSmem<HD>;
    if (BH > 65535) return ATTN_ERR_SHAPE;
    CUtensorMap mA, mW;
    if (!make_tmap_bf16_3d(&mA, A, HD, (uint64_t)n, (uint64_t)BH, 128) ||
        !make_tmap_bf16_3d(&mW, W, HD, HD, (uint64_t)wu, HD))
        return ATTN_ERR_LAUNCH;
    if (cudaFuncSetAttribute(wproj_kernel<HD>, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)L::kBytes) != cudaSuccess)
        return ATTN_ERR_LAUNCH;
    const ProjArgs a{(__nv_bfloat16 *)out, status, n, wu};
    const dim3 grid((unsigned)((n + 127) / 128), (unsigned)BH);
    launch_begin("wproj", s);
    wproj_kernel<HD><<<grid, kProjThreads, L::kBytes, s>>>(mA, mW, a);
    launch_end(s);
    return cudaGetLastError() == cudaSuccess ? ATTN_OK : ATTN_ERR_LAUNCH;
}

template <int HD>
attn_status launch_project_persistent(const void *A, const void *W, void *out, int n, long BH, long wu, uint32_t *status,
                                      cudaStream_t s)
{
    using L = ProjPSmem<HD>;
    CUtensorMap mA, mW, mOut;
    if (!make_tmap_bf16_3d(&mA, A, HD, (uint64_t)n, (uint64_t)BH, 128) ||
        !make_tmap_bf16_3d(&mW, W, HD, HD, (uint64_t)wu, HD) ||
        !make_tmap_bf16_3d(&mOut, out, HD, (uint64_t)n, (uint64_t)BH, 128))
        return ATTN_ERR_LAUNCH;
    if (cudaFuncSetAttribute(wproj_persistent_kernel<HD>, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)L::kBytes) !=
        cudaSuccess)
        return ATTN_ERR_LAUNCH;
    ProjPArgs a{};
    a.status = status;
    a.tiles_per_unit = (n + 127) / 128;
    a.total_tiles = (long)a.tiles_per_unit * BH;
    a.weight_units = wu;
    const long ctas = (long)sm_count() * (HD == 64 ? 2 : 1);
    const unsigned grid = (unsigned)(a.total_tiles < ctas ? a.total_tiles : ctas);
    launch_begin("wproj", s);
    wproj_persistent_kernel<HD><<<grid, kProjThreads, L::kBytes, s>>>(mA, mW, mOut, a);
    launch_end(s);
    return cudaGetLastError() == cudaSuccess ? ATTN_OK : ATTN_ERR_LAUNCH;
}

template <int HD>
attn_status launch_grad(const void *A, const void *G, float *g, int n, long BH, long wu, uint32_t *status, cudaStream_t s)
{
    using L = GradSmem<HD>;
    CUtensorMap mA, mG;
    if (!make_tmap_bf16_3d(&mA, A, HD, (uint64_t)n, (uint64_t)BH, L::TR) ||
        !make_tmap_bf16_3d(&mG, G, HD, (uint64_t)n, (uint64_t)BH, L::TR))
        return ATTN_ERR_LAUNCH;
    if (cudaFuncSetAttribute(wgrad_kernel<HD>, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)L::kBytes) != cudaSuccess)
        return ATTN_ERR_LAUNCH;
    GradArgs a{};
    a.g = g; a.status = status; a.n = n;
    a.tiles_per_unit = (n + L::TR - 1) / L::TR;
    a.total_tiles = (long)a.tiles_per_unit * BH;
    a.weight_units = wu;
    const long sms = sm_count();
    const unsigned grid = (unsigned)(a.total_tiles < sms ? a.total_tiles : sms);
    launch_begin("wgrad", s);
    wgrad_kernel<HD><<<grid, kGradThreads, L::kBytes, s>>>(mA, mG, a);
    launch_end(s);
    return cudaGetLastError() == cudaSuccess ? ATTN_OK : ATTN_ERR_LAUNCH;
}

template <int HD>
attn_status launch_grad_acc(const void *A, const float *G, float *g, int n, long BH, long wu, uint32_t *status, cudaStream_t s)
{
    using L = GradAccSmem<HD>;
    CUtensorMap mA, mG;
    if (!make_tmap_bf16_3d(&mA, A, HD, (uint64_t)n, (uint64_t)BH, L::TR) ||
        !make_tmap_f32_3d(&mG, G, HD, (uint64_t)n, (uint64_t)BH, L::TR))
        return ATTN_ERR_LAUNCH;
    if (cudaFuncSetAttribute(wgrad_acc_kernel<HD>, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)L::kBytes) != cudaSuccess)
        return ATTN_ERR_LAUNCH;
    if (cudaMemsetAsync(g, 0, (size_t)wu * HD * HD * sizeof(float), s) != cudaSuccess) return ATTN_ERR_LAUNCH;
    GradArgs a{};
    a.g = g; a.status = status; a.n = n;
    a.tiles_per_unit = (n + L::TR - 1) / L::TR;
    a.total_tiles = (long)a.tiles_per_unit * BH;
    a.weight_units = wu;
    const long sms = sm_count();
    const unsigned grid = (unsigned)(a.total_tiles < sms ? a.total_tiles : sms);
    launch_begin("wgrad_acc", s);
    wgrad_acc_kernel<HD><<<grid, kGradThreads, L::kBytes, s>>>(mA, mG, a);
    launch_end(s);
    return cudaGetLastError() == cudaSuccess ? ATTN_OK : ATTN_ERR_LAUNCH;
}

template <typename T>
attn_status launch_simt_project(const void *A, const void *W, void *out, int n, int d, long BH, long wu, cudaStream_t s)
{
    const size_t total = (size_t)BH * n * d;
    size_t blocks = (total + 255) / 256;
    if (blocks > (size_t)sm_count() * 16) blocks = (size_t)sm_count() * 16;
    launch_begin("wproj_simt", s);
    simt_project_kernel<T><<<(unsigned)blocks, 256, 0, s>>>((const T *)A, (const T *)W, (T *)out, total, n, d, wu);
    launch_end(s);
    return cudaGetLastError() == cudaSuccess ? ATTN_OK : ATTN_ERR_LAUNCH;
}

template <typename T>
attn_status launch_simt_grad(const void *A, const void *G, float *g, int n, int d, long BH, long wu, cudaStream_t s)
{
    const int rows_per_block = 64;
    if (BH > 65535) return ATTN_ERR_SHAPE;
    const dim3 grid((unsigned)((n + rows_per_block - 1) / rows_per_block), (unsigned)BH);
    launch_begin("wgrad_simt", s);
    simt_wgrad_kernel<T><<<grid, 256, 0, s>>>((const T *)A, (const T *)G, g, n, d, wu, rows_per_block);
    launch_end(s);
    return cudaGetLastError() == cudaSuccess ? ATTN_OK : ATTN_ERR_LAUNCH;
}

attn_status project_impl(const void *A, const void *W, void *out, int n, int d, long BH, long wu, int dt, uint32_t *status,
                         cudaStream_t s)
{
    if (use_tc(d, dt)) {
        if (d == 64) return launch_project_persistent<64>(A, W, out, n, BH, wu, status, s);
        if (d == 128) return launch_project_persistent<128>(A, W, out, n, BH, wu, status, s);
        return launch_project<256>(A, W, out, n, BH, wu, status, s);   // W alone takes 128 KB: one tile per CTA
    }
    if (dt == ATTN_F32) return launch_simt_project<float>(A, W, out, n, d, BH, wu, s);
    return launch_simt_project<__nv_bfloat16>(A, W, out, n, d, BH, wu, s);
}

attn_status grad_impl(const void *A, const void *G, float *g, int n, int d, long BH, long wu, int dt, uint32_t *status,
                      cudaStream_t s)
{
    if (cudaMemsetAsync(g, 0, (size_t)wu * d * d * sizeof(float), s) != cudaSuccess) return ATTN_ERR_LAUNCH;
    if (use_tc(d, dt)) {
        if (d == 64) return launch_grad<64>(A, G, g, n, BH, wu, status, s);
        if (d == 128) return launch_grad<128>(A, G, g, n, BH, wu, status, s);
        return launch_grad<256>(A, G, g, n, BH, wu, status, s);
    }
    if (dt == ATTN_F32) return launch_simt_grad<float>(A, G, g, n, d, BH, wu, s);
    return launch_simt_grad<__nv_bfloat16>(A, G, g, n, d, BH, wu, s);
}

}  // namespace
}  // namespace attn

using namespace attn;

extern "C" {

attn_status attn_project(const void *A, const void *W, void *out, int n, int d, int heads, int batch, int weight_units,
                         int dt, void *workspace, size_t workspace_bytes, void *cuda_stream)
{
    if (!A || !W || !out) return ATTN_ERR_NULL;
    attn_status st = check_common(n, d, heads, batch, weight_units, dt, workspace, workspace_bytes);
    if (st != ATTN_OK) return st;
    if (!aligned16(A) || !aligned16(W) || !aligned16(out)) return ATTN_ERR_ALIGN;
    if ((st = check_arch()) != ATTN_OK) return st;
    cudaStream_t s = (cudaStream_t)cuda_stream;
    if (cudaMemsetAsync(workspace, 0, 4, s) != cudaSuccess) return ATTN_ERR_LAUNCH;
    return project_impl(A, W, out, n, d, (long)heads * batch, weight_units, dt, (uint32_t *)workspace, s);
}

attn_status attn_weight_grad(const void *A, const void *G, float *g, int n, int d, int heads, int batch, int weight_units,
                             int dt, void *workspace, size_t workspace_bytes, void *cuda_stream)
{
    if (!A || !G || !g) return ATTN_ERR_NULL;
    attn_status st = check_common(n, d, heads, batch, weight_units, dt, workspace, workspace_bytes);
    if (st != ATTN_OK) return st;
    if (!aligned16(A) || !aligned16(G) || !aligned16(g)) return ATTN_ERR_ALIGN;
    if ((st = check_arch()) != ATTN_OK) return st;
    cudaStream_t s = (cudaStream_t)cuda_stream;
    if (cudaMemsetAsync(workspace, 0, 4, s) != cudaSuccess) return ATTN_ERR_LAUNCH;
    return grad_impl(A, G, g, n, d, (long)heads * batch, weight_units, dt, (uint32_t *)workspace, s);
}

size_t attn_weights_bwd_workspace_bytes(int n, int d, int heads, int batch, const attn_mask *mask, int dt,
                                        const attn_cfg *cfg)
{
    const size_t inner = attn_bwd_workspace_bytes(n, d, heads, batch, mask, dt, cfg);
    if (inner == 0) return 0;
    const size_t tensor = align_up((size_t)n * d * heads * batch * (dt == ATTN_F32 ? 4 : 2), 256);
    return align_up(inner, 256) + 3 * tensor;
}

attn_status attn_weights_bwd(const void *A1, const void *A2, const void *A3, const void *S, const void *h, const void *O,
                             const void *dO, const float *LSE, float *gX, float *gY, int n, int d, int heads, int batch,
                             int weight_units, const attn_mask *mask, int dt, float scale, const attn_cfg *cfg,
                             void *workspace, size_t workspace_bytes, void *cuda_stream)
{
    if (!A1 || !A2 || !S || !h || !O || !dO || !LSE || !gX) return ATTN_ERR_NULL;
    if (gY && !A3) return ATTN_ERR_NULL;
    attn_status st = check_common(n, d, heads, batch, weight_units, dt, workspace, workspace_bytes);
    if (st != ATTN_OK) return st;
    const size_t inner = attn_bwd_workspace_bytes(n, d, heads, batch, mask, dt, cfg);
    if (inner == 0) return ATTN_ERR_TILE;
    const size_t tensor = align_up((size_t)n * d * heads * batch * (dt == ATTN_F32 ? 4 : 2), 256);
    if (workspace_bytes < align_up(inner, 256) + 3 * tensor) return ATTN_ERR_WORKSPACE;
    if (!aligned16(A1) || (A3 && !aligned16(A3)) || !aligned16(gX) || (gY && !aligned16(gY))) return ATTN_ERR_ALIGN;
    uint8_t *base = (uint8_t *)workspace;
    void *dS = base + align_up(inner, 256), *dK = (uint8_t *)dS + tensor, *dh = (uint8_t *)dK + tensor;
    // gradients of S = A1 X (p A2, times the scale), of A2 and of h = A3 Y (f^T dO)
    // where the backward leaves dS (the gradient of S = A1 X) in its fp32 accumulator, gX is formed from that
    const float *acc = nullptr;
    const bool from_acc = use_tc(d, dt);
    st = bwd_internal(S, A2, h, O, dO, LSE, dS, dK, dh, n, d, heads, batch, mask, dt, scale, cfg, workspace, inner,
                      cuda_stream, from_acc, &acc);
    if (st != ATTN_OK) return st;
    cudaStream_t s = (cudaStream_t)cuda_stream;
    const long BH = (long)heads * batch;
    if (acc)
        st = d == 64    ? launch_grad_acc<64>(A1, acc, gX, n, BH, weight_units, (uint32_t *)workspace, s)
             : d == 128 ? launch_grad_acc<128>(A1, acc, gX, n, BH, weight_units, (uint32_t *)workspace, s)
                        : launch_grad_acc<256>(A1, acc, gX, n, BH, weight_units, (uint32_t *)workspace, s);
    else
        st = grad_impl(A1, dS, gX, n, d, BH, weight_units, dt, (uint32_t *)workspace, s);
    if (st != ATTN_OK) return st;
    if (gY) st = grad_impl(A3, dh, gY, n, d, BH, weight_units, dt, (uint32_t *)workspace, s);
    return st;
}

}  // extern "C"

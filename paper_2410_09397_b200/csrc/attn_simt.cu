// fp32 FMA kernels for exact attention: forward, backward (dQ; dK and dV), the
// D = rowsum(dO o O) pre-pass and the block-mask index build.
//
// These kernels keep every product and sum in fp32 on the CUDA cores, which is what
// the 1e-4 tolerance of fp32 inputs needs (a single-pass tf32 tensor-core product
// does not hold it).  They accept any n, any d that is a multiple of 8 up to 256, and
// all three mask kinds, so they also serve as the general path for shapes the
// tensor-core kernels do not take.
//
// Tiling: a CTA of 256 threads owns 64 rows (queries, or keys in the dK/dV kernel)
// and walks the other sequence dimension in tiles of 64; the head dimension is walked
// in chunks of 64.  Score tiles live in shared memory only (the large-cache scheme of
// Appendix D: the n x n matrices are never written to device memory).
#include <cuda_bf16.h>
#include <math.h>

#include "attn_internal.h"

namespace attn {
namespace {

constexpr int TS = 64;        // tile edge
constexpr int LD = TS + 1;    // padded shared-memory row
constexpr int NT = 256;       // threads per CTA

template <typename T> __device__ __forceinline__ float to_f(T v);
template <> __device__ __forceinline__ float to_f<float>(float v) { return v; }
template <> __device__ __forceinline__ float to_f<__nv_bfloat16>(__nv_bfloat16 v) { return __bfloat162float(v); }
template <typename T> __device__ __forceinline__ T from_f(float v);
template <> __device__ __forceinline__ float from_f<float>(float v) { return v; }
template <> __device__ __forceinline__ __nv_bfloat16 from_f<__nv_bfloat16>(float v) { return __float2bfloat16_rn(v); }

struct MaskDev {
    int kind, block, nb;  // element mask: block = n, nb = 32-bit words per row
    const uint8_t *bits;  // already offset to this head's [nb][nb] mask (element mask: its [n][nb] bitmap)
};

__device__ __forceinline__ bool keep(const MaskDev &m, int i, int j)
{
    if (m.kind == ATTN_MASK_NONE) return true;
    if (m.kind == ATTN_MASK_CAUSAL) return j <= i;
    if (m.kind == ATTN_MASK_BLOCK_SPARSE_CAUSAL && j > i) return false;
    if (m.kind == ATTN_MASK_ELEMENT)
        return (reinterpret_cast<const uint32_t *>(m.bits)[(size_t)i * m.nb + j / 32] >> (j % 32)) & 1u;
    return m.bits[(size_t)(i / m.block) * m.nb + j / m.block] != 0;
}

// Does the tile rows [i0, i1] x cols [j0, j1] (inclusive, already clipped to n-1) keep anything?
__device__ __forceinline__ bool tile_any(const MaskDev &m, int i0, int i1, int j0, int j1)
{
    if (m.kind == ATTN_MASK_NONE) return true;
    if (m.kind == ATTN_MASK_CAUSAL) return j0 <= i1;
    if (m.kind == ATTN_MASK_BLOCK_SPARSE_CAUSAL && j0 > i1) return false;
    if (m.kind == ATTN_MASK_ELEMENT) return true;   // the fp32 kernels visit every tile of an element mask
    for (int I = i0 / m.block; I <= i1 / m.block; ++I)
        for (int J = j0 / m.block; J <= j1 / m.block; ++J)
            if (m.bits[(size_t)I * m.nb + J]) return true;
    return false;
}

__device__ __forceinline__ MaskDev head_mask(int kind, int block, int nb, const uint8_t *bits, int mask_heads, long bh)
{
    MaskDev m{kind, block, nb, bits};
    if (mask_is_block(kind) && mask_heads != 1) m.bits = bits + (size_t)bh * nb * nb;
    if (mask_is_element(kind) && mask_heads != 1) m.bits = bits + (size_t)bh * block * nb * sizeof(uint32_t);
    return m;
}

// dst[r][c] = src[(row0 + r) * d + col0 + c] for r, c < 64; zero outside n x d.
template <typename T>
__device__ __forceinline__ void load_chunk(float *dst, const T *src, int row0, int col0, int n, int d)
{
    const int c = threadIdx.x % TS, r0 = threadIdx.x / TS;
#pragma unroll
    for (int it = 0; it < TS / (NT / TS); ++it) {
        int r = r0 + it * (NT / TS);
        int gr = row0 + r, gc = col0 + c;
        dst[r * LD + c] = (gr < n && gc < d) ? to_f(src[(size_t)gr * d + gc]) : 0.f;
    }
}

// acc[r][c] += sum_k A[ty*4 + r][k] * B[tx + 16c][k]
__device__ __forceinline__ void mm_nt(float (&acc)[4][4], const float *A, const float *B, int ty, int tx)
{
#pragma unroll 8
    for (int k = 0; k < TS; ++k) {
        float a[4], b[4];
#pragma unroll
        for (int r = 0; r < 4; ++r) a[r] = A[(ty * 4 + r) * LD + k];
#pragma unroll
        for (int c = 0; c < 4; ++c) b[c] = B[(tx + 16 * c) * LD + k];
#pragma unroll
        for (int r = 0; r < 4; ++r)
#pragma unroll
            for (int c = 0; c < 4; ++c) acc[r][c] = fmaf(a[r], b[c], acc[r][c]);
    }
}

// acc[r][c] += sum_k A[ty*4 + r][k] * B[k][tx + 16c]
__device__ __forceinline__ void mm_nn(float (&acc)[4][4], const float *A, const float *B, int ty, int tx)
{
#pragma unroll 8
    for (int k = 0; k < TS; ++k) {
        float a[4], b[4];
#pragma unroll
        for (int r = 0; r < 4; ++r) a[r] = A[(ty * 4 + r) * LD + k];
#pragma unroll
        for (int c = 0; c < 4; ++c) b[c] = B[k * LD + tx + 16 * c];
#pragma unroll
        for (int r = 0; r < 4; ++r)
#pragma unroll
            for (int c = 0; c < 4; ++c) acc[r][c] = fmaf(a[r], b[c], acc[r][c]);
    }
}

// acc[r][c] += sum_k A[k][ty*4 + r] * B[k][tx + 16c]
__device__ __forceinline__ void mm_tn(float (&acc)[4][4], const float *A, const float *B, int ty, int tx)
{
#pragma unroll 8
    for (int k = 0; k < TS; ++k) {
        float a[4], b[4];
#pragma unroll
        for (int r = 0; r < 4; ++r) a[r] = A[k * LD + ty * 4 + r];
#pragma unroll
        for (int c = 0; c < 4; ++c) b[c] = B[k * LD + tx + 16 * c];
#pragma unroll
        for (int r = 0; r < 4; ++r)
#pragma unroll
            for (int c = 0; c < 4; ++c) acc[r][c] = fmaf(a[r], b[c], acc[r][c]);
    }
}

__device__ __forceinline__ float group16_max(float v)
{
#pragma unroll
    for (int o = 8; o > 0; o >>= 1) v = fmaxf(v, __shfl_xor_sync(0xffffffffu, v, o));
    return v;
}
__device__ __forceinline__ float group16_sum(float v)
{
#pragma unroll
    for (int o = 8; o > 0; o >>= 1) v += __shfl_xor_sync(0xffffffffu, v, o);
    return v;
}

struct SimtArgs {
    const void *Q, *K, *V, *O, *dO;
    const float *LSE, *D;
    void *Oout, *dQ, *dK, *dV;
    float *LSEout;
    int n, d;
    int mask_kind, block, nb, mask_heads;
    const uint8_t *bits;
    float scale;
};

// ---------------------------------------------------------------- forward
// Steps F1-F3: scores, running row max / row sum, O = diag(l)^-1 exp(S - m) V.
template <typename T, int DCH>
__global__ void __launch_bounds__(NT) simt_fwd_kernel(SimtArgs a)
{
    extern __shared__ float sm[];
    float *sA = sm, *sB = sm + TS * LD, *sS = sm + 2 * TS * LD;
    const int tx = threadIdx.x % 16, ty = threadIdx.x / 16;
    const long bh = blockIdx.y;
    const int i0 = blockIdx.x * TS, n = a.n, d = a.d;
    const T *Q = (const T *)a.Q + (size_t)bh * n * d, *K = (const T *)a.K + (size_t)bh * n * d,
            *V = (const T *)a.V + (size_t)bh * n * d;
    const MaskDev mk = head_mask(a.mask_kind, a.block, a.nb, a.bits, a.mask_heads, bh);
    const int i1 = min(i0 + TS, n) - 1;

    float m[4], l[4], acc_o[4][DCH * 4];
#pragma unroll
    for (int r = 0; r < 4; ++r) {
        m[r] = -INFINITY;
        l[r] = 0.f;
#pragma unroll
        for (int c = 0; c < DCH * 4; ++c) acc_o[r][c] = 0.f;
    }
    for (int j0 = 0; j0 < n; j0 += TS) {
        if (!tile_any(mk, i0, i1, j0, min(j0 + TS, n) - 1)) continue;
        float acc[4][4] = {};
        for (int ch = 0; ch < DCH && ch * TS < d; ++ch) {
            load_chunk(sA, Q, i0, ch * TS, n, d);
            load_chunk(sB, K, j0, ch * TS, n, d);
            __syncthreads();
            mm_nt(acc, sA, sB, ty, tx);
            __syncthreads();
        }
#pragma unroll
        for (int r = 0; r < 4; ++r) {
            const int i = i0 + ty * 4 + r;
            float s[4], mx = -INFINITY;
#pragma unroll
            for (int c = 0; c < 4; ++c) {
                const int j = j0 + tx + 16 * c;
                s[c] = (i < n && j < n && keep(mk, i, j)) ? acc[r][c] * a.scale : -INFINITY;
                mx = fmaxf(mx, s[c]);
            }
            mx = group16_max(mx);
            const float m_new = fmaxf(m[r], mx);
            float alpha = 1.f, rs = 0.f, p[4] = {0.f, 0.f, 0.f, 0.f};
            if (m_new != -INFINITY) {
                alpha = expf(m[r] - m_new);
#pragma unroll
                for (int c = 0; c < 4; ++c) {
                    p[c] = expf(s[c] - m_new);
                    rs += p[c];
                }
            }
            rs = group16_sum(rs);
            l[r] = l[r] * alpha + rs;
            m[r] = m_new;
#pragma unroll
            for (int c = 0; c < DCH * 4; ++c) acc_o[r][c] *= alpha;
#pragma unroll
            for (int c = 0; c < 4; ++c) sS[(ty * 4 + r) * LD + tx + 16 * c] = p[c];
        }
        __syncthreads();
#pragma unroll
        for (int ch = 0; ch < DCH; ++ch) {
            if (ch * TS >= d) break;
            load_chunk(sB, V, j0, ch * TS, n, d);
            __syncthreads();
            float t[4][4];
#pragma unroll
            for (int r = 0; r < 4; ++r)
#pragma unroll
                for (int c = 0; c < 4; ++c) t[r][c] = acc_o[r][ch * 4 + c];
            mm_nn(t, sS, sB, ty, tx);
#pragma unroll
            for (int r = 0; r < 4; ++r)
#pragma unroll
                for (int c = 0; c < 4; ++c) acc_o[r][ch * 4 + c] = t[r][c];
            __syncthreads();
        }
    }
    T *O = (T *)a.Oout + (size_t)bh * n * d;
#pragma unroll
    for (int r = 0; r < 4; ++r) {
        const int i = i0 + ty * 4 + r;
        if (i >= n) continue;
        const float inv = l[r] > 0.f ? 1.f / l[r] : 0.f;
#pragma unroll
        for (int c = 0; c < DCH * 4; ++c) {
            const int col = (c / 4) * TS + tx + 16 * (c % 4);
            if (col < d) O[(size_t)i * d + col] = from_f<T>(acc_o[r][c] * inv);
        }
        if (tx == 0) a.LSEout[(size_t)bh * n + i] = l[r] > 0.f ? m[r] + logf(l[r]) : -INFINITY;
    }
}

// One score tile of the backward: P = exp(S - LSE) into sP (optional) and
// dS = P o (dP - D) into sdS, for queries i0.. and keys j0.. (steps B1-B3).
template <typename T, int DCH>
__device__ __forceinline__ void bwd_tile(const SimtArgs &a, const MaskDev &mk, const T *Q, const T *K, const T *V,
                                         const T *dO, const float *LSE, const float *D, int i0, int j0,
                                         float *sA, float *sB, float *sP, float *sdS, int ty, int tx)
{
    const int n = a.n, d = a.d;
    float acc[4][4] = {}, accp[4][4] = {};
    for (int ch = 0; ch < DCH && ch * TS < d; ++ch) {
        load_chunk(sA, Q, i0, ch * TS, n, d);
        load_chunk(sB, K, j0, ch * TS, n, d);
        __syncthreads();
        mm_nt(acc, sA, sB, ty, tx);
        __syncthreads();
        load_chunk(sA, dO, i0, ch * TS, n, d);
        load_chunk(sB, V, j0, ch * TS, n, d);
        __syncthreads();
        mm_nt(accp, sA, sB, ty, tx);
        __syncthreads();
    }
#pragma unroll
    for (int r = 0; r < 4; ++r) {
        const int i = i0 + ty * 4 + r;
        const float lse = i < n ? LSE[i] : -INFINITY;
        const float Di = i < n ? D[i] : 0.f;
#pragma unroll
        for (int c = 0; c < 4; ++c) {
            const int j = j0 + tx + 16 * c;
            float p = 0.f;
            if (i < n && j < n && lse != -INFINITY && keep(mk, i, j)) p = expf(acc[r][c] * a.scale - lse);
            if (sP) sP[(ty * 4 + r) * LD + tx + 16 * c] = p;
            sdS[(ty * 4 + r) * LD + tx + 16 * c] = p * (accp[r][c] - Di);
        }
    }
    __syncthreads();
}

// ---------------------------------------------------------------- backward: dQ (step B6)
template <typename T, int DCH>
__global__ void __launch_bounds__(NT) simt_bwd_dq_kernel(SimtArgs a)
{
    extern __shared__ float sm[];
    float *sA = sm, *sB = sm + TS * LD, *sdS = sm + 2 * TS * LD;
    const int tx = threadIdx.x % 16, ty = threadIdx.x / 16;
    const long bh = blockIdx.y;
    const int i0 = blockIdx.x * TS, n = a.n, d = a.d;
    const size_t off = (size_t)bh * n * d;
    const T *Q = (const T *)a.Q + off, *K = (const T *)a.K + off, *V = (const T *)a.V + off,
            *dO = (const T *)a.dO + off;
    const float *LSE = a.LSE + (size_t)bh * n, *D = a.D + (size_t)bh * n;
    const MaskDev mk = head_mask(a.mask_kind, a.block, a.nb, a.bits, a.mask_heads, bh);
    const int i1 = min(i0 + TS, n) - 1;
    float acc_q[4][DCH * 4];
#pragma unroll
    for (int r = 0; r < 4; ++r)
#pragma unroll
        for (int c = 0; c < DCH * 4; ++c) acc_q[r][c] = 0.f;
    for (int j0 = 0; j0 < n; j0 += TS) {
        if (!tile_any(mk, i0, i1, j0, min(j0 + TS, n) - 1)) continue;
        bwd_tile<T, DCH>(a, mk, Q, K, V, dO, LSE, D, i0, j0, sA, sB, nullptr, sdS, ty, tx);
#pragma unroll
        for (int ch = 0; ch < DCH; ++ch) {
            if (ch * TS >= d) break;
            load_chunk(sB, K, j0, ch * TS, n, d);
            __syncthreads();
            float t[4][4];
#pragma unroll
            for (int r = 0; r < 4; ++r)
#pragma unroll
                for (int c = 0; c < 4; ++c) t[r][c] = acc_q[r][ch * 4 + c];
            mm_nn(t, sdS, sB, ty, tx);
#pragma unroll
            for (int r = 0; r < 4; ++r)
#pragma unroll
                for (int c = 0; c < 4; ++c) acc_q[r][ch * 4 + c] = t[r][c];
            __syncthreads();
        }
    }
    T *dQ = (T *)a.dQ + off;
#pragma unroll
    for (int r = 0; r < 4; ++r) {
        const int i = i0 + ty * 4 + r;
        if (i >= n) continue;
#pragma unroll
        for (int c = 0; c < DCH * 4; ++c) {
            const int col = (c / 4) * TS + tx + 16 * (c % 4);
            if (col < d) dQ[(size_t)i * d + col] = from_f<T>(acc_q[r][c] * a.scale);
        }
    }
}

// ---------------------------------------------------------------- backward: dK, dV (steps B4, B5)
// blockIdx.z selects which group of OCH 64-column chunks of dK / dV this CTA produces.
template <typename T, int DCH, int OCH>
__global__ void __launch_bounds__(NT) simt_bwd_dkdv_kernel(SimtArgs a)
{
    extern __shared__ float sm[];
    float *sA = sm, *sB = sm + TS * LD, *sP = sm + 2 * TS * LD, *sdS = sm + 3 * TS * LD;
    const int tx = threadIdx.x % 16, ty = threadIdx.x / 16;
    const long bh = blockIdx.y;
    const int j0 = blockIdx.x * TS, n = a.n, d = a.d;
    const int ch0 = blockIdx.z * OCH;
    const size_t off = (size_t)bh * n * d;
    const T *Q = (const T *)a.Q + off, *K = (const T *)a.K + off, *V = (const T *)a.V + off,
            *dO = (const T *)a.dO + off;
    const float *LSE = a.LSE + (size_t)bh * n, *D = a.D + (size_t)bh * n;
    const MaskDev mk = head_mask(a.mask_kind, a.block, a.nb, a.bits, a.mask_heads, bh);
    const int j1 = min(j0 + TS, n) - 1;
    float acc_k[4][OCH * 4], acc_v[4][OCH * 4];
#pragma unroll
    for (int r = 0; r < 4; ++r)
#pragma unroll
        for (int c = 0; c < OCH * 4; ++c) acc_k[r][c] = acc_v[r][c] = 0.f;
    for (int i0 = 0; i0 < n; i0 += TS) {
        if (!tile_any(mk, i0, min(i0 + TS, n) - 1, j0, j1)) continue;
        bwd_tile<T, DCH>(a, mk, Q, K, V, dO, LSE, D, i0, j0, sA, sB, sP, sdS, ty, tx);
#pragma unroll
        for (int oc = 0; oc < OCH; ++oc) {
            const int ch = ch0 + oc;
            if (ch * TS >= d) break;
            load_chunk(sA, dO, i0, ch * TS, n, d);
            load_chunk(sB, Q, i0, ch * TS, n, d);
            __syncthreads();
            float t[4][4];
#pragma unroll
            for (int r = 0; r < 4; ++r)
#pragma unroll
                for (int c = 0; c < 4; ++c) t[r][c] = acc_v[r][oc * 4 + c];
            mm_tn(t, sP, sA, ty, tx);
#pragma unroll
            for (int r = 0; r < 4; ++r)
#pragma unroll
                for (int c = 0; c < 4; ++c) {
                    acc_v[r][oc * 4 + c] = t[r][c];
                    t[r][c] = acc_k[r][oc * 4 + c];
                }
            mm_tn(t, sdS, sB, ty, tx);
#pragma unroll
            for (int r = 0; r < 4; ++r)
#pragma unroll
                for (int c = 0; c < 4; ++c) acc_k[r][oc * 4 + c] = t[r][c];
            __syncthreads();
        }
    }
    T *dK = (T *)a.dK + off, *dV = (T *)a.dV + off;
#pragma unroll
    for (int r = 0; r < 4; ++r) {
        const int j = j0 + ty * 4 + r;
        if (j >= n) continue;
#pragma unroll
        for (int c = 0; c < OCH * 4; ++c) {
            const int col = (ch0 + c / 4) * TS + tx + 16 * (c % 4);
            if (col < d) {
                dK[(size_t)j * d + col] = from_f<T>(acc_k[r][c] * a.scale);
                dV[(size_t)j * d + col] = from_f<T>(acc_v[r][c]);
            }
        }
    }
}

// ---------------------------------------------------------------- D = rowsum(dO o O) (step B0)
// Memory-bound: every lane issues 16-byte loads; a row is shared by `lanes_per_row`
// adjacent lanes and summed with xor shuffles.  Requires (d * sizeof(T)) % 16 == 0.
template <typename T>
__global__ void __launch_bounds__(256) preprocess_kernel(const T *__restrict__ O, const T *__restrict__ dO,
                                                         float *__restrict__ D, size_t rows, int d,
                                                         int lanes_per_row)
{
    constexpr int VE = 16 / sizeof(T);                 // elements per 16-byte vector
    const int vec_per_row = d / VE;                    // lanes_per_row: largest power of two <= min(32, vec_per_row)
    const int rows_per_warp = 32 / lanes_per_row;
    const int lane = threadIdx.x % 32;
    const size_t warp = ((size_t)blockIdx.x * blockDim.x + threadIdx.x) / 32;
    const size_t nwarps = (size_t)gridDim.x * blockDim.x / 32;
    const int sub = lane / lanes_per_row, lr = lane % lanes_per_row;
    if (vec_per_row == lanes_per_row) {
        // one vector per lane and row: four row groups per step, all eight loads in flight before any is used
        constexpr int U = 4;
        const size_t step = (size_t)rows_per_warp * U;
        for (size_t base = warp * step; base < rows; base += nwarps * step) {
            uint4 xo[U], xg[U];
#pragma unroll
            for (int u = 0; u < U; ++u) {
                const size_t row = base + (size_t)u * rows_per_warp + sub;
                xo[u] = xg[u] = make_uint4(0u, 0u, 0u, 0u);
                if (row < rows) {
                    xo[u] = __ldcs(reinterpret_cast<const uint4 *>(O + row * d) + lr);
                    xg[u] = __ldcs(reinterpret_cast<const uint4 *>(dO + row * d) + lr);
                }
            }
#pragma unroll
            for (int u = 0; u < U; ++u) {
                const size_t row = base + (size_t)u * rows_per_warp + sub;
                const T *eo = reinterpret_cast<const T *>(&xo[u]), *eg = reinterpret_cast<const T *>(&xg[u]);
                float s = 0.f;
#pragma unroll
                for (int e = 0; e < VE; ++e) s = fmaf(to_f(eo[e]), to_f(eg[e]), s);
                for (int o = lanes_per_row / 2; o > 0; o >>= 1) s += __shfl_xor_sync(0xffffffffu, s, o);
                if (row < rows && lr == 0) D[row] = s;
            }
        }
        return;
    }
    for (size_t base = warp * rows_per_warp; base < rows; base += nwarps * rows_per_warp) {
        const size_t row = base + sub;
        float s = 0.f;
        if (row < rows) {
            const uint4 *po = reinterpret_cast<const uint4 *>(O + row * d);
            const uint4 *pg = reinterpret_cast<const uint4 *>(dO + row * d);
            for (int v = lr; v < vec_per_row; v += lanes_per_row) {
                uint4 xo = __ldg(po + v), xg = __ldg(pg + v);
                const T *eo = reinterpret_cast<const T *>(&xo), *eg = reinterpret_cast<const T *>(&xg);
#pragma unroll
                for (int e = 0; e < VE; ++e) s = fmaf(to_f(eo[e]), to_f(eg[e]), s);
            }
        }
        for (int o = lanes_per_row / 2; o > 0; o >>= 1) s += __shfl_xor_sync(0xffffffffu, s, o);
        if (row < rows && lr == 0) D[row] = s;
    }
}

// ---------------------------------------------------------------- block-mask index build
// One CTA per (mask head, block row) for the CSR half and per (mask head, block
// column) for the CSC half; ordered compaction by a single warp-free scan (nb is small).
// `ratio` > 1: the mask has nbm = about ratio * nb blocks per side, and block (I, J) of the lists is a
// super-block that is kept if any of its ratio x ratio mask blocks is.
__global__ void block_index_kernel(const uint8_t *bits, int nb, int nbm, int ratio, int *row_ptr, int *col_idx, int *col_ptr,
                                   int *row_idx)
{
    const int h = blockIdx.y, r = blockIdx.x;
    const uint8_t *mm = bits + (size_t)h * nbm * nbm;
    auto kept = [&](int I, int J) {
        for (int x = I * ratio; x < min((I + 1) * ratio, nbm); ++x)
            for (int y = J * ratio; y < min((J + 1) * ratio, nbm); ++y)
                if (mm[(size_t)x * nbm + y]) return true;
        return false;
    };
    if (threadIdx.x == 0) {
        int *cidx = col_idx + (size_t)h * nb * nb + (size_t)r * nb;
        int c = 0;
        for (int j = 0; j < nb; ++j)
            if (kept(r, j)) cidx[c++] = j;
        row_ptr[(size_t)h * 2 * nb + 2 * r] = r * nb;          // start, in col_idx of this head
        row_ptr[(size_t)h * 2 * nb + 2 * r + 1] = r * nb + c;  // end
    } else if (threadIdx.x == 32) {
        int *ridx = row_idx + (size_t)h * nb * nb + (size_t)r * nb;
        int c = 0;
        for (int i = 0; i < nb; ++i)
            if (kept(i, r)) ridx[c++] = i;
        col_ptr[(size_t)h * 2 * nb + 2 * r] = r * nb;
        col_ptr[(size_t)h * 2 * nb + 2 * r + 1] = r * nb + c;
    }
}

SimtArgs make_args(const Problem &p)
{
    SimtArgs a{};
    a.Q = p.Q; a.K = p.K; a.V = p.V; a.O = p.O; a.dO = p.dO;
    a.LSE = p.LSE; a.D = p.D;
    a.Oout = p.Oout; a.LSEout = p.LSEout; a.dQ = p.dQ; a.dK = p.dK; a.dV = p.dV;
    a.n = p.n; a.d = p.d;
    a.mask_kind = p.mask_kind; a.block = p.block; a.nb = p.nb; a.mask_heads = p.mask_heads;
    a.bits = p.block_mask;
    if (mask_is_element(p.mask_kind)) { a.block = p.n; a.nb = (p.n + 31) / 32; }
    a.scale = p.scale;
    return a;
}

template <typename K>
attn_status launch(const char *name, K kernel, dim3 grid, size_t smem, cudaStream_t s, const SimtArgs &a)
{
    if (cudaFuncSetAttribute(kernel, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)smem) != cudaSuccess)
        return ATTN_ERR_LAUNCH;
    launch_begin(name, s);
    kernel<<<grid, NT, smem, s>>>(a);
    launch_end(s);
    return cudaGetLastError() == cudaSuccess ? ATTN_OK : ATTN_ERR_LAUNCH;
}

template <typename T>
attn_status fwd_t(const Problem &p)
{
    const SimtArgs a = make_args(p);
    const dim3 grid((p.n + TS - 1) / TS, (unsigned)p.BH);
    const size_t smem = 3 * TS * LD * sizeof(float);
    if (p.d <= 64) return launch("simt_fwd", simt_fwd_kernel<T, 1>, grid, smem, p.stream, a);
    if (p.d <= 128) return launch("simt_fwd", simt_fwd_kernel<T, 2>, grid, smem, p.stream, a);
    return launch("simt_fwd", simt_fwd_kernel<T, 4>, grid, smem, p.stream, a);
}

template <typename T>
attn_status bwd_t(const Problem &p)
{
    const SimtArgs a = make_args(p);
    const dim3 grid((p.n + TS - 1) / TS, (unsigned)p.BH);
    const size_t smem3 = 3 * TS * LD * sizeof(float), smem4 = 4 * TS * LD * sizeof(float);
    attn_status st;
    if (p.d <= 64) {
        st = launch("simt_bwd_dkdv", simt_bwd_dkdv_kernel<T, 1, 1>, grid, smem4, p.stream, a);
        if (st == ATTN_OK) st = launch("simt_bwd_dq", simt_bwd_dq_kernel<T, 1>, grid, smem3, p.stream, a);
    } else if (p.d <= 128) {
        st = launch("simt_bwd_dkdv", simt_bwd_dkdv_kernel<T, 2, 2>, grid, smem4, p.stream, a);
        if (st == ATTN_OK) st = launch("simt_bwd_dq", simt_bwd_dq_kernel<T, 2>, grid, smem3, p.stream, a);
    } else {
        st = launch("simt_bwd_dkdv", simt_bwd_dkdv_kernel<T, 4, 2>, dim3(grid.x, grid.y, 2), smem4, p.stream, a);
        if (st == ATTN_OK) st = launch("simt_bwd_dq", simt_bwd_dq_kernel<T, 4>, grid, smem3, p.stream, a);
    }
    return st;
}

}  // namespace

attn_status simt_fwd(const Problem &p)
{
    return p.dt == ATTN_F32 ? fwd_t<float>(p) : fwd_t<__nv_bfloat16>(p);
}

attn_status simt_bwd(const Problem &p)
{
    attn_status st = preprocess_D(p.O, p.dO, p.D, (size_t)p.BH * p.n, p.d, p.dt, p.stream);
    if (st != ATTN_OK) return st;
    return p.dt == ATTN_F32 ? bwd_t<float>(p) : bwd_t<__nv_bfloat16>(p);
}

attn_status preprocess_D(const void *O, const void *dO, float *D, size_t rows, int d, int dt, cudaStream_t s)
{
    if (rows == 0) return ATTN_OK;
    const int elem = dt == ATTN_F32 ? 4 : 2;
    if (d <= 0 || (d * elem) % 16 != 0) return ATTN_ERR_SHAPE;
    const int vec_per_row = d * elem / 16;
    int lanes = 1;
    while (lanes * 2 <= vec_per_row && lanes < 32) lanes *= 2;
    const size_t rows_per_warp = 32 / lanes;
    const size_t warps = (rows + rows_per_warp - 1) / rows_per_warp;
    size_t blocks = (warps + 7) / 8;
    const size_t cap = (size_t)sm_count() * 8;      // eight resident CTAs of 256 threads per SM, grid-stride beyond that
    if (blocks > cap) blocks = cap;
    launch_begin("bwd_preprocess_D", s);
    if (dt == ATTN_F32)
        preprocess_kernel<float><<<(unsigned)blocks, 256, 0, s>>>((const float *)O, (const float *)dO, D, rows, d,
                                                                lanes);
    else
        preprocess_kernel<__nv_bfloat16><<<(unsigned)blocks, 256, 0, s>>>((const __nv_bfloat16 *)O,
                                                                         (const __nv_bfloat16 *)dO, D, rows, d, lanes);
    launch_end(s);
    return cudaGetLastError() == cudaSuccess ? ATTN_OK : ATTN_ERR_LAUNCH;
}

// ---------------------------------------------------------------- element masks
// One warp per 32 x 32 block of the bitmap: writes the transposed block (row j, bit i) for the key-stationary
// kernels and marks the 128 x 128 tile as kept if the block has a bit set.  Bits beyond n are dropped here, so
// the kernels never see them.  grid (words, ceil(n / 32), mask_heads), 32 threads.
__global__ void element_mask_prepare_kernel(const uint32_t *__restrict__ rowbits, uint32_t *__restrict__ colbits,
                                            uint8_t *__restrict__ tilemask, int n, int words, int nb)
{
    const int wj = blockIdx.x, ri = blockIdx.y, h = blockIdx.z, lane = threadIdx.x;
    const int i = ri * 32 + lane;
    uint32_t w = i < n ? rowbits[((size_t)h * n + i) * words + wj] : 0u;
    const int jrem = n - wj * 32;                       // valid columns in this word
    if (jrem < 32) w &= (1u << jrem) - 1u;
    uint32_t mine = 0;
#pragma unroll
    for (int c = 0; c < 32; ++c) {
        const uint32_t col = __ballot_sync(0xffffffffu, (w >> c) & 1u);   // bit r = entry (ri * 32 + r, wj * 32 + c)
        if (lane == c) mine = col;
    }
    const int j = wj * 32 + lane;
    if (j < n) colbits[((size_t)h * n + j) * words + ri] = mine;
    if (__any_sync(0xffffffffu, w != 0u) && lane == 0) tilemask[((size_t)h * nb + ri / 4) * nb + wj / 4] = 1;
}

__global__ void coo_scatter_kernel(const int *__restrict__ rows, const int *__restrict__ cols, const int *__restrict__ heads,
                                   size_t nnz, int n, int mask_heads, int words, uint32_t *__restrict__ bitmap)
{
    for (size_t e = (size_t)blockIdx.x * blockDim.x + threadIdx.x; e < nnz; e += (size_t)gridDim.x * blockDim.x) {
        const int i = rows[e], j = cols[e], h = heads ? heads[e] : 0;
        if (i < 0 || i >= n || j < 0 || j >= n || h < 0 || h >= mask_heads) continue;
        atomicOr(bitmap + ((size_t)h * n + i) * words + j / 32, 1u << (j % 32));
    }
}

attn_status build_block_index(const Problem &p)
{
    if (!mask_is_block(p.mask_kind) || !p.row_ptr) return ATTN_OK;
    if (p.fine.mode == 2) {
        // element mask: transposed bitmap and the mask of 128 x 128 tiles, from which the lists below are built
        if (cudaMemsetAsync(p.tilemask, 0, (size_t)p.mask_heads * p.nb * p.nb, p.stream) != cudaSuccess) return ATTN_ERR_LAUNCH;
        launch_begin("element_mask_prepare", p.stream);
        element_mask_prepare_kernel<<<dim3(p.fine.words, (p.n + 31) / 32, p.mask_heads), 32, 0, p.stream>>>(
            p.fine.rowbits, p.colbits, p.tilemask, p.n, p.fine.words, p.nb);
        launch_end(p.stream);
        if (cudaGetLastError() != cudaSuccess) return ATTN_ERR_LAUNCH;
    }
    launch_begin("block_index", p.stream);
    const int nbm = p.fine.mode == 1 ? p.fine.nb : p.nb, ratio = p.fine.mode == 1 ? 128 / p.fine.block : 1;
    block_index_kernel<<<dim3(p.nb, p.mask_heads), 64, 0, p.stream>>>(p.block_mask, p.nb, nbm, ratio, p.row_ptr, p.col_idx,
                                                                      p.col_ptr, p.row_idx);
    launch_end(p.stream);
    return cudaGetLastError() == cudaSuccess ? ATTN_OK : ATTN_ERR_LAUNCH;
}

}  // namespace attn

extern "C" attn_status attn_mask_from_coo(const int *rows, const int *cols, const int *heads, size_t nnz, int n, int mask_heads,
                                          uint32_t *bitmap, void *cuda_stream)
{
    if (!bitmap || (nnz && (!rows || !cols))) return ATTN_ERR_NULL;
    if (n < 1 || mask_heads < 1) return ATTN_ERR_SHAPE;
    if (((uintptr_t)bitmap & 3) != 0) return ATTN_ERR_ALIGN;
    cudaStream_t s = static_cast<cudaStream_t>(cuda_stream);
    const int words = (n + 31) / 32;
    if (cudaMemsetAsync(bitmap, 0, (size_t)mask_heads * n * words * sizeof(uint32_t), s) != cudaSuccess) return ATTN_ERR_LAUNCH;
    if (nnz == 0) return ATTN_OK;
    size_t blocks = (nnz + 255) / 256;
    if (blocks > (size_t)attn::sm_count() * 16) blocks = (size_t)attn::sm_count() * 16;
    attn::launch_begin("mask_from_coo", s);
    attn::coo_scatter_kernel<<<(unsigned)blocks, 256, 0, s>>>(rows, cols, heads, nnz, n, mask_heads, words, bitmap);
    attn::launch_end(s);
    return cudaGetLastError() == cudaSuccess ? ATTN_OK : ATTN_ERR_LAUNCH;
}

// C-ABI entry points of libattn_b200: argument validation, workspace layout,
// algorithm selection and the closed-form I/O bounds.  No kernel lives here.
#include <math.h>
#include <string.h>

#include "attn_internal.h"

namespace attn {
namespace {

struct Args {
    int n, d, heads, batch, dt;
    const attn_mask *mask;
    const attn_cfg *cfg;
};

int elem_size(int dt) { return dt == ATTN_F32 ? 4 : 2; }

// block edges the tensor-core kernels take: whole 128 x 128 tiles, or 32 / 64 (several blocks per tile)
bool tc_block_ok(int block) { return block > 0 && (block % 128 == 0 || block == 64 || block == 32); }

// Resolves algo / tiles; returns ATTN_OK or the validation error.
attn_status resolve_cfg(const Args &a, int backward, attn_cfg *out)
{
    attn_cfg c{};
    if (a.cfg) c = *a.cfg;
    if (c.algo < ATTN_ALGO_AUTO || c.algo > ATTN_ALGO_SIMT) return ATTN_ERR_TILE;
    if (c.tile_q < 0 || c.tile_k < 0 || c.tile_d < 0) return ATTN_ERR_TILE;
    if (c.algo == ATTN_ALGO_AUTO) {
        attn_cfg probe = c;
        probe.algo = ATTN_ALGO_FUSED;
        const bool tc_ok = a.dt == ATTN_BF16 && (a.n % 8) == 0 && tc_cfg_supported(a.d, probe, backward) &&
                           !(a.mask && mask_is_block(a.mask->kind) && !tc_block_ok(a.mask->block));
        c.algo = tc_ok ? ATTN_ALGO_FUSED : ATTN_ALGO_SIMT;
        // d = 256 backward: the fused tile set does not fit on chip; the small-cache algorithm takes it
        probe.algo = ATTN_ALGO_MATERIALIZED;
        if (!tc_ok && backward && a.dt == ATTN_BF16 && a.d == 256 && (a.n % 8) == 0 &&
            !(a.mask && (mask_is_block(a.mask->kind) || mask_is_element(a.mask->kind))) && tc_cfg_supported(a.d, probe, backward))
            c.algo = ATTN_ALGO_MATERIALIZED;
    }
    if (c.algo == ATTN_ALGO_MATERIALIZED && !backward) {   // its forward is the fused one, with that kernel's own tiles
        c.algo = ATTN_ALGO_FUSED;
        c.tile_q = c.tile_k = c.tile_d = 0;
    }
    // a configuration that names a backward tile shape may be handed to the forward as well (one cfg for a
    // forward / backward pair): the forward then runs with its own tiles
    if (c.algo == ATTN_ALGO_FUSED && !backward && a.dt == ATTN_BF16 && !tc_cfg_supported(a.d, c, 0) &&
        tc_cfg_supported(a.d, c, 1))
        c.tile_q = c.tile_k = c.tile_d = 0;
    if (c.algo == ATTN_ALGO_SIMT) {
        if ((c.tile_q && c.tile_q != 64) || (c.tile_k && c.tile_k != 64) || (c.tile_d && c.tile_d != 64))
            return ATTN_ERR_TILE;
        c.tile_q = c.tile_k = c.tile_d = 64;
    } else {
        if (a.dt != ATTN_BF16) return ATTN_ERR_DTYPE;
        if (a.d != 64 && a.d != 128 && a.d != 256) return ATTN_ERR_SHAPE;
        if (a.n % 8 != 0) return ATTN_ERR_SHAPE;
        if (a.mask && mask_is_block(a.mask->kind) && !tc_block_ok(a.mask->block)) return ATTN_ERR_MASK;
        if (c.algo == ATTN_ALGO_MATERIALIZED && a.mask && (mask_is_block(a.mask->kind) || mask_is_element(a.mask->kind)))
            return ATTN_ERR_MASK;
        if (!tc_cfg_supported(a.d, c, backward)) return ATTN_ERR_TILE;
        // fill defaults the way the kernels resolve them
        attn_cfg list[32];
        const int cnt = attn_supported_cfgs(a.d, a.dt, list, 32);
        for (int i = 0; i < cnt; ++i) {
            if (list[i].algo != c.algo) continue;
            attn_cfg cand = list[i];
            cand.deterministic = c.deterministic;
            if (!tc_cfg_supported(a.d, cand, backward)) continue;
            if ((c.tile_q == 0 || c.tile_q == list[i].tile_q) && (c.tile_k == 0 || c.tile_k == list[i].tile_k) &&
                (c.tile_d == 0 || c.tile_d == list[i].tile_d)) {
                c.tile_q = list[i].tile_q; c.tile_k = list[i].tile_k; c.tile_d = list[i].tile_d;
                break;
            }
        }
    }
    *out = c;
    return ATTN_OK;
}

attn_status check_shape(const Args &a)
{
    if (a.dt != ATTN_F32 && a.dt != ATTN_BF16) return ATTN_ERR_DTYPE;
    if (a.n < 1 || a.heads < 1 || a.batch < 1) return ATTN_ERR_SHAPE;
    if (a.d < 8 || a.d > 256 || a.d % 8 != 0) return ATTN_ERR_SHAPE;
    if ((long)a.batch * a.heads > 65535) return ATTN_ERR_SHAPE;
    if ((double)a.batch * a.heads * a.n * a.d > 1.7e10) return ATTN_ERR_SHAPE;
    if (a.mask) {
        const attn_mask &m = *a.mask;
        if (m.kind < ATTN_MASK_NONE || m.kind > ATTN_MASK_ELEMENT) return ATTN_ERR_MASK;
        if (mask_is_block(m.kind) || mask_is_element(m.kind)) {
            if (mask_is_block(m.kind) && m.block < 1) return ATTN_ERR_MASK;
            if (m.mask_heads != 1 && m.mask_heads != a.batch * a.heads) return ATTN_ERR_MASK;
        }
    }
    return ATTN_OK;
}

attn_status layout(const Args &a, int backward, attn_cfg *cfg_out, WorkspaceLayout *L)
{
    attn_status st = check_shape(a);
    if (st != ATTN_OK) return st;
    attn_cfg c;
    st = resolve_cfg(a, backward, &c);
    if (st != ATTN_OK) return st;
    if (cfg_out) *cfg_out = c;
    memset(L, 0, sizeof(*L));
    size_t off = 0;
    L->status = off; off += 256;
    const size_t BH = (size_t)a.batch * a.heads;
    if (backward) { L->D = off; off += align_up(BH * a.n * sizeof(float), 256); }
    const bool element = a.mask && mask_is_element(a.mask->kind);
    const bool sparse = a.mask && (mask_is_block(a.mask->kind) || element);
    if (sparse && c.algo != ATTN_ALGO_SIMT) {
        // fine blocks and element masks: lists of the 128 x 128 tiles that keep anything
        const int eff = (element || a.mask->block < 128) ? 128 : a.mask->block;
        const size_t nb = (a.n + eff - 1) / eff, mh = a.mask->mask_heads;
        L->row_ptr = off; off += align_up(mh * 2 * nb * sizeof(int), 256);
        L->col_idx = off; off += align_up(mh * nb * nb * sizeof(int), 256);
        L->col_ptr = off; off += align_up(mh * 2 * nb * sizeof(int), 256);
        L->row_idx = off; off += align_up(mh * nb * nb * sizeof(int), 256);
        if (element) {
            L->tilemask = off; off += align_up(mh * nb * nb, 256);
            L->colbits = off; off += align_up(mh * (size_t)a.n * ((a.n + 31) / 32) * sizeof(uint32_t), 256);
        }
    }
    if (backward && (c.algo == ATTN_ALGO_FUSED || c.algo == ATTN_ALGO_MATERIALIZED)) { L->nLSE2 = off; off += align_up(BH * a.n * sizeof(float), 256); }
    if (backward && c.algo == ATTN_ALGO_FUSED && !c.deterministic) {
        L->dQ_acc = off; off += align_up(BH * a.n * a.d * sizeof(float), 256);
    }
    if (backward && c.algo == ATTN_ALGO_MATERIALIZED) {
        // P, dP, dS for as many heads at a time as fit in about 1 GiB each (at least one head).
        const size_t per_head = (size_t)a.n * a.n * 2;
        size_t mh = (size_t(1) << 30) / per_head;
        if (mh < 1) mh = 1;
        if (mh > BH) mh = BH;
        L->mat_heads = (int)mh;
        L->matP = off; off += align_up(mh * per_head, 256);
        L->matdP = off; off += align_up(mh * per_head, 256);
        L->matdS = off; off += align_up(mh * per_head, 256);
    }
    L->total = off;
    return ATTN_OK;
}

bool aligned16(const void *p) { return ((uintptr_t)p & 15) == 0; }

attn_status check_arch()
{
    int dev = 0, major = 0;
    if (cudaGetDevice(&dev) != cudaSuccess) return ATTN_ERR_ARCH;
    if (cudaDeviceGetAttribute(&major, cudaDevAttrComputeCapabilityMajor, dev) != cudaSuccess) return ATTN_ERR_ARCH;
    return major == 10 ? ATTN_OK : ATTN_ERR_ARCH;
}

}  // namespace

int sm_count()
{
    int dev = 0, sms = 0;
    if (cudaGetDevice(&dev) != cudaSuccess ||
        cudaDeviceGetAttribute(&sms, cudaDevAttrMultiProcessorCount, dev) != cudaSuccess || sms <= 0)
        return 1;
    return sms;
}

namespace {

attn_status fill_problem(Problem &p, const Args &a, int backward, float scale, void *workspace, size_t workspace_bytes,
                         void *stream)
{
    WorkspaceLayout L;
    attn_cfg c;
    attn_status st = layout(a, backward, &c, &L);
    if (st != ATTN_OK) return st;
    if (a.mask && (mask_is_block(a.mask->kind) || mask_is_element(a.mask->kind)) && !a.mask->block_mask) return ATTN_ERR_NULL;
    if (a.mask && mask_is_element(a.mask->kind) && ((uintptr_t)a.mask->block_mask & 3) != 0) return ATTN_ERR_ALIGN;
    if (!workspace || workspace_bytes < L.total) return ATTN_ERR_WORKSPACE;
    if (((uintptr_t)workspace & 255) != 0) return ATTN_ERR_ALIGN;
    if (!(scale >= 0.f) || isinf(scale)) return ATTN_ERR_SHAPE;
    p.n = a.n; p.d = a.d; p.heads = a.heads; p.batch = a.batch;
    p.BH = (long)a.batch * a.heads;
    p.dt = a.dt;
    p.mask_kind = a.mask ? a.mask->kind : ATTN_MASK_NONE;
    p.block = mask_is_block(p.mask_kind) ? a.mask->block : 0;
    p.mask_heads = (mask_is_block(p.mask_kind) || mask_is_element(p.mask_kind)) ? a.mask->mask_heads : 1;
    p.nb = p.block ? (a.n + p.block - 1) / p.block : 0;
    p.block_mask = (mask_is_block(p.mask_kind) || mask_is_element(p.mask_kind)) ? a.mask->block_mask : nullptr;
    p.fine = FineMask{};
    if (p.block && p.block < 128 && c.algo != ATTN_ALGO_SIMT) {
        p.fine.mode = 1; p.fine.bits = p.block_mask; p.fine.block = p.block; p.fine.nb = p.nb;
        p.block = 128;
        p.nb = (a.n + 127) / 128;
    }
    p.scale = scale == 0.f ? 1.0f / sqrtf((float)a.d) : scale;
    p.cfg = c;
    char *w = (char *)workspace;
    p.status = (uint32_t *)(w + L.status);
    p.D = backward ? (float *)(w + L.D) : nullptr;
    p.nLSE2 = L.nLSE2 ? (float *)(w + L.nLSE2) : nullptr;
    p.row_ptr = L.row_ptr ? (int *)(w + L.row_ptr) : nullptr;
    p.col_idx = L.col_idx ? (int *)(w + L.col_idx) : nullptr;
    p.col_ptr = L.col_ptr ? (int *)(w + L.col_ptr) : nullptr;
    p.row_idx = L.row_idx ? (int *)(w + L.row_idx) : nullptr;
    p.tilemask = L.tilemask ? (uint8_t *)(w + L.tilemask) : nullptr;
    p.colbits = L.colbits ? (uint32_t *)(w + L.colbits) : nullptr;
    if (mask_is_element(p.mask_kind) && c.algo != ATTN_ALGO_SIMT) {
        // the tensor-core kernels see a block mask of 128 x 128 tiles (built from the bitmap) with the bits applied inside the tiles
        p.fine.mode = 2; p.fine.rowbits = (const uint32_t *)a.mask->block_mask; p.fine.colbits = p.colbits;
        p.fine.n = a.n; p.fine.words = (a.n + 31) / 32;
        p.mask_kind = ATTN_MASK_BLOCK_SPARSE;
        p.block = 128;
        p.nb = (a.n + 127) / 128;
        p.block_mask = p.tilemask;
    }
    p.dQ_acc = L.dQ_acc ? (float *)(w + L.dQ_acc) : nullptr;
    p.matP = L.matP ? w + L.matP : nullptr;
    p.matdP = L.matdP ? w + L.matdP : nullptr;
    p.matdS = L.matdS ? w + L.matdS : nullptr;
    p.mat_heads = L.mat_heads;
    p.stream = (cudaStream_t)stream;
    return ATTN_OK;
}

}  // namespace
}  // namespace attn

namespace attn {
namespace {
constexpr int kTimingPool = 256;
struct Timing {
    bool on = false;
    int count = 0;
    bool open = false;
    cudaEvent_t ev[2 * kTimingPool];
    const char *names[kTimingPool];
} g_timing;
unsigned long long g_launches = 0;
}  // namespace

void launch_begin(const char *name, cudaStream_t s)
{
    ++g_launches;
    g_timing.open = false;
    if (g_timing.on && g_timing.count < kTimingPool) {
        g_timing.names[g_timing.count] = name;
        cudaEventRecord(g_timing.ev[2 * g_timing.count], s);
        g_timing.open = true;
    }
}

void launch_end(cudaStream_t s)
{
    if (g_timing.open) {
        cudaEventRecord(g_timing.ev[2 * g_timing.count + 1], s);
        ++g_timing.count;
        g_timing.open = false;
    }
}

attn_status bwd_internal(const void *Q, const void *K, const void *V, const void *O, const void *dO, const float *LSE,
                         void *dQ, void *dK, void *dV, int n, int d, int heads, int batch, const attn_mask *mask, int dt,
                         float scale, const attn_cfg *cfg, void *workspace, size_t workspace_bytes, void *cuda_stream,
                         bool keep_acc, const float **dQ_acc)
{
    if (dQ_acc) *dQ_acc = nullptr;
    if (!Q || !K || !V || !O || !dO || !LSE || !dQ || !dK || !dV) return ATTN_ERR_NULL;
    Problem p{};
    const Args a{n, d, heads, batch, dt, mask, cfg};
    attn_status st = fill_problem(p, a, 1, scale, workspace, workspace_bytes, cuda_stream);
    if (st != ATTN_OK) return st;
    if (!aligned16(Q) || !aligned16(K) || !aligned16(V) || !aligned16(O) || !aligned16(dO) || !aligned16(dQ) ||
        !aligned16(dK) || !aligned16(dV) || ((uintptr_t)LSE & 3))
        return ATTN_ERR_ALIGN;
    if ((st = check_arch()) != ATTN_OK) return st;
    p.Q = Q; p.K = K; p.V = V; p.O = O; p.dO = dO; p.LSE = LSE; p.dQ = dQ; p.dK = dK; p.dV = dV;
    if (cudaMemsetAsync(p.status, 0, 4, p.stream) != cudaSuccess) return ATTN_ERR_LAUNCH;
    if (p.cfg.algo == ATTN_ALGO_SIMT) return simt_bwd(p);
    if ((st = build_block_index(p)) != ATTN_OK) return st;
    if (p.cfg.algo == ATTN_ALGO_MATERIALIZED) return mat_bwd(p);
    if (keep_acc && dQ_acc && p.dQ_acc) {
        // the fused kernels leave the final dQ in the fp32 accumulator; without a destination the conversion is skipped
        p.dQ = nullptr;
        *dQ_acc = p.dQ_acc;
    }
    return tc_bwd(p);
}
}  // namespace attn

using namespace attn;

extern "C" {

attn_status attn_fwd(const void *Q, const void *K, const void *V, void *O, float *LSE, int n, int d, int heads,
                     int batch, const attn_mask *mask, int dt, float scale, const attn_cfg *cfg, void *workspace,
                     size_t workspace_bytes, void *cuda_stream)
{
    if (!Q || !K || !V || !O || !LSE) return ATTN_ERR_NULL;
    Problem p{};
    const Args a{n, d, heads, batch, dt, mask, cfg};
    attn_status st = fill_problem(p, a, 0, scale, workspace, workspace_bytes, cuda_stream);
    if (st != ATTN_OK) return st;
    if (!aligned16(Q) || !aligned16(K) || !aligned16(V) || !aligned16(O) || ((uintptr_t)LSE & 3)) return ATTN_ERR_ALIGN;
    if ((st = check_arch()) != ATTN_OK) return st;
    p.Q = Q; p.K = K; p.V = V; p.Oout = O; p.LSEout = LSE;
    if (cudaMemsetAsync(p.status, 0, 4, p.stream) != cudaSuccess) return ATTN_ERR_LAUNCH;
    if (p.cfg.algo == ATTN_ALGO_SIMT) return simt_fwd(p);
    if ((st = build_block_index(p)) != ATTN_OK) return st;
    return tc_fwd(p);
}

attn_status attn_bwd(const void *Q, const void *K, const void *V, const void *O, const void *dO, const float *LSE,
                     void *dQ, void *dK, void *dV, int n, int d, int heads, int batch, const attn_mask *mask, int dt,
                     float scale, const attn_cfg *cfg, void *workspace, size_t workspace_bytes, void *cuda_stream)
{
    return attn::bwd_internal(Q, K, V, O, dO, LSE, dQ, dK, dV, n, d, heads, batch, mask, dt, scale, cfg, workspace,
                              workspace_bytes, cuda_stream, false, nullptr);
}

attn_status attn_bwd_preprocess(const void *O, const void *dO, float *D, size_t rows, int d, int dt, void *cuda_stream)
{
    if (!O || !dO || !D) return ATTN_ERR_NULL;
    if (dt != ATTN_F32 && dt != ATTN_BF16) return ATTN_ERR_DTYPE;
    if (d < 8 || d > 256 || d % 8 != 0) return ATTN_ERR_SHAPE;
    if (!aligned16(O) || !aligned16(dO) || ((uintptr_t)D & 3)) return ATTN_ERR_ALIGN;
    attn_status st = check_arch();
    if (st != ATTN_OK) return st;
    return preprocess_D(O, dO, D, rows, d, dt, (cudaStream_t)cuda_stream);
}

size_t attn_fwd_workspace_bytes(int n, int d, int heads, int batch, const attn_mask *mask, int dt, const attn_cfg *cfg)
{
    WorkspaceLayout L;
    const Args a{n, d, heads, batch, dt, mask, cfg};
    return layout(a, 0, nullptr, &L) == ATTN_OK ? L.total : 0;
}

size_t attn_bwd_workspace_bytes(int n, int d, int heads, int batch, const attn_mask *mask, int dt, const attn_cfg *cfg)
{
    WorkspaceLayout L;
    const Args a{n, d, heads, batch, dt, mask, cfg};
    return layout(a, 1, nullptr, &L) == ATTN_OK ? L.total : 0;
}

attn_status attn_workspace_status(const void *workspace, void *cuda_stream)
{
    if (!workspace) return ATTN_ERR_NULL;
    uint32_t word = 0;
    if (cudaMemcpyAsync(&word, workspace, 4, cudaMemcpyDeviceToHost, (cudaStream_t)cuda_stream) != cudaSuccess)
        return ATTN_ERR_LAUNCH;
    if (cudaStreamSynchronize((cudaStream_t)cuda_stream) != cudaSuccess) return ATTN_ERR_LAUNCH;
    return word == 0 ? ATTN_OK : ATTN_ERR_DEVICE_TIMEOUT;
}

int attn_supported_cfgs(int d, int dt, attn_cfg *out, int max_out)
{
    int cnt = 0;
    auto add = [&](int tq, int tk, int td, int algo) {
        if (out && cnt < max_out) out[cnt] = attn_cfg{tq, tk, td, algo, 0};
        ++cnt;
    };
    if (d >= 8 && d <= 256 && d % 8 == 0 && (dt == ATTN_F32 || dt == ATTN_BF16)) add(64, 64, 64, ATTN_ALGO_SIMT);
    if (dt == ATTN_BF16 && (d == 64 || d == 128 || d == 256)) {
        const int tiles[][4] = {
            {128, 128, 0, ATTN_ALGO_FUSED},
            {128, 64, 0, ATTN_ALGO_FUSED},
            {64, 128, 0, ATTN_ALGO_FUSED},
            {256, 128, 64, ATTN_ALGO_MATERIALIZED},   // the first entry of an algorithm is its default
            {256, 64, 64, ATTN_ALGO_MATERIALIZED},
            {256, 32, 64, ATTN_ALGO_MATERIALIZED},
            {128, 128, 64, ATTN_ALGO_MATERIALIZED},
            {128, 64, 64, ATTN_ALGO_MATERIALIZED},
            {128, 32, 64, ATTN_ALGO_MATERIALIZED},
        };
        for (auto &t : tiles) {
            attn_cfg c{t[0], t[1], t[2] ? t[2] : d, t[3], 0};
            if (tc_cfg_supported(d, c, 1) || tc_cfg_supported(d, c, 0)) add(c.tile_q, c.tile_k, c.tile_d, c.algo);
        }
    }
    return cnt;
}

size_t attn_cfg_onchip_elems(int d, int dt, const attn_cfg *cfg, int backward)
{
    const Args a{8, d, 1, 1, dt, nullptr, cfg};
    attn_cfg c;
    if (check_shape(a) != ATTN_OK || resolve_cfg(a, backward, &c) != ATTN_OK) return 0;
    if (c.algo == ATTN_ALGO_SIMT) {
        // shared-memory tiles of the fp32 kernels: 3 (forward, dQ) or 4 (dK/dV) padded 64 x 64 float tiles
        return (size_t)(backward ? 4 : 3) * 64 * 65;
    }
    return tc_cfg_onchip_bytes(d, c, backward) / elem_size(dt);
}

double attn_io_bound_elems(double n, double d, double M, int backward)
{
    if (!(n > 0) || !(d > 0) || !(M > 0)) return 0.0;
    const double large = backward ? (n * n * d * d + n * d * d * d) / M : n * n * d * d / M;
    const double small = backward ? (n * n * d + n * d * d) / sqrt(M) : n * n * d / sqrt(M);
    return large < small ? large : small;
}

double attn_io_bound_sparse_elems(double z_input, double z_qk, double M)
{
    if (!(z_input > 0) || !(z_qk > 0) || !(M > 0)) return 0.0;
    const double large = z_input * z_input / M;
    const double small = z_input * sqrt(z_qk) / sqrt(M);
    return large < small ? large : small;
}

unsigned long long attn_kernel_launches(void) { return g_launches; }

attn_status attn_timing_enable(int on)
{
    if (on && !g_timing.on) {
        for (int i = 0; i < 2 * kTimingPool; ++i)
            if (cudaEventCreate(&g_timing.ev[i]) != cudaSuccess) return ATTN_ERR_LAUNCH;
        g_timing.count = 0;
        g_timing.on = true;
    } else if (!on && g_timing.on) {
        for (int i = 0; i < 2 * kTimingPool; ++i) cudaEventDestroy(g_timing.ev[i]);
        g_timing.on = false;
        g_timing.count = 0;
    }
    return ATTN_OK;
}

int attn_timing_collect(float *ms, const char **names, int max)
{
    if (!g_timing.on) return 0;
    int out = 0;
    for (int i = 0; i < g_timing.count; ++i) {
        float t = 0.f;
        if (cudaEventSynchronize(g_timing.ev[2 * i + 1]) != cudaSuccess) break;
        if (cudaEventElapsedTime(&t, g_timing.ev[2 * i], g_timing.ev[2 * i + 1]) != cudaSuccess) break;
        if (out < max) {
            if (ms) ms[out] = t;
            if (names) names[out] = g_timing.names[i];
            ++out;
        }
    }
    g_timing.count = 0;
    return out;
}

const char *attn_status_str(int status)
{
    switch (status) {
    case ATTN_OK: return "ok";
    case ATTN_ERR_NULL: return "null pointer";
    case ATTN_ERR_SHAPE: return "unsupported shape";
    case ATTN_ERR_DTYPE: return "unsupported dtype";
    case ATTN_ERR_ALIGN: return "misaligned pointer";
    case ATTN_ERR_TILE: return "unsupported tile configuration";
    case ATTN_ERR_MASK: return "bad mask";
    case ATTN_ERR_WORKSPACE: return "workspace missing or too small";
    case ATTN_ERR_ARCH: return "device is not sm_100";
    case ATTN_ERR_LAUNCH: return "CUDA launch failed";
    case ATTN_ERR_DEVICE_TIMEOUT: return "kernel gave up on a bounded wait";
    }
    return "unknown status";
}

}  // extern "C"

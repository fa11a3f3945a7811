/*
 * attn.h -- exact softmax attention, forward and backward, for NVIDIA B200 (sm_100a).
 *
 * C ABI.  Plain pointers and sizes only.  Unless a parameter says "host", every
 * pointer is DEVICE memory owned by the caller; the library allocates nothing and
 * frees nothing.  All work is enqueued on the given CUDA
 * stream (a cudaStream_t passed as void*; NULL = the legacy default stream) and the
 * calls return without synchronising.
 *
 * What is computed, per (batch, head), for Q, K, V, dO of shape n x d:
 *
 *   S_ij  = scale * sum_c Q_ic K_jc            kept (i,j) only; masked = excluded
 *   LSE_i = ln sum_j exp(S_ij)                  (Definitions B.3, B.4: l = exp(S) 1)
 *   P_ij  = exp(S_ij - LSE_i)                   (Definition B.5: f = diag(l)^-1 exp(S))
 *   O     = P V                                 (Definition B.7; Definition 3.1)
 *   dP    = dO V^T                              (Definition B.8: q)
 *   D_i   = sum_c dO_ic O_ic                    (Definition B.9, second matrix form)
 *   dS    = P o (dP - D 1^T)                    (Definition B.9: p)
 *   dQ    = scale * dS K,  dK = scale * dS^T Q  (chain rule through Definition 3.2,
 *   dV    = P^T dO                               dL/dX = A1^T p A2, with Q = A1 X, K = A2)
 *
 * The paper's inputs A1 X, A2, A3 Y are the caller's Q, K, V: the projections sit
 * in front of this boundary (Section 3.1, remark on Q, K, V), and the 1/sqrt(d)
 * factor the paper folds into X is the explicit `scale`.
 *
 * Layout: Q, K, V, O, dO, dQ, dK, dV are [batch, heads, n, d] contiguous, d fastest,
 * element type `dt`; LSE is float [batch, heads, n], natural logarithm.  Base
 * pointers must be 16-byte aligned.  Outputs are overwritten, never accumulated into.
 * A query row with no kept key gets O = 0, LSE = -inf and contributes no gradient.
 *
 * Errors: argument errors are returned synchronously, before anything is enqueued.
 * Errors found by a kernel (a bounded wait that ran out) are written to the 4-byte
 * status word at the start of `workspace`; read it with attn_workspace_status().
 * A device that is not compute capability 10.x gets ATTN_ERR_ARCH: there is no
 * fallback path of any kind.
 */
#ifndef ATTN_B200_H
#define ATTN_B200_H

#include <stddef.h>
#include <stdint.h>

#ifdef __cplusplus
extern "C" {
#endif

typedef enum {
    ATTN_OK = 0,
    ATTN_ERR_NULL = 1,           /* a required pointer is NULL */
    ATTN_ERR_SHAPE = 2,          /* n, d, heads or batch out of the supported range */
    ATTN_ERR_DTYPE = 3,          /* unknown dtype, or dtype not supported by the chosen algorithm */
    ATTN_ERR_ALIGN = 4,          /* a base pointer is not 16-byte aligned */
    ATTN_ERR_TILE = 5,           /* tile_q / tile_k / tile_d not in attn_supported_cfgs() */
    ATTN_ERR_MASK = 6,           /* bad mask description */
    ATTN_ERR_WORKSPACE = 7,      /* workspace NULL or smaller than attn_*_workspace_bytes() */
    ATTN_ERR_ARCH = 8,           /* current device is not sm_100 */
    ATTN_ERR_LAUNCH = 9,         /* the CUDA runtime refused a launch or a tensor-map encode */
    ATTN_ERR_DEVICE_TIMEOUT = 10 /* a kernel gave up on a bounded wait (status word only) */
} attn_status;

typedef enum { ATTN_F32 = 0, ATTN_BF16 = 1 } attn_dtype;

typedef enum { ATTN_MASK_NONE = 0, ATTN_MASK_CAUSAL = 1, ATTN_MASK_BLOCK_SPARSE = 2,
               ATTN_MASK_BLOCK_SPARSE_CAUSAL = 3, ATTN_MASK_ELEMENT = 4 } attn_mask_kind;

/* Which (i, j) score entries are kept.  NULL means ATTN_MASK_NONE.
 *   CAUSAL:       keep j <= i (one n for queries and keys).
 *   BLOCK_SPARSE: keep (i, j) iff block_mask[h][i / block][j / block] != 0, where
 *                 block_mask is DEVICE uint8 [mask_heads][nb][nb], nb = ceil(n / block);
 *                 mask_heads is 1 (shared by every batch and head) or batch * heads.
 *                 The tensor-core algorithms need block to be a multiple of 128, or 64 or 32:
 *                 with the two fine sizes they visit every 128 x 128 tile that keeps at
 *                 least one block and drop the other blocks' entries inside the tile.
 *   BLOCK_SPARSE_CAUSAL: both at once -- keep (i, j) iff its block is kept and j <= i
 *                 (same fields as BLOCK_SPARSE; blocks above the diagonal are never visited).
 *   ELEMENT:      any set of kept entries, one bit each: block_mask points to a DEVICE bitmap of
 *                 32-bit words [mask_heads][n][ceil(n / 32)], bit (j % 32) of word j / 32 of row i
 *                 set iff (i, j) is kept; `block` is ignored.  attn_mask_from_coo() builds the
 *                 bitmap from a coordinate list, the form in which Section 4.1 stores a sparse
 *                 matrix.  FUSED and SIMT algorithms only; the tensor-core kernels visit the
 *                 128 x 128 tiles that keep at least one entry.
 * This is the sparse setting of Section 4.1 with Z_QK = the number of kept entries;
 * a masked score is minus infinity, not a stored zero. */
typedef struct {
    int kind;                  /* attn_mask_kind */
    int block;
    const uint8_t *block_mask; /* device */
    int mask_heads;
} attn_mask;

/* Which algorithm runs.  The tile sizes play the role of the paper's cache size M.
 *   FUSED        large-cache regime (Appendix D): score tiles never leave the SM.
 *   MATERIALIZED small-cache regime (Appendix C): P, dP and dS are written to and
 *                re-read from device memory in tile_q x tile_k blocks (tile_q 256 or 128,
 *                tile_k 128, 64 or 32; default 256 x 128), the head dimension walked in
 *                tile_d = 64 chunks (backward only; its forward is FUSED).
 *   SIMT         fp32 FMA kernels without tensor cores; the only choice for ATTN_F32.
 *   AUTO         ATTN_F32 -> SIMT; ATTN_BF16 -> FUSED.                              */
typedef enum { ATTN_ALGO_AUTO = 0, ATTN_ALGO_FUSED = 1, ATTN_ALGO_MATERIALIZED = 2, ATTN_ALGO_SIMT = 3 } attn_algo;

/* NULL or all zeros = defaults.  deterministic != 0 forbids floating-point atomics
 * (results are then bitwise repeatable run to run). */
typedef struct {
    int tile_q, tile_k, tile_d;
    int algo; /* attn_algo */
    int deterministic;
} attn_cfg;

/* Forward pass (Definition 3.1): writes O [batch,heads,n,d] and LSE [batch,heads,n].
 * n >= 1; d a multiple of 8 up to 256 (SIMT) or one of 64, 128, 256 (tensor-core
 * algorithms, which also need n to be a multiple of 8).  scale = 0 means 1/sqrt(d).
 * workspace: at least attn_fwd_workspace_bytes(), 256-byte aligned, device. */
attn_status attn_fwd(const void *Q, const void *K, const void *V, void *O, float *LSE,
                     int n, int d, int heads, int batch, const attn_mask *mask,
                     int dt /* attn_dtype */, float scale, const attn_cfg *cfg,
                     void *workspace, size_t workspace_bytes, void *cuda_stream);

/* Backward pass (Definitions B.8, B.9 and 3.2; Algorithm "large cache phase 2" with
 * dQ, dK, dV in place of the weight gradient): reads Q, K, V, dO and the forward's
 * O and LSE, writes dQ, dK, dV.  Same constraints as attn_fwd. */
attn_status attn_bwd(const void *Q, const void *K, const void *V, const void *O, const void *dO,
                     const float *LSE, void *dQ, void *dK, void *dV,
                     int n, int d, int heads, int batch, const attn_mask *mask,
                     int dt, float scale, const attn_cfg *cfg,
                     void *workspace, size_t workspace_bytes, void *cuda_stream);

/* D_i = sum_c dO_ic O_ic for `rows` rows of length d (the vector v of Definition B.9
 * and of the large-cache phase-2 algorithm).  D is float [rows].  attn_bwd runs this
 * itself; it is exported because it is the memory-bound step of the path. */
attn_status attn_bwd_preprocess(const void *O, const void *dO, float *D, size_t rows, int d, int dt,
                                void *cuda_stream);

/* ---- The attention weights (the paper's own inputs and gradient target) ------------
 *
 * Definition 3.1 writes the scores as A1 X A2^T and the values as A3 Y with d x d weight
 * matrices X (query and key weights folded into one) and Y; Definition 3.2 asks for
 * dL/dX = A1^T p A2.  With S = A1 X the library's Q is S, its K is A2, its V is h = A3 Y,
 * and dL/dS = attn_bwd's dQ, so dL/dX = A1^T dQ and dL/dY = A3^T dV.
 *
 * Tensors A, out, G: [batch, heads, n, d] like Q.  Weights W: [weight_units][d][d],
 * element (k, c) multiplies input feature k into output feature c; unit u = batch index *
 * heads + head uses matrix u mod weight_units, and weight_units is 1 (one matrix for
 * all units), heads (shared over the batch) or batch * heads.  d is a multiple of 8, at
 * most 256.  bf16 with d in {64, 128, 256} runs on the tensor cores, everything else on
 * fp32 FMAs.  `workspace` (device, 256-byte aligned, at least 256 bytes for the first two
 * calls) holds the status word that attn_workspace_status() reads.  All pointers are
 * caller-owned device memory, 16-byte aligned; the calls are asynchronous on cuda_stream. */

/* out = A W per unit: S = A1 X or h = A3 Y (Appendix D, phase 1 of the large-cache
 * algorithm).  out has the dtype of A and is fully overwritten. */
attn_status attn_project(const void *A, const void *W, void *out, int n, int d, int heads, int batch,
                         int weight_units, int dt, void *workspace, size_t workspace_bytes, void *cuda_stream);

/* g[w] = sum over the units u with u mod weight_units = w of A_u^T G_u, float
 * [weight_units][d][d], fully overwritten (Definition 3.2 with G = p A2; the last two
 * products of phase 2 of the large-cache algorithm, Appendix D).  The sum over units and
 * row tiles uses fp32 atomic adds: results vary in the last bits from run to run. */
attn_status attn_weight_grad(const void *A, const void *G, float *g, int n, int d, int heads, int batch,
                             int weight_units, int dt, void *workspace, size_t workspace_bytes, void *cuda_stream);

/* Phase 2 of the large-cache algorithm as a whole (Appendix D): from A1, A2, A3, the
 * projected S = A1 X and h = A3 Y, the forward's O and LSE (= ln l) and dO, computes
 * gX = dL/dX = A1^T p A2 (times `scale` when the scores carry one) and, unless gY is NULL
 * (the paper treats Y as fixed), gY = dL/dY = A3^T f^T dO.  Runs attn_bwd with Q = S,
 * K = A2, V = h into workspace buffers, then the two weight-gradient products; where the
 * backward accumulates dQ in fp32 (fused algorithm with atomics, bf16) gX is formed
 * from that accumulator and no bf16 copy of dQ is written.  mask, scale, cfg as in
 * attn_bwd; workspace of attn_weights_bwd_workspace_bytes() bytes. */
attn_status attn_weights_bwd(const void *A1, const void *A2, const void *A3, const void *S, const void *h,
                             const void *O, const void *dO, const float *LSE, float *gX, float *gY,
                             int n, int d, int heads, int batch, int weight_units, const attn_mask *mask,
                             int dt, float scale, const attn_cfg *cfg,
                             void *workspace, size_t workspace_bytes, void *cuda_stream);
size_t attn_weights_bwd_workspace_bytes(int n, int d, int heads, int batch, const attn_mask *mask, int dt,
                                        const attn_cfg *cfg);

/* attn_bwd for callers that cannot allocate device memory (the paper has no
 * counterpart: this is a convenience of the library, not a step of the method).
 *
 * Who needs it: code that is handed Q, K, V, O, dO, LSE and the output tensors but has
 * no allocator it may call at that moment -- a plug-in inside a framework whose memory
 * pool is frozen, a real-time loop that must not call cudaMalloc.
 * Such a caller cannot provide attn_bwd's `workspace`.  This entry point uses instead a
 * fixed scratch array of attn_noalloc_scratch_bytes() = 8 MiB that is part of the
 * library image (every GPU that loads the library holds these 8 MiB until the process
 * exits).  It calls no cudaMalloc / cudaFree and no allocating library routine.
 *
 *  - Same arguments, results and errors as attn_bwd, without workspace arguments.
 *  - Limit: attn_bwd_workspace_bytes() of the problem must not exceed 8 MiB (for the
 *    fused bf16 algorithm roughly batch*heads*n*d <= 2 Mi elements); larger problems
 *    get ATTN_ERR_WORKSPACE and must use attn_bwd.
 *  - The first call on each device looks up the array's device address (with that
 *    device current); make that first call before starting any stream capture.
 *  - All calls on a device share the one array and it keeps the previous call's
 *    contents; the parts that must start at zero are cleared by every call.  Two calls
 *    that overlap on the GPU (different streams, no ordering) race on it: serialise them.
 *  - Device-side errors (a bounded wait that ran out) land in the array's first word:
 *    attn_noalloc_status() synchronises `cuda_stream` and returns it, like
 *    attn_workspace_status() does for a caller-owned workspace; it allocates nothing either. */
attn_status attn_bwd_noalloc(const void *Q, const void *K, const void *V, const void *O, const void *dO,
                             const float *LSE, void *dQ, void *dK, void *dV,
                             int n, int d, int heads, int batch, const attn_mask *mask,
                             int dt, float scale, const attn_cfg *cfg, void *cuda_stream);
size_t attn_noalloc_scratch_bytes(void);
attn_status attn_noalloc_status(void *cuda_stream);

/* Workspace sizes in bytes for the same arguments (0 on invalid arguments). */
size_t attn_fwd_workspace_bytes(int n, int d, int heads, int batch, const attn_mask *mask, int dt,
                                const attn_cfg *cfg);
size_t attn_bwd_workspace_bytes(int n, int d, int heads, int batch, const attn_mask *mask, int dt,
                                const attn_cfg *cfg);

/* Synchronises `cuda_stream`, then returns the status word a kernel may have set in
 * `workspace` (ATTN_OK if none did). */
attn_status attn_workspace_status(const void *workspace, void *cuda_stream);

/* Tile configurations that attn_fwd / attn_bwd accept for (d, dt): fills up to
 * max_out entries of `out` (host), returns how many exist. */
int attn_supported_cfgs(int d, int dt, attn_cfg *out /* host */, int max_out);

/* On-chip elements (shared memory + tensor memory, counted in elements of the
 * operand type) one CTA of this configuration holds: the paper's M (Section 3.3
 * counts the cache in items).  0 on an unsupported configuration. */
size_t attn_cfg_onchip_elems(int d, int dt, const attn_cfg *cfg, int backward);

/* Closed-form I/O bounds, constant factor 1, in elements, per head.
 * backward != 0: min{(n^2 d^2 + n d^3)/M, (n^2 d + n d^2)/sqrt(M)} (Theorem 1.1);
 * backward == 0: min{n^2 d^2/M, n^2 d/sqrt(M)} (Table 1, forward). */
double attn_io_bound_elems(double n, double d, double M, int backward);
/* min{Z_input^2/M, Z_input sqrt(Z_QK)/sqrt(M)} (Theorem 1.2). */
double attn_io_bound_sparse_elems(double z_input, double z_qk, double M);

/* I/O of the library's own tilings in the same model (Section 3.3: a cache of M items in front of
 * a large memory; here the cache is one CTA's shared + tensor memory).  Replays on the host the loop
 * nest of the kernels that `cfg` selects for one head of n x d with the given mask (ATTN_MASK_NONE
 * or ATTN_MASK_CAUSAL) and counts the elements that cross the SM boundary: operand tiles loaded,
 * results stored, and fp32 partial sums added into memory (the fused backward's dQ).  Passes that
 * belong to the call are included (D pre-pass, accumulator clear and conversion, the materialised
 * path's P, dP, dS round trips).  The sum is what Theorem 1.1 bounds from below at
 * M = attn_cfg_onchip_elems(); comparing the two shows how close a tile shape is to the bound and
 * how the I/O falls as the tile -- the cache -- grows (Figure 1 of the introduction).  Host only.
 * The materialised backward can also be replayed at d = 512 and 1024 (multiples of 64), sizes no kernel of
 * the library runs: its blocks then hold fewer than d^2 elements, the small-cache side of Theorem 1.1. */
typedef struct { double loads, stores, reductions; } attn_io_count; /* elements, per head */
attn_status attn_io_replay(int n, int d, int mask_kind, int dt, const attn_cfg *cfg, int backward,
                           attn_io_count *out /* host */);

/* Builds the bitmap of an ATTN_MASK_ELEMENT mask from a coordinate list (Section 4.1 stores a sparse
 * matrix as the coordinates of its entries): clears `bitmap` (DEVICE, mask_heads * n * ceil(n / 32)
 * 32-bit words, 4-byte aligned) and sets the bit of every (rows[e], cols[e]) of mask heads[e], e < nnz.
 * rows, cols, heads: DEVICE int32 arrays of nnz entries; heads == NULL puts every entry into mask 0.
 * An entry whose row, column or head is out of range is ignored; duplicates are harmless.
 * Enqueued on cuda_stream; returns after validating the arguments. */
attn_status attn_mask_from_coo(const int *rows, const int *cols, const int *heads, size_t nnz, int n,
                               int mask_heads, uint32_t *bitmap, void *cuda_stream);

const char *attn_status_str(int status);

/* ---- diagnostics (process-wide state; not thread-safe; off by default) ----
 * attn_kernel_launches: kernels this library has launched since it was loaded.
 * attn_timing_enable(1): from now on every kernel launch is bracketed by two CUDA
 *   events recorded on the launching stream (a fixed pool of 256 launches; later
 *   launches go untimed until collected).  attn_timing_enable(0) releases the pool.
 * attn_timing_collect: synchronises on the recorded events, writes each launch's
 *   device time in milliseconds to ms[] and a pointer to its static kernel name to
 *   names[] (both host arrays of `max` entries), empties the pool and returns the
 *   number of launches written.  This is how a caller obtains per-kernel times for
 *   roofline arithmetic without a profiler. */
unsigned long long attn_kernel_launches(void);
attn_status attn_timing_enable(int on);
int attn_timing_collect(float *ms /* host */, const char **names /* host */, int max);

/* Self-test of the bounded waits (no counterpart in the paper): every wait inside the
 * tensor-core kernels gives up after a time limit, sets the workspace status word to
 * ATTN_ERR_DEVICE_TIMEOUT and lets the kernel run to its normal end.  This call enqueues
 * one warp that waits, for at most `limit_us` microseconds (1 .. 100000), on a barrier
 * nothing arrives at; afterwards attn_workspace_status(workspace) is
 * ATTN_ERR_DEVICE_TIMEOUT and the context is as usable as before.  workspace: device,
 * at least 256 bytes; its first two words are overwritten (word 1: bit 0 / bit 1 set if
 * the first / second wait wrongly reported success). */
attn_status attn_selftest_wait_timeout(void *workspace, size_t workspace_bytes, unsigned limit_us,
                                       void *cuda_stream);

#ifdef __cplusplus
}
#endif
#endif /* ATTN_B200_H */

// Host side of the tensor-core path: TMA tensor-map encoding through the driver entry
// point (the library does not link against libcuda, so it still loads on a machine
// without a driver), and the self-test of the bounded waits.
#include <cudaTypedefs.h>

#include "attn_internal.h"
#include "tc_common.cuh"

namespace attn {
namespace {

PFN_cuTensorMapEncodeTiled_v12000 encode_fn()
{
    static PFN_cuTensorMapEncodeTiled_v12000 fn = nullptr;
    if (!fn) {
        void *p = nullptr;
        cudaDriverEntryPointQueryResult q;
        if (cudaGetDriverEntryPoint("cuTensorMapEncodeTiled", &p, cudaEnableDefault, &q) == cudaSuccess &&
            q == cudaDriverEntryPointSuccess)
            fn = reinterpret_cast<PFN_cuTensorMapEncodeTiled_v12000>(p);
    }
    return fn;
}

}  // namespace

bool make_tmap_bf16_3d(CUtensorMap *out, const void *base, uint64_t dim0, uint64_t dim1, uint64_t dim2, uint32_t box1)
{
    auto fn = encode_fn();
    if (!fn) return false;
    cuuint64_t dims[3] = {dim0, dim1, dim2};
    cuuint64_t strides[2] = {dim0 * 2, dim0 * dim1 * 2};
    cuuint32_t box[3] = {64, box1, 1};
    cuuint32_t estr[3] = {1, 1, 1};
    return fn(out, CU_TENSOR_MAP_DATA_TYPE_BFLOAT16, 3, const_cast<void *>(base), dims, strides, box, estr,
              CU_TENSOR_MAP_INTERLEAVE_NONE, CU_TENSOR_MAP_SWIZZLE_128B, CU_TENSOR_MAP_L2_PROMOTION_L2_256B,
              CU_TENSOR_MAP_FLOAT_OOB_FILL_NONE) == CUDA_SUCCESS;
}

bool make_tmap_f32_3d(CUtensorMap *out, const void *base, uint64_t dim0, uint64_t dim1, uint64_t dim2, uint32_t box1)
{
    auto fn = encode_fn();
    if (!fn) return false;
    cuuint64_t dims[3] = {dim0, dim1, dim2};
    cuuint64_t strides[2] = {dim0 * 4, dim0 * dim1 * 4};
    cuuint32_t box[3] = {32, box1, 1};
    cuuint32_t estr[3] = {1, 1, 1};
    return fn(out, CU_TENSOR_MAP_DATA_TYPE_FLOAT32, 3, const_cast<void *>(base), dims, strides, box, estr,
              CU_TENSOR_MAP_INTERLEAVE_NONE, CU_TENSOR_MAP_SWIZZLE_128B, CU_TENSOR_MAP_L2_PROMOTION_L2_256B,
              CU_TENSOR_MAP_FLOAT_OOB_FILL_NONE) == CUDA_SUCCESS;
}

bool make_tmap_bf16_3d_box(CUtensorMap *out, const void *base, uint64_t dim0, uint64_t dim1, uint64_t dim2, uint64_t pitch_elems,
                           uint32_t box0, uint32_t box1, int swizzle_bytes)
{
    auto fn = encode_fn();
    if (!fn) return false;
    cuuint64_t dims[3] = {dim0, dim1, dim2};
    cuuint64_t strides[2] = {pitch_elems * 2, pitch_elems * dim1 * 2};
    cuuint32_t box[3] = {box0, box1, 1};
    cuuint32_t estr[3] = {1, 1, 1};
    return fn(out, CU_TENSOR_MAP_DATA_TYPE_BFLOAT16, 3, const_cast<void *>(base), dims, strides, box, estr,
              CU_TENSOR_MAP_INTERLEAVE_NONE, swizzle_bytes == 64 ? CU_TENSOR_MAP_SWIZZLE_64B : CU_TENSOR_MAP_SWIZZLE_128B,
              CU_TENSOR_MAP_L2_PROMOTION_L2_256B, CU_TENSOR_MAP_FLOAT_OOB_FILL_NONE) == CUDA_SUCCESS;
}

bool make_tmap_bf16_2d(CUtensorMap *out, const void *base, uint64_t cols, uint64_t rows, uint64_t pitch_bytes,
                       uint32_t box_rows)
{
    auto fn = encode_fn();
    if (!fn) return false;
    cuuint64_t dims[2] = {cols, rows};
    cuuint64_t strides[1] = {pitch_bytes};
    cuuint32_t box[2] = {64, box_rows};
    cuuint32_t estr[2] = {1, 1};
    return fn(out, CU_TENSOR_MAP_DATA_TYPE_BFLOAT16, 2, const_cast<void *>(base), dims, strides, box, estr,
              CU_TENSOR_MAP_INTERLEAVE_NONE, CU_TENSOR_MAP_SWIZZLE_128B, CU_TENSOR_MAP_L2_PROMOTION_L2_256B,
              CU_TENSOR_MAP_FLOAT_OOB_FILL_NONE) == CUDA_SUCCESS;
}

// One warp waits, under `limit_ns`, on a barrier that nothing ever arrives at: the wait runs out, the status
// word is set and the kernel returns normally.  Exercises the bounded-wait path of the tensor-core kernels.
__global__ void wait_timeout_selftest_kernel(uint32_t *status, unsigned long long limit_ns, uint32_t *waited_ok)
{
    __shared__ uint64_t bar;
    __shared__ uint32_t flag;
    if (threadIdx.x == 0) {
        flag = 0;
        tc::mbar_init(&bar, 1);
        tc::fence_barrier_init();
    }
    __syncthreads();
    const tc::Abort ab{&flag, status, limit_ns};
    const bool done = tc::mbar_wait(&bar, 0, ab);        // phase 0 never completes
    const bool again = tc::mbar_wait(&bar, 0, ab);       // after an abort, later waits return at once
    if (threadIdx.x == 0) *waited_ok = (done ? 1u : 0u) | (again ? 2u : 0u);
}

}  // namespace attn

extern "C" attn_status attn_selftest_wait_timeout(void *workspace, size_t workspace_bytes, unsigned limit_us,
                                                  void *cuda_stream)
{
    if (!workspace) return ATTN_ERR_NULL;
    if (workspace_bytes < 256 || limit_us == 0 || limit_us > 100000) return ATTN_ERR_WORKSPACE;
    uint32_t *w = static_cast<uint32_t *>(workspace);
    cudaStream_t s = static_cast<cudaStream_t>(cuda_stream);
    if (cudaMemsetAsync(w, 0, 8, s) != cudaSuccess) return ATTN_ERR_LAUNCH;
    attn::launch_begin("selftest_wait_timeout", s);
    attn::wait_timeout_selftest_kernel<<<1, 32, 0, s>>>(w, (unsigned long long)limit_us * 1000ull, w + 1);
    attn::launch_end(s);
    return cudaGetLastError() == cudaSuccess ? ATTN_OK : ATTN_ERR_LAUNCH;
}

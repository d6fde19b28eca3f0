// One-time set-up of the tensor-core path: the driver entry point that encodes tensor maps, and the
// per-device shared-memory opt-in of every kernel.
#include <mutex>

#include "tensor_common.cuh"

namespace {

typedef CUresult (*EncodeTiledFn)(CUtensorMap*, CUtensorMapDataType, cuuint32_t, void*, const cuuint64_t*,
                                  const cuuint64_t*, const cuuint32_t*, const cuuint32_t*, CUtensorMapInterleave,
                                  CUtensorMapSwizzle, CUtensorMapL2promotion, CUtensorMapFloatOOBfill);
EncodeTiledFn g_encode = nullptr;
std::once_flag g_once;
cudaError_t g_init_err = cudaSuccess;

}  // namespace

bool as_tc::make_map(CUtensorMap* m, const void* base, int cols, int rows, int slices, int box_rows) {
  if (g_encode == nullptr) return false;
  cuuint64_t dims[3] = {(cuuint64_t)cols, (cuuint64_t)rows, (cuuint64_t)slices};
  cuuint64_t strides[2] = {(cuuint64_t)cols * 2, (cuuint64_t)cols * 2 * (cuuint64_t)rows};
  cuuint32_t box[3] = {64u, (cuuint32_t)box_rows, 1u};
  cuuint32_t estr[3] = {1u, 1u, 1u};
  return g_encode(m, CU_TENSOR_MAP_DATA_TYPE_BFLOAT16, 3, const_cast<void*>(base), dims, strides, box, estr,
                  CU_TENSOR_MAP_INTERLEAVE_NONE, CU_TENSOR_MAP_SWIZZLE_128B, CU_TENSOR_MAP_L2_PROMOTION_L2_256B,
                  CU_TENSOR_MAP_FLOAT_OOB_FILL_NONE) == CUDA_SUCCESS;
}

namespace {

// One CTA whose threads wait, with the kernels' own bounded wait, on an mbarrier that nobody arrives at.  No
// copy and no MMA is in flight: when the limit has passed the wait gives up, raises the status bit and the
// kernel returns.
__global__ void expire_wait_kernel(uint32_t* status, long long limit_cycles) {
  __shared__ uint64_t bar;
  __shared__ uint32_t abort_flag;
  if (threadIdx.x == 0) {
    abort_flag = 0u;
    sm100::mbar_init(sm100::smem_u32(&bar), 1);
    sm100::fence_barrier_init();
  }
  __syncthreads();
  const sm100::WaitCtx wc{status, &abort_flag};
  sm100::mbar_wait_limit(sm100::smem_u32(&bar), 0, wc, limit_cycles);
}

}  // namespace

cudaError_t as_tensor_expire_wait(uint32_t* status, long long limit_cycles, cudaStream_t st) {
  expire_wait_kernel<<<1, 64, 0, st>>>(status, limit_cycles);
  return cudaGetLastError();
}

cudaError_t as_tensor_init() {
  std::call_once(g_once, [] {
    void* fn = nullptr;
    cudaDriverEntryPointQueryResult q;
    cudaError_t e = cudaGetDriverEntryPoint("cuTensorMapEncodeTiled", &fn, cudaEnableDefault, &q);
    if (e != cudaSuccess || q != cudaDriverEntryPointSuccess || fn == nullptr) {
      g_init_err = (e != cudaSuccess) ? e : cudaErrorNotSupported;
      return;
    }
    g_encode = reinterpret_cast<EncodeTiledFn>(fn);
  });
  if (g_init_err != cudaSuccess) return g_init_err;
  // shared-memory opt-in is per device; cheap enough to repeat
  cudaError_t e;
  if ((e = as_tensor_init_qpass()) != cudaSuccess) return e;
  if ((e = as_tensor_init_kpass()) != cudaSuccess) return e;
  return as_tensor_init_qstream();
}

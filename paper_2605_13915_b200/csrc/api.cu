// Status strings, the device status word, workspace initialisation and tensor-map encoding.
#include <mutex>

#include "host_common.h"
#include "sm100.cuh"

namespace msd {

__device__ unsigned g_status_word[4];

unsigned* device_status_ptr() {
  static std::mutex mu;
  static unsigned* cache[64] = {};
  int dev = 0;
  if (cudaGetDevice(&dev) != cudaSuccess || dev < 0 || dev >= 64) return nullptr;
  std::lock_guard<std::mutex> lock(mu);
  if (!cache[dev]) {
    void* p = nullptr;
    if (cudaGetSymbolAddress(&p, g_status_word) != cudaSuccess) return nullptr;
    cache[dev] = static_cast<unsigned*>(p);
  }
  return cache[dev];
}

int sm_count() {
  static int cache[64] = {};
  int dev = 0;
  if (cudaGetDevice(&dev) != cudaSuccess || dev < 0 || dev >= 64) return 148;
  if (!cache[dev]) {
    int n = 0;
    if (cudaDeviceGetAttribute(&n, cudaDevAttrMultiProcessorCount, dev) != cudaSuccess || n <= 0) n = 148;
    cache[dev] = n;
  }
  return cache[dev];
}

using EncodeFn = CUresult (*)(CUtensorMap*, CUtensorMapDataType, cuuint32_t, void*, const cuuint64_t*, const cuuint64_t*,
                              const cuuint32_t*, const cuuint32_t*, CUtensorMapInterleave, CUtensorMapSwizzle,
                              CUtensorMapL2promotion, CUtensorMapFloatOOBfill);

static EncodeFn encode_fn() {
  static EncodeFn fn = nullptr;
  static std::once_flag once;
  std::call_once(once, [] {
    void* p = nullptr;
    cudaDriverEntryPointQueryResult q;
    if (cudaGetDriverEntryPoint("cuTensorMapEncodeTiled", &p, cudaEnableDefault, &q) == cudaSuccess &&
        q == cudaDriverEntryPointSuccess)
      fn = reinterpret_cast<EncodeFn>(p);
  });
  return fn;
}

bool encode_tmap_2d(CUtensorMap* out, CUtensorMapDataType dtype, const void* base, uint64_t inner, uint64_t outer,
                    uint64_t row_stride_bytes, uint32_t box_inner, uint32_t box_outer, CUtensorMapSwizzle swizzle) {
  EncodeFn fn = encode_fn();
  if (!fn) return false;
  cuuint64_t dims[2] = {inner, outer};
  cuuint64_t strides[1] = {row_stride_bytes};
  cuuint32_t box[2] = {box_inner, box_outer};
  cuuint32_t estr[2] = {1, 1};
  return fn(out, dtype, 2, const_cast<void*>(base), dims, strides, box, estr, CU_TENSOR_MAP_INTERLEAVE_NONE, swizzle,
            CU_TENSOR_MAP_L2_PROMOTION_L2_256B, CU_TENSOR_MAP_FLOAT_OOB_FILL_NONE) == CUDA_SUCCESS;
}

bool encode_tmap_3d(CUtensorMap* out, CUtensorMapDataType dtype, const void* base, uint64_t d0, uint64_t d1, uint64_t d2,
                    uint64_t stride1_bytes, uint64_t stride2_bytes, uint32_t b0, uint32_t b1, uint32_t b2,
                    CUtensorMapSwizzle swizzle) {
  EncodeFn fn = encode_fn();
  if (!fn) return false;
  cuuint64_t dims[3] = {d0, d1, d2};
  cuuint64_t strides[2] = {stride1_bytes, stride2_bytes};
  cuuint32_t box[3] = {b0, b1, b2};
  cuuint32_t estr[3] = {1, 1, 1};
  return fn(out, dtype, 3, const_cast<void*>(base), dims, strides, box, estr, CU_TENSOR_MAP_INTERLEAVE_NONE, swizzle,
            CU_TENSOR_MAP_L2_PROMOTION_L2_256B, CU_TENSOR_MAP_FLOAT_OOB_FILL_NONE) == CUDA_SUCCESS;
}

}  // namespace msd

namespace msd {
// Exercises the give-up path of the bounded waits without harming anything: one warp waits on a barrier that nobody
// ever arrives on, with a short cycle budget; when it runs out the wait records MSD_ERR_TIMEOUT in the status word,
// raises the CTA's abort flag (which the second warp, waiting with the full budget, sees at once) and the kernel ends.
__global__ void timeout_selftest_kernel(unsigned* status, long long budget) {
  __shared__ __align__(8) uint64_t never;
  __shared__ int abort_flag;
  if (threadIdx.x == 0) {
    mbar_init(&never, 1);
    abort_flag = 0;
    mbar_init_fence();
  }
  __syncthreads();
  volatile int* abort = &abort_flag;
  if (threadIdx.x < 32) wait_bounded_cycles(&never, 0, abort, status, budget);
  else wait_bounded(&never, 0, abort, status);
}
}  // namespace msd

extern "C" {

const char* msd_status_string(msd_status_t s) {
  switch (s) {
    case MSD_OK: return "ok";
    case MSD_ERR_NULL_POINTER: return "null pointer";
    case MSD_ERR_BAD_SHAPE: return "bad shape";
    case MSD_ERR_BAD_ALIGNMENT: return "bad alignment";
    case MSD_ERR_UNSUPPORTED: return "unsupported";
    case MSD_ERR_WORKSPACE_TOO_SMALL: return "workspace too small";
    case MSD_ERR_CUDA: return "CUDA error";
    case MSD_ERR_TIMEOUT: return "device-side wait timed out";
  }
  return "unknown status";
}

msd_status_t msd_last_device_status(void* stream) {
  unsigned* p = msd::device_status_ptr();
  if (!p) return MSD_ERR_CUDA;
  cudaStream_t s = static_cast<cudaStream_t>(stream);
  if (cudaStreamSynchronize(s) != cudaSuccess) return MSD_ERR_CUDA;
  unsigned v = 0;
  if (cudaMemcpyAsync(&v, p, sizeof(v), cudaMemcpyDeviceToHost, s) != cudaSuccess) return MSD_ERR_CUDA;
  if (cudaStreamSynchronize(s) != cudaSuccess) return MSD_ERR_CUDA;
  if (v != 0) {
    if (cudaMemsetAsync(p, 0, sizeof(unsigned), s) != cudaSuccess) return MSD_ERR_CUDA;
    if (cudaStreamSynchronize(s) != cudaSuccess) return MSD_ERR_CUDA;
  }
  return v == 0 ? MSD_OK : (v == MSD_ERR_TIMEOUT ? MSD_ERR_TIMEOUT : MSD_ERR_CUDA);
}

msd_status_t msd_debug_timeout_selftest(int64_t budget_cycles, void* stream) {
  unsigned* p = msd::device_status_ptr();
  if (!p) return MSD_ERR_CUDA;
  if (budget_cycles < 1000) budget_cycles = 1000;
  if (budget_cycles > 200000000LL) budget_cycles = 200000000LL;      // a tenth of a second at most
  msd::timeout_selftest_kernel<<<1, 64, 0, static_cast<cudaStream_t>(stream)>>>(p, static_cast<long long>(budget_cycles));
  return msd::launch_status();
}

msd_status_t msd_workspace_init(void* workspace, size_t workspace_bytes, void* stream) {
  if (!workspace && workspace_bytes) return MSD_ERR_NULL_POINTER;
  if (workspace_bytes == 0) return MSD_OK;
  return cudaMemsetAsync(workspace, 0, workspace_bytes, static_cast<cudaStream_t>(stream)) == cudaSuccess ? MSD_OK
                                                                                                             : MSD_ERR_CUDA;
}

}  // extern "C"

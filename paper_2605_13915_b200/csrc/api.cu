// Status strings, the device status word, workspace initialisation and tensor-map encoding.
#include <atomic>
#include <cstdlib>
#include <cstring>
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
  static std::atomic<int> cache[64] = {};
  int dev = 0;
  if (cudaGetDevice(&dev) != cudaSuccess || dev < 0 || dev >= 64) return 148;
  if (!cache[dev]) {
    int n = 0;
    if (cudaDeviceGetAttribute(&n, cudaDevAttrMultiProcessorCount, dev) != cudaSuccess || n <= 0) n = 148;
    cache[dev] = n;
  }
  return cache[dev];
}

static const char* const kOptionNames[OPT_COUNT] = {
    "MSD_NO_PDL", "MSD_GEMM_MODE", "MSD_GEMM_CTAS", "MSD_P8_PAIR", "MSD_P8_KSPLIT", "MSD_W4_PAIR", "MSD_W4_TILEN", "MSD_W4_KSPLIT",
    "MSD_ATTN_SPLITS", "MSD_ATTN_CHUNK_TILES", "MSD_ATTN_BALANCED"};
static int g_options[OPT_COUNT];
static std::mutex g_options_mu;
static bool g_options_read = false;

static void read_options_locked() {
  for (int i = 0; i < OPT_COUNT; ++i) {
    const char* e = getenv(kOptionNames[i]);
    g_options[i] = (e && *e) ? atoi(e) : -1;
  }
  g_options_read = true;
}

int option(Option o) {
  std::lock_guard<std::mutex> lock(g_options_mu);
  if (!g_options_read) read_options_locked();
  return g_options[o];
}

// returns false for an unknown name
static bool set_option(const char* name, int value) {
  std::lock_guard<std::mutex> lock(g_options_mu);
  if (!g_options_read) read_options_locked();
  for (int i = 0; i < OPT_COUNT; ++i)
    if (strcmp(name, kOptionNames[i]) == 0) { g_options[i] = value; return true; }
  return false;
}

static void reset_options() {
  std::lock_guard<std::mutex> lock(g_options_mu);
  read_options_locked();
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

// Encoded tensor maps are kept in a small direct-mapped cache keyed by everything that goes into them: a serving loop
// calls with the same buffers and shapes over and over, and an encode costs a microsecond or two of host time.
struct TmapKey {
  int dtype, rank, swizzle;
  const void* base;
  uint64_t dims[3], strides[2];
  uint32_t box[3];
  bool operator==(const TmapKey& o) const {
    return dtype == o.dtype && rank == o.rank && swizzle == o.swizzle && base == o.base && dims[0] == o.dims[0] &&
           dims[1] == o.dims[1] && dims[2] == o.dims[2] && strides[0] == o.strides[0] && strides[1] == o.strides[1] &&
           box[0] == o.box[0] && box[1] == o.box[1] && box[2] == o.box[2];
  }
};
constexpr int kTmapCacheSlots = 256;
struct TmapSlot { bool used; TmapKey key; CUtensorMap map; };
static TmapSlot g_tmap_cache[kTmapCacheSlots];
static std::mutex g_tmap_mu;

static bool encode_cached(CUtensorMap* out, const TmapKey& k) {
  uint64_t h = reinterpret_cast<uintptr_t>(k.base) * 0x9E3779B97F4A7C15ull;
  h ^= (k.dims[0] * 31 + k.dims[1]) * 0xC2B2AE3D27D4EB4Full + k.dims[2] * 131 + k.box[0] * 7 + k.box[1] * 3 + k.box[2] + k.strides[0] +
       static_cast<uint64_t>(k.swizzle) * 17 + static_cast<uint64_t>(k.dtype);
  TmapSlot& slot = g_tmap_cache[(h >> 20) % kTmapCacheSlots];
  {
    std::lock_guard<std::mutex> lock(g_tmap_mu);
    if (slot.used && slot.key == k) { *out = slot.map; return true; }
  }
  EncodeFn fn = encode_fn();
  if (!fn) return false;
  cuuint64_t dims[3] = {k.dims[0], k.dims[1], k.dims[2]};
  cuuint64_t strides[2] = {k.strides[0], k.strides[1]};
  cuuint32_t box[3] = {k.box[0], k.box[1], k.box[2]};
  cuuint32_t estr[3] = {1, 1, 1};
  if (fn(out, static_cast<CUtensorMapDataType>(k.dtype), static_cast<cuuint32_t>(k.rank), const_cast<void*>(k.base), dims, strides, box,
         estr, CU_TENSOR_MAP_INTERLEAVE_NONE, static_cast<CUtensorMapSwizzle>(k.swizzle), CU_TENSOR_MAP_L2_PROMOTION_L2_256B,
         CU_TENSOR_MAP_FLOAT_OOB_FILL_NONE) != CUDA_SUCCESS)
    return false;
  std::lock_guard<std::mutex> lock(g_tmap_mu);
  slot.used = true;
  slot.key = k;
  slot.map = *out;
  return true;
}

bool encode_tmap_2d(CUtensorMap* out, CUtensorMapDataType dtype, const void* base, uint64_t inner, uint64_t outer,
                    uint64_t row_stride_bytes, uint32_t box_inner, uint32_t box_outer, CUtensorMapSwizzle swizzle) {
  TmapKey k = {};
  k.dtype = static_cast<int>(dtype); k.rank = 2; k.swizzle = static_cast<int>(swizzle); k.base = base;
  k.dims[0] = inner; k.dims[1] = outer; k.strides[0] = row_stride_bytes; k.box[0] = box_inner; k.box[1] = box_outer;
  return encode_cached(out, k);
}

bool encode_tmap_3d(CUtensorMap* out, CUtensorMapDataType dtype, const void* base, uint64_t d0, uint64_t d1, uint64_t d2,
                    uint64_t stride1_bytes, uint64_t stride2_bytes, uint32_t b0, uint32_t b1, uint32_t b2,
                    CUtensorMapSwizzle swizzle) {
  TmapKey k = {};
  k.dtype = static_cast<int>(dtype); k.rank = 3; k.swizzle = static_cast<int>(swizzle); k.base = base;
  k.dims[0] = d0; k.dims[1] = d1; k.dims[2] = d2; k.strides[0] = stride1_bytes; k.strides[1] = stride2_bytes;
  k.box[0] = b0; k.box[1] = b1; k.box[2] = b2;
  return encode_cached(out, k);
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
  return v == 0 ? MSD_OK : (v == MSD_ERR_TIMEOUT ? MSD_ERR_TIMEOUT : (v == MSD_ERR_BAD_SHAPE ? MSD_ERR_BAD_SHAPE : MSD_ERR_CUDA));
}

msd_status_t msd_debug_timeout_selftest(int64_t budget_cycles, void* stream) {
  unsigned* p = msd::device_status_ptr();
  if (!p) return MSD_ERR_CUDA;
  if (budget_cycles < 1000) budget_cycles = 1000;
  if (budget_cycles > 200000000LL) budget_cycles = 200000000LL;      // a tenth of a second at most
  msd::timeout_selftest_kernel<<<1, 64, 0, static_cast<cudaStream_t>(stream)>>>(p, static_cast<long long>(budget_cycles));
  return msd::launch_status();
}

msd_status_t msd_debug_set_option(const char* name, int32_t value) {
  if (!name) return MSD_ERR_NULL_POINTER;
  return msd::set_option(name, value) ? MSD_OK : MSD_ERR_UNSUPPORTED;
}

void msd_debug_reset_options(void) { msd::reset_options(); }

msd_status_t msd_workspace_init(void* workspace, size_t workspace_bytes, void* stream) {
  if (!workspace && workspace_bytes) return MSD_ERR_NULL_POINTER;
  if (workspace_bytes == 0) return MSD_OK;
  return cudaMemsetAsync(workspace, 0, workspace_bytes, static_cast<cudaStream_t>(stream)) == cudaSuccess ? MSD_OK
                                                                                                             : MSD_ERR_CUDA;
}

}  // extern "C"

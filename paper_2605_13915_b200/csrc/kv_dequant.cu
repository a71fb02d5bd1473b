// The step the MSD attention removes (Sec. 2.3 / Sec. 6.4 "Dequant"): an INT8 KV cache with one scale per token and KV
// head is expanded to BF16 in memory, bf16(s * q), before a BF16 attention kernel reads it.  Kept as a comparison
// kernel only: 1 byte read and 2 bytes written per element on top of the 2 bytes per element the attention then reads.
#include <cuda_bf16.h>

#include "host_common.h"

namespace msd {

__global__ void __launch_bounds__(256)
kv_dequant_bf16_kernel(const int8_t* __restrict__ cache, const float* __restrict__ scale, int64_t rows, int D,
                       __nv_bfloat16* __restrict__ out) {
  const int chunks_per_row = D >> 4;          // 16 codes per thread and step
  const int64_t total = rows * chunks_per_row;
  for (int64_t i = static_cast<int64_t>(blockIdx.x) * blockDim.x + threadIdx.x; i < total;
       i += static_cast<int64_t>(gridDim.x) * blockDim.x) {
    const int64_t row = i / chunks_per_row;   // (token, head) pair
    const float s = __ldg(scale + row);
    const uint4 v = __ldg(reinterpret_cast<const uint4*>(cache) + i);
    const uint32_t w[4] = {v.x, v.y, v.z, v.w};
    uint32_t o[8];
#pragma unroll
    for (int j = 0; j < 8; ++j) {
      const int b0 = static_cast<int8_t>((w[j >> 1] >> (16 * (j & 1))) & 0xFF);
      const int b1 = static_cast<int8_t>((w[j >> 1] >> (16 * (j & 1) + 8)) & 0xFF);
      const __nv_bfloat162 h = __floats2bfloat162_rn(s * static_cast<float>(b0), s * static_cast<float>(b1));
      o[j] = *reinterpret_cast<const uint32_t*>(&h);
    }
    uint4* dst = reinterpret_cast<uint4*>(out) + 2 * i;
    dst[0] = make_uint4(o[0], o[1], o[2], o[3]);
    dst[1] = make_uint4(o[4], o[5], o[6], o[7]);
  }
}

}  // namespace msd

extern "C" msd_status_t msd_kv_dequant_bf16(const int8_t* cache, const float* scale, int64_t T, int32_t H, int32_t D,
                                            void* out_bf16, void* stream) {
  using namespace msd;
  if (T < 0 || H < 1 || D < 16 || D % 16 != 0) return MSD_ERR_BAD_SHAPE;
  if (T == 0) return MSD_OK;
  if (!cache || !scale || !out_bf16) return MSD_ERR_NULL_POINTER;
  if (!aligned(cache, 16) || !aligned(out_bf16, 16) || !aligned(scale, 4)) return MSD_ERR_BAD_ALIGNMENT;
  const int64_t total = T * H * (D >> 4);
  int64_t blocks = (total + 255) / 256;
  const int64_t cap = static_cast<int64_t>(sm_count()) * 16;
  if (blocks > cap) blocks = cap;
  kv_dequant_bf16_kernel<<<static_cast<unsigned>(blocks), 256, 0, static_cast<cudaStream_t>(stream)>>>(
      cache, scale, T * H, D, static_cast<__nv_bfloat16*>(out_bf16));
  return launch_status();
}

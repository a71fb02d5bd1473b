// Online activation decomposition kernels.
//   INT8  (Sec. 3.2, Eqs. alpha..x2; Alg. 1 lines 1-5): one CTA per row, 128-bit BF16 loads, warp-shuffle
//          row maximum, IEEE FP32 division + round-half-to-even, packed 128-bit INT8 stores.
//   MXFP4 (Sec. 3.2.1, Alg. 2, on the E2M1 grid): one thread per 32-element block - the block maximum needs
//          no cross-thread reduction and beta follows from alpha by a shift.
#include <cuda_bf16.h>
#include <cuda_fp4.h>

#include <cstdlib>

#include "host_common.h"
#include "quant.cuh"
#include "sm100.cuh"

namespace msd {

// 256 threads x 64 registers leave room for a CTA of the dependent GEMM (192 threads x ~224 registers) on the same SM,
// so that GEMM can start prefetching weights everywhere while this kernel still runs.
constexpr int kDecCache = 4;   // 16-element chunks a thread keeps in registers between the two passes (K <= 16384)


template <int kDecThreads>
__global__ void __launch_bounds__(kDecThreads)
decompose_int8_kernel(const uint16_t* __restrict__ x, int64_t ldx, int K, int8_t* __restrict__ q1,
                      int8_t* __restrict__ q2, float* __restrict__ alpha_out, float* __restrict__ beta_out,
                      float c1, float c2) {
  // the GEMM launched behind this kernel as its programmatic dependent may become resident now and prefetch weights
  pdl_launch_dependents();
  const int row = blockIdx.x;
  const uint4* xr = reinterpret_cast<const uint4*>(x + static_cast<int64_t>(row) * ldx);
  const int nchunks = K >> 4;
  uint4 ca[kDecCache], cb[kDecCache];
  float m = 0.0f;
#pragma unroll
  for (int j = 0; j < kDecCache; ++j) {
    const int c = threadIdx.x + j * kDecThreads;
    if (c < nchunks) {
      ca[j] = __ldg(xr + 2 * c);
      cb[j] = __ldg(xr + 2 * c + 1);
      m = fmaxf(m, chunk_absmax(ca[j], cb[j]));
    }
  }
  for (int c = threadIdx.x + kDecCache * kDecThreads; c < nchunks; c += kDecThreads)
    m = fmaxf(m, chunk_absmax(__ldg(xr + 2 * c), __ldg(xr + 2 * c + 1)));

  __shared__ float warp_max[kDecThreads / 32];
#pragma unroll
  for (int o = 16; o > 0; o >>= 1) m = fmaxf(m, __shfl_xor_sync(0xffffffffu, m, o));
  if ((threadIdx.x & 31) == 0) warp_max[threadIdx.x >> 5] = m;
  __syncthreads();
  m = warp_max[0];
#pragma unroll
  for (int w = 1; w < kDecThreads / 32; ++w) m = fmaxf(m, warp_max[w]);

  const float alpha = __fdiv_rn(m, c1);            // Eq. alpha (c1 = 127, or 127.49 with fractional scaling, Sec. 3.3)
  const float beta = __fdiv_rn(alpha, c2);         // Eq. beta  (c2 = 254, or 254.98)
  // reciprocals only steer the fast path of quant_i8; infinities (tiny scales) simply send every element to the division
  const float inv_alpha = alpha > 0.0f ? __frcp_rn(alpha) : 0.0f;
  const float inv_beta = beta > 0.0f ? __frcp_rn(beta) : 0.0f;
  if (threadIdx.x == 0) {
    alpha_out[row] = alpha;
    beta_out[row] = beta;
  }
  uint4* o1 = reinterpret_cast<uint4*>(q1 + static_cast<int64_t>(row) * K);
  uint4* o2 = reinterpret_cast<uint4*>(q2 + static_cast<int64_t>(row) * K);
#pragma unroll
  for (int j = 0; j < kDecCache; ++j) {
    const int c = threadIdx.x + j * kDecThreads;
    if (c < nchunks) {
      uint4 r1, r2;
      chunk_quantize(ca[j], cb[j], alpha, beta, inv_alpha, inv_beta, r1, r2);
      o1[c] = r1;
      o2[c] = r2;
    }
  }
  for (int c = threadIdx.x + kDecCache * kDecThreads; c < nchunks; c += kDecThreads) {
    uint4 r1, r2;
    chunk_quantize(__ldg(xr + 2 * c), __ldg(xr + 2 * c + 1), alpha, beta, inv_alpha, inv_beta, r1, r2);
    o1[c] = r1;
    o2[c] = r2;
  }
}

// ---- MXFP4 ------------------------------------------------------------------------------------------------------
constexpr int kMxThreads = 256;

// 2^e as an FP32 number for e in [-126, 127]
__device__ __forceinline__ float pow2f(int e) { return __uint_as_float(static_cast<uint32_t>(e + 127) << 23); }

// The first `rl.blocks` CTAs do the (independent) scale relayout `rl`, the others the decomposition, 256 consecutive
// 32-element blocks (row-major) per CTA and round.
__global__ void __launch_bounds__(kMxThreads)
decompose_mxfp4_kernel(const uint16_t* __restrict__ x, int64_t ldx, int64_t M, int K, uint8_t* __restrict__ q1,
                       uint8_t* __restrict__ q2, uint8_t* __restrict__ e1, uint8_t* __restrict__ e2, int sf_kgroups,
                       const SfRelayout rl, const RowGroups rg) {
  pdl_launch_dependents();
  const int kblocks = K >> 5;
  const int64_t nblocks = M * kblocks;
  if (static_cast<int>(blockIdx.x) < rl.blocks) {
    __shared__ uint32_t sm_rl[kSfRelayoutSmemWords];
    sf_relayout(rl, blockIdx.x, rl.blocks, sm_rl);
    return;
  }
  const int64_t units = (nblocks + kMxThreads - 1) / kMxThreads;
  // whole warps of valid blocks and word-aligned scale positions (the scale arrays are then 4-byte aligned as well)
  const bool pack4 = (kblocks & 3) == 0 && ((reinterpret_cast<uintptr_t>(e1) | reinterpret_cast<uintptr_t>(e2)) & 3) == 0;
  for (int64_t u = blockIdx.x - rl.blocks; u < units; u += gridDim.x - rl.blocks) {
    const int64_t b = u * kMxThreads + threadIdx.x;
    const unsigned lanes = __ballot_sync(0xffffffffu, b < nblocks);      // the lanes of this warp that have a block
    if (b < nblocks) {
    const int64_t row_in = b / kblocks;
    const int kb = static_cast<int>(b - row_in * kblocks);
    const uint4* src = reinterpret_cast<const uint4*>(x + row_in * ldx + kb * 32);
    int64_t row = row_in;                   // where the row's components and scales go
    if (rg.n > 0) {
      int g = 0;
      while (g + 1 < rg.n && row_in >= rg.off[g + 1]) ++g;
      row = static_cast<int64_t>(g) * 128 + (row_in - rg.off[g]);
    }
    uint32_t w[16];
#pragma unroll
    for (int i = 0; i < 4; ++i) {
      const uint4 t = __ldg(src + i);
      w[4 * i] = t.x; w[4 * i + 1] = t.y; w[4 * i + 2] = t.z; w[4 * i + 3] = t.w;
    }
    uint32_t m2 = 0;       // maximum of |x| as BF16 bits (monotone in the value for finite inputs), both halves at once
#pragma unroll
    for (int i = 0; i < 16; ++i) m2 = __vmaxu2(m2, w[i] & 0x7FFF7FFFu);
    const uint32_t mbits = max(m2 & 0xFFFFu, m2 >> 16);
    const int expf = static_cast<int>(mbits >> 7);
    int a = -123;
    if (expf > 0) a = max(-123, (expf - 127) - 2 + (((mbits & 0x7Fu) > 0x10u) ? 1 : 0));
    a = min(a, 127);
    const int bexp = a - 4;                                   // beta = alpha / 16
    // x / alpha and r / beta are exact multiplications by a power of two: a is in [-123, 126] for finite BF16 inputs
    // (largest exponent 127, minus 2, plus at most 1), so 2^-a and 2^(4-a) are normal FP32 numbers
    const float sa = pow2f(max(-a, -126)), sb = pow2f(-bexp);
    const float alpha = pow2f(a);
    uint32_t o1[4] = {0, 0, 0, 0}, o2[4] = {0, 0, 0, 0};
#pragma unroll
    for (int i = 0; i < 16; ++i) {
      const float v0 = bf16lo(w[i]), v1 = bf16hi(w[i]);
      const __nv_fp4x2_storage_t c1 =
          __nv_cvt_float2_to_fp4x2(make_float2(v0 * sa, v1 * sa), __NV_E2M1, cudaRoundNearest);
      const float2 d1 = __half22float2(__half2(__nv_cvt_fp4x2_to_halfraw2(c1, __NV_E2M1)));
      const float r0 = __fmaf_rn(-alpha, d1.x, v0), r1 = __fmaf_rn(-alpha, d1.y, v1);   // exact residuals
      const __nv_fp4x2_storage_t c2 =
          __nv_cvt_float2_to_fp4x2(make_float2(r0 * sb, r1 * sb), __NV_E2M1, cudaRoundNearest);
      o1[i >> 2] |= static_cast<uint32_t>(c1) << (8 * (i & 3));
      o2[i >> 2] |= static_cast<uint32_t>(c2) << (8 * (i & 3));
    }
    *reinterpret_cast<uint4*>(q1 + row * (K >> 1) + kb * 16) = make_uint4(o1[0], o1[1], o1[2], o1[3]);
    *reinterpret_cast<uint4*>(q2 + row * (K >> 1) + kb * 16) = make_uint4(o2[0], o2[1], o2[2], o2[3]);
    // sf_kgroups == 0: row-major [M, K/32]; otherwise the 512-byte blocks (128 rows x 4 scales) the block-scaled
    // MMA's shared-memory -> TMEM scale copy expects: block (row/128, kb/4), byte (row%32)*16 + ((row/32)%4)*4 + kb%4
    const int64_t so = sf_kgroups == 0
                           ? row * kblocks + kb
                           : ((row >> 7) * sf_kgroups + (kb >> 2)) * 512 + (row & 31) * 16 + ((row >> 5) & 3) * 4 + (kb & 3);
    if (pack4) {
      // four neighbouring lanes hold the four scales of one aligned 32-bit word (kblocks is a multiple of 4)
      uint32_t w1 = static_cast<uint32_t>(a + 127) << (8 * (threadIdx.x & 3)), w2 = static_cast<uint32_t>(bexp + 127) << (8 * (threadIdx.x & 3));
      w1 |= __shfl_xor_sync(lanes, w1, 1); w2 |= __shfl_xor_sync(lanes, w2, 1);
      w1 |= __shfl_xor_sync(lanes, w1, 2); w2 |= __shfl_xor_sync(lanes, w2, 2);
      if ((threadIdx.x & 3) == 0) {
        *reinterpret_cast<uint32_t*>(e1 + so) = w1;
        *reinterpret_cast<uint32_t*>(e2 + so) = w2;
      }
    } else {
      e1[so] = static_cast<uint8_t>(a + 127);
      e2[so] = static_cast<uint8_t>(bexp + 127);
    }
    }
  }
}

msd_status_t launch_decompose_int8(const void* x_bf16, int64_t M, int64_t K, int64_t ldx, int8_t* q1, int8_t* q2,
                                   float* alpha, float* beta, float c1, float c2, cudaStream_t stream) {
  if (M == 0) return MSD_OK;
  // A plain launch (chaining it to its predecessor as a programmatic dependent measured slower: its loads then queue
  // behind the weight prefetch of the GEMM that follows it).
  // this kernel sits on the critical path of the GEMM behind it: more threads per row = shorter latency
  const int threads = K >= 8192 ? 1024 : (K >= 2048 ? 512 : 256);
  cudaError_t err;
  if (threads >= 1024)
    err = launch_pdl(decompose_int8_kernel<1024>, dim3(static_cast<unsigned>(M)), dim3(1024), 0, stream, false,
                     static_cast<const uint16_t*>(x_bf16), static_cast<int64_t>(ldx), static_cast<int>(K), q1, q2, alpha, beta, c1, c2);
  else if (threads >= 512)
    err = launch_pdl(decompose_int8_kernel<512>, dim3(static_cast<unsigned>(M)), dim3(512), 0, stream, false,
                     static_cast<const uint16_t*>(x_bf16), static_cast<int64_t>(ldx), static_cast<int>(K), q1, q2, alpha, beta, c1, c2);
  else
    err = launch_pdl(decompose_int8_kernel<256>, dim3(static_cast<unsigned>(M)), dim3(256), 0, stream, false,
                     static_cast<const uint16_t*>(x_bf16), static_cast<int64_t>(ldx), static_cast<int>(K), q1, q2, alpha, beta, c1, c2);
  return err == cudaSuccess ? MSD_OK : MSD_ERR_CUDA;
}

msd_status_t launch_decompose_mxfp4(const void* x_bf16, int64_t M, int64_t K, int64_t ldx, uint8_t* q1, uint8_t* q2,
                                    uint8_t* e1, uint8_t* e2, int sf_kgroups, cudaStream_t stream, SfRelayout* relayout,
                                    const RowGroups* groups) {
  if (M == 0) return MSD_OK;
  const int per_sm = 32, rl_per_sm = (relayout && relayout->matrices > 1) ? 16 : 4;
  SfRelayout rl = {};
  if (relayout) {
    rl = *relayout;
    const int64_t rb = static_cast<int64_t>(rl.row_blocks) * ((rl.sf_kgroups + 31) / 32) * (rl.matrices > 1 ? rl.matrices : 1);   // units
    rl.blocks = static_cast<int>(rb < rl_per_sm * sm_count() ? rb : rl_per_sm * sm_count());
    relayout->blocks = rl.blocks;
  }
  RowGroups rg = {};
  if (groups) rg = *groups;
  const int64_t nblocks = M * (K >> 5);
  const int64_t want = (nblocks + kMxThreads - 1) / kMxThreads;
  const int64_t cap = static_cast<int64_t>(sm_count()) * per_sm;
  const unsigned grid = static_cast<unsigned>(want < cap ? want : cap) + static_cast<unsigned>(rl.blocks);
  static bool carve_done = false;
  if (!carve_done) {
    cudaFuncSetAttribute(decompose_mxfp4_kernel, cudaFuncAttributePreferredSharedMemoryCarveout, cudaSharedmemCarveoutMaxShared);
    carve_done = true;
  }
  decompose_mxfp4_kernel<<<grid, kMxThreads, 0, stream>>>(static_cast<const uint16_t*>(x_bf16), ldx, M,
                                                          static_cast<int>(K), q1, q2, e1, e2, sf_kgroups, rl, rg);
  return launch_status();
}

}  // namespace msd

extern "C" {

msd_status_t msd_decompose_int8_ex(const void* x_bf16, int64_t M, int64_t K, int64_t ldx, int8_t* q1, int8_t* q2,
                                   float* alpha, float* beta, msd_scaling_t scaling, void* stream) {
  if (scaling != MSD_SCALING_DEFAULT && scaling != MSD_SCALING_FRACTIONAL) return MSD_ERR_UNSUPPORTED;
  if (M < 0 || K <= 0 || K % 16 != 0 || ldx < K || ldx % 8 != 0 || M > 0x7FFFFFFF || K > 0x7FFFFFF0) return MSD_ERR_BAD_SHAPE;
  if (M == 0) return MSD_OK;
  if (!x_bf16 || !q1 || !q2 || !alpha || !beta) return MSD_ERR_NULL_POINTER;
  if (!msd::aligned(x_bf16, 16) || !msd::aligned(q1, 16) || !msd::aligned(q2, 16) || !msd::aligned(alpha, 4) ||
      !msd::aligned(beta, 4))
    return MSD_ERR_BAD_ALIGNMENT;
  return msd::launch_decompose_int8(x_bf16, M, K, ldx, q1, q2, alpha, beta, msd::scaling_c1(scaling), msd::scaling_c2(scaling),
                                    static_cast<cudaStream_t>(stream));
}

msd_status_t msd_decompose_int8(const void* x_bf16, int64_t M, int64_t K, int64_t ldx, int8_t* q1, int8_t* q2,
                                float* alpha, float* beta, void* stream) {
  return msd_decompose_int8_ex(x_bf16, M, K, ldx, q1, q2, alpha, beta, MSD_SCALING_DEFAULT, stream);
}

msd_status_t msd_decompose_mxfp4(const void* x_bf16, int64_t M, int64_t K, int64_t ldx, uint8_t* q1, uint8_t* q2,
                                 uint8_t* e8m0_1, uint8_t* e8m0_2, void* stream) {
  if (M < 0 || K <= 0 || K % 32 != 0 || ldx < K || ldx % 8 != 0 || K > 0x7FFFFFE0) return MSD_ERR_BAD_SHAPE;
  if (M == 0) return MSD_OK;
  if (!x_bf16 || !q1 || !q2 || !e8m0_1 || !e8m0_2) return MSD_ERR_NULL_POINTER;
  if (!msd::aligned(x_bf16, 16) || !msd::aligned(q1, 16) || !msd::aligned(q2, 16)) return MSD_ERR_BAD_ALIGNMENT;
  return msd::launch_decompose_mxfp4(x_bf16, M, K, ldx, q1, q2, e8m0_1, e8m0_2, 0, static_cast<cudaStream_t>(stream));
}

}  // extern "C"

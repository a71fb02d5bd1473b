// W8A16 comparison kernel with the dequantization fused into the GEMM (the stronger of the two baselines MSD is measured
// against; Sec. 2.3 "kernel optimization methods reduce its cost"): the INT8 weights are read from HBM once, as in MSD,
// converted to BF16 (exactly) by twelve warps on their way from the TMA staging buffer into TENSOR MEMORY, from where they are
// the A operand of BF16 x BF16 -> FP32 MMAs (tcgen05.mma kind::f16, A in tensor memory, the BF16 activations as B in
// shared memory); the per-channel weight scale is applied to the sums.  No decomposition kernel, no second component:
//   y[m,n] = w_scale[n] * sum_k x[m,k] * float(w[n,k])          (the INT8 values are exact in BF16)
// Decode regime only (M <= 128).  The weight rows sit on the MMA M axis as in the MSD decode kernel: one band of up to
// 128 rows per CTA when the bands are at least 64 rows high, else 128-row tiles with the K stages of a tile split over
// several CTAs (FP32 partial results, added by ksplit_reduce_kernel in a fixed order).
//
// Warp roles: 0 = TMA producer, 1 = MMA issuer and TMEM owner, 2..13 = converters; 2..5 then run the epilogue.
// A stage holds kw K blocks of 64 elements: INT8 weights [kw][rows][64 B] (64-byte swizzle: a converter thread reads
// its own row 16 bytes at a time without bank conflicts) and BF16 activations [kw][Mp][128 B] (128-byte swizzle).
// A converter thread owns one weight row (= tensor-memory lane) of one K block: 64 bytes in, 32 columns of
// two BF16 values out (tcgen05.st).  Two sets of kw x 32 columns alternate.  (With the converted weights written to shared memory
// instead, every weight byte crossed the shared-memory port seven times and the kernel ran at 27-29 us where this one
// needs less; that version is what the TMA-to-MMA path of MSD avoids.)
#include <cuda_bf16.h>

#include "host_common.h"
#include "sm100.cuh"

namespace msd {

constexpr int kFzConvWarps = 12;             // three per warp scheduler and tensor-memory lane quadrant
constexpr int kFzThreads = 64 + 32 * kFzConvWarps;
constexpr int kFzMaxStages = 8;
constexpr int kFzBlockK = 64;               // elements per K block: 64 B of INT8 weights, 128 B of BF16 activations
constexpr int kFzAccCols = 128;             // tensor-memory columns of the accumulator; the operand sets follow
constexpr int kFzTmemCols = 512;

struct FzParams {
  int M, Mp, N, K;
  int band_h;            // weight rows per work item along N (multiple of 8, <= 128)
  int bands;             // work items along N
  int ksplit, kper;      // K splits per band and K stages per split
  int kstages;           // K stages in all: ceil(K / (64 kw))
  int kw;                // K blocks per stage: 3 or 6 (a multiple of the three converter warps per lane quadrant)
  int stages;            // pipeline stages
  int ytype;
  const float* w_scale;
  void* y;
  float* part;           // ksplit > 1: [ksplit][M][N] FP32
  unsigned* status;
};

// 16 signed bytes -> 16 BF16 values (exact), two per word.  x ^ 0x80 is the byte of x + 128; 0x4B0000uu is the float
// 2^23 + uu, so one byte permute and one subtraction give float(x), whose upper half is its BF16 form (|x| <= 128 has 8
// significant bits): 2.75 instructions per element.  (The FP16 route - 0x64uu is 1024 + uu, one packed subtraction per
// two elements, 1.25 instructions per element - needs an FP16 A operand against the BF16 activations; an MMA of
// kind::f16 with the two operand formats set differently raised an illegal-instruction error, so both are BF16.)
__device__ __forceinline__ void cvt_s8x16_bf16(const uint4& v, uint32_t (&o)[8]) {
  const uint32_t w[4] = {v.x ^ 0x80808080u, v.y ^ 0x80808080u, v.z ^ 0x80808080u, v.w ^ 0x80808080u};
#pragma unroll
  for (int i = 0; i < 4; ++i) {
    const float f0 = __uint_as_float(__byte_perm(w[i], 0x4B000000u, 0x7650)) - 8388736.0f;
    const float f1 = __uint_as_float(__byte_perm(w[i], 0x4B000000u, 0x7651)) - 8388736.0f;
    const float f2 = __uint_as_float(__byte_perm(w[i], 0x4B000000u, 0x7652)) - 8388736.0f;
    const float f3 = __uint_as_float(__byte_perm(w[i], 0x4B000000u, 0x7653)) - 8388736.0f;
    o[2 * i] = __byte_perm(__float_as_uint(f0), __float_as_uint(f1), 0x7632);
    o[2 * i + 1] = __byte_perm(__float_as_uint(f2), __float_as_uint(f3), 0x7632);
  }
}

__global__ void __launch_bounds__(kFzThreads, 1)
gemm_w8a16_fused_kernel(const __grid_constant__ CUtensorMap tmap_w, const __grid_constant__ CUtensorMap tmap_x, const FzParams p) {
  extern __shared__ uint8_t smem_dyn[];
  __shared__ __align__(8) uint64_t full_bar[kFzMaxStages], empty_bar[kFzMaxStages], conv_full[2], conv_free[2], tfull_bar;
  __shared__ uint32_t tmem_base_slot;
  __shared__ int abort_flag;

  const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
  if (p.stages < 1 || p.stages > kFzMaxStages || p.kw < 1 || p.band_h < 8) return;        // malformed plan: touch nothing
  uint8_t* smem = reinterpret_cast<uint8_t*>((reinterpret_cast<uintptr_t>(smem_dyn) + 1023) & ~static_cast<uintptr_t>(1023));
  const int w_stage_bytes = p.kw * p.band_h * kFzBlockK;                 // INT8 staging of a stage (a multiple of 512)
  const int x_chunk_bytes = p.Mp * 128;
  const int stage_bytes = ((w_stage_bytes + 1023) & ~1023) + p.kw * x_chunk_bytes;
  const int x_off = (w_stage_bytes + 1023) & ~1023;

  const int band = blockIdx.x / p.ksplit, split = blockIdx.x - band * p.ksplit;
  const int row0 = band * p.band_h;
  const int ks0 = split * p.kper, ks1 = min(ks0 + p.kper, p.kstages);
  const int nst = ks1 - ks0;

  if (threadIdx.x == 0) {
    for (int s = 0; s < p.stages; ++s) { mbar_init(&full_bar[s], 1); mbar_init(&empty_bar[s], 1); }
    for (int b = 0; b < 2; ++b) { mbar_init(&conv_full[b], kFzConvWarps); mbar_init(&conv_free[b], 1); }     // the two operand sets
    mbar_init(&tfull_bar, 1);
    abort_flag = 0;
    mbar_init_fence();
    tma_prefetch_desc(&tmap_w);
    tma_prefetch_desc(&tmap_x);
  }
  if (warp == 1) tmem_alloc(&tmem_base_slot, kFzTmemCols);
  tc_fence_before();
  __syncthreads();
  tc_fence_after();
  const uint32_t tmem_base = tmem_base_slot;
  volatile int* abort = &abort_flag;

  if (warp == 0) {
    // ------------------------------ TMA producer ------------------------------
    if (lane == 0) {
      const uint64_t pol_w = policy_evict_first(), pol_x = policy_evict_last();
      const uint32_t tx = static_cast<uint32_t>(w_stage_bytes + p.kw * x_chunk_bytes);
      bool ok = true;
      for (int i = 0; i < nst && ok; ++i) {
        const int s = i % p.stages;
        if (i >= p.stages) ok = wait_bounded(&empty_bar[s], ((i / p.stages) - 1) & 1, abort, p.status);
        if (!ok) break;
        uint8_t* dst = smem + s * stage_bytes;
        mbar_arrive_expect_tx(&full_bar[s], tx);
        tma_load_3d_hint(dst, &tmap_w, 0, row0, (ks0 + i) * p.kw, &full_bar[s], pol_w);
        tma_load_3d_hint(dst + x_off, &tmap_x, 0, 0, (ks0 + i) * p.kw, &full_bar[s], pol_x);
      }
      if (!ok) {      // give copies already in flight a bounded time to land before the CTA goes away
        const long long t0 = clock64();
        while (clock64() - t0 < 2000000LL) {}
      }
    }
  } else if (warp == 1) {
    // ------------------------------ MMA issuer ------------------------------
    if (lane == 0) {
      const uint32_t idesc = idesc_dense(/*D=F32*/ 1, /*A=BF16*/ 1, /*B=BF16*/ 1, 0, 0, 128, p.Mp);
      const uint64_t op_desc = smem_desc(0, 16, 1024, kSwizzle128B);
      bool ok = true;
      for (int i = 0; i < nst && ok; ++i) {
        const int s = i % p.stages, b = i & 1;
        ok = wait_bounded(&full_bar[s], (i / p.stages) & 1, abort, p.status);          // the activation chunks of the stage
        if (ok) ok = wait_bounded(&conv_full[b], (i >> 1) & 1, abort, p.status);       // its weights, converted
        if (!ok) break;
        tc_fence_after();
        const uint32_t at = tmem_base + kFzAccCols + b * (p.kw * 32);      // operand set b: 32 columns per K block
        const uint64_t xd = op_desc + (smem_u32(smem + s * stage_bytes + x_off) >> 4);
        for (int c = 0; c < p.kw; ++c) {
#pragma unroll
          for (int k = 0; k < 4; ++k)        // 16 BF16 elements per MMA: 8 columns of A, 32 bytes of every B row
            mma_f16_ts(tmem_base, at + c * 32 + k * 8, xd + ((c * x_chunk_bytes) >> 4) + 2 * k, idesc,
                       (i > 0 || c > 0 || k > 0) ? 1u : 0u);
        }
        tc_commit(&empty_bar[s]);         // the stage (its activation chunks; the converters are long done with the weights)
        tc_commit(&conv_free[b]);         // the operand set may be overwritten
      }
      if (ok) tc_commit(&tfull_bar);
    }
  } else {
    // ------------------------------ converters (warps 2..13), then epilogue (warps 2..5) ------------------------------
    const int quad = warp & 3;                      // tensor-memory lane quadrant this warp may touch
    const int grp = (warp - 2) >> 2;                // 0..2: which K blocks of a stage (c = grp, grp + 3)
    const int r = quad * 32 + lane;                 // weight row of the band = tensor-memory lane
    const uint32_t trow = tmem_base + (static_cast<uint32_t>(quad * 32) << 16);
    const int sw = (r >> 1) & 3;                    // 64-byte swizzle: the 16-byte piece index is XORed with (row / 2) % 4
    bool ok = true;
    for (int i = 0; i < nst && ok; ++i) {
      const int s = i % p.stages, b = i & 1;
      ok = wait_bounded(&full_bar[s], (i / p.stages) & 1, abort, p.status);
      if (ok && i >= 2) ok = wait_bounded(&conv_free[b], ((i >> 1) - 1) & 1, abort, p.status);
      if (!ok) break;
      tc_fence_after();
      const uint8_t* src = smem + s * stage_bytes;
      for (int c = grp; c < p.kw; c += 3) {
        uint32_t o[32];
        if (r < p.band_h) {
          const uint8_t* row = src + (c * p.band_h + r) * kFzBlockK;
#pragma unroll
          for (int pc = 0; pc < 4; ++pc) {
            uint32_t h[8];
            cvt_s8x16_bf16(*reinterpret_cast<const uint4*>(row + ((pc ^ sw) << 4)), h);
#pragma unroll
            for (int j = 0; j < 8; ++j) o[8 * pc + j] = h[j];
          }
        } else {
#pragma unroll
          for (int j = 0; j < 32; ++j) o[j] = 0u;     // rows past the band: zeros (their sums are never stored)
        }
        tmem_st32(trow + kFzAccCols + b * (p.kw * 32) + c * 32, o);
      }
      tmem_st_wait();
      tc_fence_before();
      __syncwarp();
      if (lane == 0) mbar_arrive(&conv_full[b]);
    }
    // epilogue: thread = weight row (TMEM lane); its sums over the tokens lie along the columns
    if (ok && warp < 6) ok = wait_bounded(&tfull_bar, 0, abort, p.status);
    if (ok && warp < 6) {
      tc_fence_after();
      const int n = row0 + r;
      const bool row_ok = r < p.band_h && n < p.N;
      const float wsc = row_ok ? __ldg(p.w_scale + n) : 0.0f;
      for (int c0 = 0; c0 < p.Mp; c0 += 16) {
        uint32_t v[16];
        tmem_ld16(trow + c0, v);
        tmem_ld_wait();
        if (row_ok) {
#pragma unroll
          for (int j = 0; j < 16; ++j) {
            const int m = c0 + j;
            if (m < p.M) {
              const float val = wsc * __uint_as_float(v[j]);
              if (p.ksplit > 1) p.part[(static_cast<size_t>(split) * p.M + m) * p.N + n] = val;
              else if (p.ytype == MSD_OUT_BF16) static_cast<__nv_bfloat16*>(p.y)[static_cast<size_t>(m) * p.N + n] = __float2bfloat16_rn(val);
              else static_cast<float*>(p.y)[static_cast<size_t>(m) * p.N + n] = val;
            }
          }
        }
      }
    }
  }

  tc_fence_before();
  __syncthreads();
  if (warp == 1) {
    tc_fence_after();
    tmem_dealloc(tmem_base, kFzTmemCols);
  }
}

struct FzPlan {
  int Mp, band_h, bands, ksplit, kper, kstages, kw, stages;
  size_t smem_bytes, bytes;
};

static FzPlan plan_fz(int64_t M, int64_t N, int64_t K) {
  FzPlan pl;
  pl.Mp = static_cast<int>((M + 15) / 16 * 16);
  const int sms = sm_count();
  // one band per SM where the bands come out at least 64 rows high, else 128-row tiles with a K split
  const int64_t g8 = (N + 7) / 8;
  int band_h = static_cast<int>(8 * ((g8 + sms - 1) / sms));
  if (band_h < 64 || band_h > 128) band_h = 128;
  pl.band_h = band_h;
  pl.bands = static_cast<int>((N + band_h - 1) / band_h);
  // K blocks per stage: wide stages read each weight row in longer runs; the activation chunks grow with M
  // six K blocks per stage (two per converter warp; 2 x 192 operand columns + 128 accumulator columns = all of tensor
  // memory), three where the activation chunks are large
  pl.kw = pl.Mp <= 32 ? 6 : 3;
  pl.kstages = static_cast<int>((K + static_cast<int64_t>(pl.kw) * kFzBlockK - 1) / (static_cast<int64_t>(pl.kw) * kFzBlockK));
  pl.ksplit = 1;
  if (2 * pl.bands <= sms) {
    int want = sms / pl.bands;
    if (want > pl.kstages / 2) want = pl.kstages / 2;
    if (want > 1) pl.ksplit = want;
  }
  pl.kper = (pl.kstages + pl.ksplit - 1) / pl.ksplit;
  pl.ksplit = (pl.kstages + pl.kper - 1) / pl.kper;
  const size_t w_stage = round_up(static_cast<size_t>(pl.kw) * band_h * kFzBlockK, 1024);
  const size_t stage = w_stage + static_cast<size_t>(pl.kw) * pl.Mp * 128;
  const size_t budget = 227 * 1024 - 2048 - 1024;
  int stages = static_cast<int>(budget / stage);
  if (stages > kFzMaxStages) stages = kFzMaxStages;
  pl.stages = stages;
  pl.smem_bytes = static_cast<size_t>(stages) * stage + 1024;
  pl.bytes = pl.ksplit > 1 ? round_up(static_cast<size_t>(pl.ksplit) * M * N * sizeof(float), 1024) : 1024;
  return pl;
}

}  // namespace msd

extern "C" {

size_t msd_gemm_w8a16_fused_dequant_workspace_bytes(int64_t M, int64_t N, int64_t K) {
  if (M < 1 || M > 128 || N < 1 || K < 64 || K % 64 != 0) return 0;
  return msd::plan_fz(M, N, K).bytes;
}

msd_status_t msd_gemm_w8a16_fused_dequant(const void* x_bf16, const int8_t* w, const float* w_scale, int64_t M, int64_t N,
                                          int64_t K, void* y, msd_out_t ytype, void* workspace, size_t workspace_bytes,
                                          void* stream) {
  using namespace msd;
  if (M < 1 || M > 128 || N < 1 || K < 64 || K % 64 != 0 || N % 8 != 0 || N > (1 << 24) || K > (1 << 24)) return MSD_ERR_BAD_SHAPE;
  if (ytype != MSD_OUT_BF16 && ytype != MSD_OUT_FP32) return MSD_ERR_UNSUPPORTED;
  if (!x_bf16 || !w || !w_scale || !y || !workspace) return MSD_ERR_NULL_POINTER;
  if (!aligned(x_bf16, 16) || !aligned(w, 16) || !aligned(y, 16) || !aligned(w_scale, 4) || !aligned(workspace, 1024))
    return MSD_ERR_BAD_ALIGNMENT;
  const FzPlan pl = plan_fz(M, N, K);
  if (pl.stages < 2) return MSD_ERR_UNSUPPORTED;
  if (workspace_bytes < pl.bytes) return MSD_ERR_WORKSPACE_TOO_SMALL;
  unsigned* status = device_status_ptr();
  if (!status) return MSD_ERR_CUDA;
  cudaStream_t s = static_cast<cudaStream_t>(stream);
  CUtensorMap tmap_w, tmap_x;
  // weights: {64 B of a K block, rows, K blocks}; activations as bytes: {128 B of a K block, rows, K blocks}
  if (!encode_tmap_3d(&tmap_w, CU_TENSOR_MAP_DATA_TYPE_UINT8, w, kFzBlockK, N, K / kFzBlockK, K, kFzBlockK, kFzBlockK,
                      static_cast<uint32_t>(pl.band_h), static_cast<uint32_t>(pl.kw), CU_TENSOR_MAP_SWIZZLE_64B) ||
      !encode_tmap_3d(&tmap_x, CU_TENSOR_MAP_DATA_TYPE_UINT8, x_bf16, 128, M, K / kFzBlockK, 2 * K, 128, 128,
                      static_cast<uint32_t>(pl.Mp), static_cast<uint32_t>(pl.kw), CU_TENSOR_MAP_SWIZZLE_128B))
    return MSD_ERR_CUDA;
  FzParams p;
  p.M = static_cast<int>(M); p.Mp = pl.Mp; p.N = static_cast<int>(N); p.K = static_cast<int>(K);
  p.band_h = pl.band_h; p.bands = pl.bands; p.ksplit = pl.ksplit; p.kper = pl.kper; p.kstages = pl.kstages; p.kw = pl.kw;
  p.stages = pl.stages; p.ytype = ytype; p.w_scale = w_scale; p.y = y;
  p.part = static_cast<float*>(workspace); p.status = status;
  static bool attr_done = false;
  if (!attr_done) {
    if (cudaFuncSetAttribute(gemm_w8a16_fused_kernel, cudaFuncAttributeMaxDynamicSharedMemorySize, 227 * 1024 - 2048) != cudaSuccess)
      return MSD_ERR_CUDA;
    attr_done = true;
  }
  gemm_w8a16_fused_kernel<<<static_cast<unsigned>(pl.bands * pl.ksplit), kFzThreads, pl.smem_bytes, s>>>(tmap_w, tmap_x, p);
  if (cudaGetLastError() != cudaSuccess) return MSD_ERR_CUDA;
  if (pl.ksplit > 1)
    return launch_ksplit_reduce(p.part, pl.ksplit, M * N, M, N, y, static_cast<int>(ytype), s, false);
  return MSD_OK;
}

}  // extern "C"

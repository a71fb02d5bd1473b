// Host-side helpers shared by the C-ABI entry points: argument checks, the device status word,
// tensor-map encoding through the driver entry point, launch-error mapping.
#pragma once
#include <cuda.h>
#include <cuda_runtime.h>
#include <stdint.h>

#include "msd.h"

namespace msd {

// Device address of this device's status word (one per device; NULL on failure).
unsigned* device_status_ptr();

int sm_count();

// Encodes a 2-D tiled tensor map: `inner` contiguous elements per row, `outer` rows, rows `row_stride_bytes`
// apart; the box is box_inner x box_outer elements.  Returns false on failure.
bool encode_tmap_2d(CUtensorMap* out, CUtensorMapDataType dtype, const void* base, uint64_t inner, uint64_t outer,
                    uint64_t row_stride_bytes, uint32_t box_inner, uint32_t box_outer, CUtensorMapSwizzle swizzle);
bool encode_tmap_3d(CUtensorMap* out, CUtensorMapDataType dtype, const void* base, uint64_t d0, uint64_t d1, uint64_t d2,
                    uint64_t stride1_bytes, uint64_t stride2_bytes, uint32_t b0, uint32_t b1, uint32_t b2,
                    CUtensorMapSwizzle swizzle);

inline bool aligned(const void* p, size_t a) { return (reinterpret_cast<uintptr_t>(p) & (a - 1)) == 0; }
inline size_t round_up(size_t v, size_t a) { return (v + a - 1) / a * a; }

inline msd_status_t launch_status() { return cudaGetLastError() == cudaSuccess ? MSD_OK : MSD_ERR_CUDA; }

// Kernel launch with the programmatic-dependent-launch attribute (the kernel may start while its predecessor in
// the stream is still running and must call griddepcontrol.wait before touching the predecessor's outputs).
template <typename... Args>
cudaError_t launch_pdl_cluster(void (*kernel)(Args...), dim3 grid, dim3 block, size_t smem, cudaStream_t stream, bool pdl,
                               unsigned cluster, Args... args) {
  cudaLaunchConfig_t cfg = {};
  cfg.gridDim = grid;
  cfg.blockDim = block;
  cfg.dynamicSmemBytes = smem;
  cfg.stream = stream;
  cudaLaunchAttribute attr[2];
  unsigned n = 0;
  if (pdl) {
    attr[n].id = cudaLaunchAttributeProgrammaticStreamSerialization;
    attr[n].val.programmaticStreamSerializationAllowed = 1;
    ++n;
  }
  if (cluster > 1) {      // grid.x must be a multiple of the cluster size
    attr[n].id = cudaLaunchAttributeClusterDimension;
    attr[n].val.clusterDim.x = cluster;
    attr[n].val.clusterDim.y = 1;
    attr[n].val.clusterDim.z = 1;
    ++n;
  }
  cfg.attrs = attr;
  cfg.numAttrs = n;
  return cudaLaunchKernelEx(&cfg, kernel, args...);
}
template <typename... Args>
cudaError_t launch_pdl(void (*kernel)(Args...), dim3 grid, dim3 block, size_t smem, cudaStream_t stream, bool pdl,
                       Args... args) {
  return launch_pdl_cluster(kernel, grid, block, smem, stream, pdl, 1u, args...);
}

// Internal entry used by the GEMM: decomposition written straight into the stacked operand buffer.
// (c1, c2): the scaling constants of the two passes, alpha = max/c1 and beta = alpha/c2.
msd_status_t launch_decompose_int8(const void* x_bf16, int64_t M, int64_t K, int64_t ldx, int8_t* q1, int8_t* q2,
                                   float* alpha, float* beta, float c1, float c2, cudaStream_t stream);
inline float scaling_c1(msd_scaling_t s) { return s == MSD_SCALING_FRACTIONAL ? 127.49f : 127.0f; }
inline float scaling_c2(msd_scaling_t s) { return s == MSD_SCALING_FRACTIONAL ? 254.98f : 254.0f; }
// Sum of K-split FP32 partial results part[s * part_stride + i], s = 0 .. ksplit-1 in that order, rounded once to y
// (gemm_w4a16.cu; N a multiple of 4).
msd_status_t launch_ksplit_reduce(const float* part, int ksplit, int64_t part_stride, int64_t M, int64_t N, void* y, int ytype,
                                  cudaStream_t s, bool pdl);

// W8A16 layer for M > 128 rows (gemm_w8a16_prefill.cu); arguments checked by the caller.
size_t w8_prefill_workspace_bytes(int64_t M, int64_t N, int64_t K);
msd_status_t w8_prefill_launch(const void* x_bf16, const int8_t* w, const float* w_scale, int64_t M, int64_t N, int64_t K,
                               void* y, int ytype, int32_t* acc_dbg, float c1, float c2, void* workspace,
                               size_t workspace_bytes, cudaStream_t stream);

// A scale relayout that rides along with the MXFP4 decomposition kernel (extra CTAs of the same launch): row-major
// E8M0 scales src[rows, kblocks] -> 512-byte blocks at dst, `row_blocks` = 2 x number of row tiles of `tile_rows` rows.
struct SfRelayout {
  const uint8_t* src;
  uint8_t* dst;
  int64_t rows;
  int kblocks, sf_kgroups, tile_rows, row_blocks;
  int matrices;        // 0 or 1: one matrix; E > 1: E matrices of `rows` rows back to back (mixture-of-experts
                       // weights), each cut into its own `row_blocks` blocks
  int blocks;          // filled in by the launcher (returned through the pointer when `ready` is used)
};
// Rows sorted by group (mixture of experts): group g owns rows [off[g], off[g+1]) and its decomposition is written as
// token tile g (rows 128 g ...) of the component and scale buffers.
constexpr int kMaxRowGroups = 64;
struct RowGroups {
  int n;                       // 0: no regrouping, output row = input row
  int off[kMaxRowGroups + 1];
};
msd_status_t launch_decompose_mxfp4(const void* x_bf16, int64_t M, int64_t K, int64_t ldx, uint8_t* q1, uint8_t* q2,
                                    uint8_t* e1, uint8_t* e2, int sf_kgroups, cudaStream_t stream,
                                    SfRelayout* relayout = nullptr, unsigned* ready = nullptr, const RowGroups* groups = nullptr);

#ifdef __CUDACC__
// Relayout of row-major E8M0 scales [rows, kblocks] into the 512-byte blocks (128 rows x 4 scales) of the block-scaled
// MMA.  Rows are first cut into tiles of `tile_rows` (a multiple of 32), every tile into two blocks (the second one
// partly used when tile_rows < 256); entries outside the matrix are written as zero.  One thread per 16 bytes of
// the result: the four scales of rows l, l+32, l+64, l+96 of one block.
__device__ inline void sf_relayout(const SfRelayout& j, int64_t first, int64_t step) {
  const int nmat = j.matrices > 1 ? j.matrices : 1;
  const int64_t per = static_cast<int64_t>(j.row_blocks) * j.sf_kgroups * 32;
  const int64_t total = per * nmat;
  for (int64_t dd = first; dd < total; dd += step) {
    const int64_t e = dd / per, d = dd - e * per;
    const uint8_t* src = j.src + e * j.rows * j.kblocks;
    const int l = static_cast<int>(d & 31);
    const int64_t blk = d >> 5;
    const int64_t tb = blk / j.sf_kgroups;
    const int kg = static_cast<int>(blk - tb * j.sf_kgroups);
    const int64_t t = tb >> 1;
    uint32_t v[4];
#pragma unroll
    for (int q = 0; q < 4; ++q) {
      const int lr = static_cast<int>(tb & 1) * 128 + l + 32 * q;
      const int64_t row = t * j.tile_rows + lr;
      v[q] = (lr < j.tile_rows && row < j.rows && 4 * kg < j.kblocks)
                 ? __ldg(reinterpret_cast<const uint32_t*>(src + row * j.kblocks + 4 * kg)) : 0u;
    }
    reinterpret_cast<uint4*>(j.dst)[dd] = make_uint4(v[0], v[1], v[2], v[3]);
  }
}
#endif


}  // namespace msd

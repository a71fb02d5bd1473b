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

// The library's few run-time switches, all testing or diagnostic aids.  Each is read from the environment variable of
// the same name ONCE, when the first call needs one, and can be set afterwards with msd_debug_set_option(); -1 = unset.
enum Option {
  OPT_NO_PDL = 0,           // MSD_NO_PDL: launch dependent kernels without programmatic dependent launch
  OPT_GEMM_MODE,            // MSD_GEMM_MODE: force a work split of the W8A16 decode kernel (0 stream-K, 1 row bands, 2 clusters)
  OPT_GEMM_CTAS,            // MSD_GEMM_CTAS: number of CTAs of that kernel
  OPT_P8_PAIR,              // MSD_P8_PAIR: W8A16 many-row kernel on CTA pairs (1) or single CTAs (0)
  OPT_P8_KSPLIT,            // MSD_P8_KSPLIT: its K split
  OPT_W4_PAIR,              // MSD_W4_PAIR: W4A16 kernel on CTA pairs (1) or single CTAs (0)
  OPT_W4_TILEN,             // MSD_W4_TILEN: tile width of the single-CTA W4A16 kernel (224 or 256)
  OPT_W4_KSPLIT,            // MSD_W4_KSPLIT: its K split
  OPT_ATTN_SPLITS,          // MSD_ATTN_SPLITS: number of context splits of the attention kernels
  OPT_ATTN_CHUNK_TILES,     // MSD_ATTN_CHUNK_TILES: tiles per context split
  OPT_ATTN_BALANCED,        // MSD_ATTN_BALANCED: 1 balanced schedule wherever a kernel for it exists, 0 never
  OPT_COUNT
};
int option(Option o);

// Encodes a 2-D tiled tensor map: `inner` contiguous elements per row, `outer` rows, rows `row_stride_bytes`
// apart; the box is box_inner x box_outer elements.  Returns false on failure.
bool encode_tmap_2d(CUtensorMap* out, CUtensorMapDataType dtype, const void* base, uint64_t inner, uint64_t outer,
                    uint64_t row_stride_bytes, uint32_t box_inner, uint32_t box_outer, CUtensorMapSwizzle swizzle);
bool encode_tmap_3d(CUtensorMap* out, CUtensorMapDataType dtype, const void* base, uint64_t d0, uint64_t d1, uint64_t d2,
                    uint64_t stride1_bytes, uint64_t stride2_bytes, uint32_t b0, uint32_t b1, uint32_t b2,
                    CUtensorMapSwizzle swizzle);

inline bool aligned(const void* p, size_t a) { return (reinterpret_cast<uintptr_t>(p) & (a - 1)) == 0; }
inline size_t round_up(size_t v, size_t a) { return (v + a - 1) / a * a; }

// attn_decode.cu: merges the context splits' partial results [rows][n_splits][4 + Dv] into out_bf16 [rows][Dv] (and lse)
msd_status_t launch_attn_combine(const float* partial, int n_splits, int Dv, void* out_bf16, float* lse, int rows, cudaStream_t s);

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

// The comparison path (dequantize to BF16, then a BF16 GEMM) for M > 128 rows, and the kernel launch that expands the
// INT8 weights to bf16(w_scale[n] * w[n,k]) (gemm_w8a16.cu).
size_t w8_prefill_base_workspace_bytes(int64_t M, int64_t N, int64_t K);
msd_status_t w8_prefill_base_launch(const void* x_bf16, const int8_t* w, const float* w_scale, int64_t M, int64_t N, int64_t K,
                                    void* y, int ytype, void* workspace, size_t workspace_bytes, cudaStream_t stream);
msd_status_t launch_dequant_w8_to_bf16(const int8_t* w, const float* w_scale, int64_t N, int64_t K, void* out_bf16, cudaStream_t stream);

// A scale relayout that rides along with the MXFP4 decomposition kernel (extra CTAs of the same launch): row-major
// E8M0 scales src[rows, kblocks] -> 512-byte blocks at dst, `row_blocks` = 2 x number of row tiles of `tile_rows` rows.
struct SfRelayout {
  const uint8_t* src;
  uint8_t* dst;
  int64_t rows;
  int kblocks, sf_kgroups, tile_rows, row_blocks;
  int matrices;        // 0 or 1: one matrix; E > 1: E matrices of `rows` rows back to back (mixture-of-experts
                       // weights), each cut into its own `row_blocks` blocks
  int blocks;          // filled in by the launcher
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
                                    SfRelayout* relayout = nullptr, const RowGroups* groups = nullptr);

#ifdef __CUDACC__
// Relayout of row-major E8M0 scales [rows, kblocks] into the 512-byte blocks (128 rows x 4 scales) of the block-scaled
// MMA.  Rows are first cut into tiles of `tile_rows` (a multiple of 32), every tile into two blocks (the second one
// partly used when tile_rows < 256); entries outside the matrix are written as zero.
// A CTA of 256 threads takes units of 128 rows x 32 K groups (128 scale bytes per row): it reads the rows in 128-byte
// runs into shared memory (a word per row and K group, rows 33 words apart) and writes the 32 blocks of the unit as
// 16-byte pieces, 512 contiguous bytes per warp - both sides coalesced.  (One thread per 16-byte piece reading its four
// words straight from global memory took 20 us for 14.7 MB of scales: every 4-byte read cost a 32-byte sector.)
constexpr int kSfRelayoutSmemWords = 128 * 33;
__device__ inline void sf_relayout(const SfRelayout& j, int cta, int ctas, uint32_t* sm /* kSfRelayoutSmemWords */) {
  const int nmat = j.matrices > 1 ? j.matrices : 1;
  const int kchunks = (j.sf_kgroups + 31) / 32;
  const int64_t units = static_cast<int64_t>(nmat) * j.row_blocks * kchunks;
  const int t = threadIdx.x;
  const int words_per_row = j.kblocks >> 2;                 // K groups that exist in the source (kblocks is a multiple of 4)
  for (int64_t u = cta; u < units; u += ctas) {
    const int kc = static_cast<int>(u % kchunks);
    const int64_t rb = u / kchunks;                          // (matrix, block row)
    const int64_t e = rb / j.row_blocks;
    const int tb = static_cast<int>(rb - e * j.row_blocks);
    const int64_t tile_row0 = static_cast<int64_t>(tb >> 1) * j.tile_rows;
    const int lr0 = (tb & 1) * 128;                          // first row of the block within its tile
    const uint32_t* src = reinterpret_cast<const uint32_t*>(j.src + e * j.rows * j.kblocks);
    // load: thread -> (row r = t / 32 + 8 i, K group c = t % 32)
    const int c = t & 31, kg = kc * 32 + c;
#pragma unroll 4
    for (int i = 0; i < 16; ++i) {
      const int r = (t >> 5) + 8 * i, lr = lr0 + r;
      const int64_t row = tile_row0 + lr;
      uint32_t v = 0;
      if (lr < j.tile_rows && row < j.rows && kg < words_per_row) v = __ldg(src + row * words_per_row + kg);
      sm[r * 33 + c] = v;
    }
    __syncthreads();
    // store: thread -> (K group c2 = t / 32 + 8 i, lane l = t % 32): the piece of rows l, l+32, l+64, l+96
    const int l = t & 31;
#pragma unroll
    for (int i = 0; i < 4; ++i) {
      const int c2 = (t >> 5) + 8 * i, kg2 = kc * 32 + c2;
      if (kg2 < j.sf_kgroups) {
        const uint4 o = make_uint4(sm[l * 33 + c2], sm[(l + 32) * 33 + c2], sm[(l + 64) * 33 + c2], sm[(l + 96) * 33 + c2]);
        reinterpret_cast<uint4*>(j.dst)[((e * j.row_blocks + tb) * j.sf_kgroups + kg2) * 32 + l] = o;
      }
    }
    __syncthreads();
  }
}
#endif


}  // namespace msd

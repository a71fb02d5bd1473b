// W8A16 MSD linear layer for the decode regime (Alg. 1; Sec. 3.9 pass fusion by stacking the two components).
//
// Roles are swapped relative to the usual GEMM: a 128-row tile of the INT8 weight is the MMA "A" operand
// (the M axis of tcgen05.mma), the stacked components [Q1; Q2] (NB = 2*ceil8(M) rows) are the "B" operand, so one
// weight tile read from HBM serves both passes and the accumulator D[128 weight rows x NB] lives in TMEM.
//
// Two work splits, chosen on the host:
//  * row partition (tall weights): the N weight rows are cut into one band per CTA (band heights h and h+8, multiples
//    of 8, at most 128), each CTA runs the whole K loop for its band and writes its outputs straight from TMEM.
//  * stream-K (few rows per SM): the (128-row tile, 128-byte K block) pairs are numbered tile-major and divided evenly
//    over the CTAs, so every SM streams the same number of weight bytes.  A CTA whose range covers a whole tile
//    finishes it alone; the CTAs that share a tile add their INT32 partial sums into the tile's meeting place in the
//    workspace and whichever arrives last reads it back, re-zeroes it and finishes (integer sums: order-free).
//
// Warp roles: warp 0 = TMA producer, warp 1 = MMA issuer (+ TMEM owner), warps 2-5 = epilogue (one per TMEM lane group).
#include <cuda_bf16.h>

#include <cstdlib>
#include <mutex>
#include <type_traits>

#include "host_common.h"
#include "quant.cuh"
#include "sm100.cuh"

namespace msd {

constexpr int kTileN = 128;        // weight rows per tile (MMA M)
constexpr int kBlockK = 128;       // K bytes per TMA box (one 128-byte swizzle row); a stage holds `kw` adjacent boxes
constexpr int kMaxStages = 16;
constexpr int kGemmThreads = 192;
constexpr int kWStageBytes = kTileN * kBlockK;
constexpr int kEpiBytes = 16 * 1024;               // epilogue transpose buffer [32 tokens][128 rows] FP32
constexpr int kSmemBudget = 227 * 1024 - 4096 - kEpiBytes;   // leaves room for the static barriers and the alignment pad

struct GemmW8Params {
  int M, Mp, NB, N, K;
  int mode;                // 0 = stream-K over 128-row tiles, 1 = one row band per CTA
  int groups8;             // ceil(N / gran): row groups divided over the CTAs in mode 1
  int gran;                // rows per group: 8 keeps every band 16-byte aligned in y, 1 balances the bands to one row
  int hmax;                // tallest band (box rows of tmap_w; tmap_w2 has hmax - gran)
  int w_chunk_bytes;       // shared-memory bytes reserved for one weight box (band rows x 128 B, 1 KB granules)
  int kw;                  // adjacent 128-byte K boxes per stage: each weight row is then read kw*128 B at a time
  int tma3d;               // 1: the kw boxes of a stage travel as ONE 3-D box {128 B, rows, kw} of a tensor map whose third
                           // dimension walks the 128-byte K blocks (needs K bytes % 128 == 0); 0: kw 2-D boxes
  int csplit;              // mode 2: CTAs per cluster = K slices per weight tile
  int pre_stages;          // stages whose weight boxes are requested before waiting for the preceding kernel
  int epi_off;             // byte offset of the epilogue's transpose buffer in dynamic shared memory
  int kb_rot_step;         // mode 1: CTA c starts its K loop at block (c * kb_rot_step) % kblocks
  int kblocks;             // K blocks per weight tile
  int num_tiles;
  long long total_blocks;  // num_tiles * kblocks
  int num_stages;
  int tmem_cols;
  int ytype;
  const float* w_scale;
  float* alpha;
  float* beta;
  void* y;
  int32_t* acc_dbg;
  int32_t* accum;          // [num_tiles][NB][128] split-K meeting place, zero between calls (INT32 or FP32 bits)
  unsigned* counters;      // [num_tiles]
  unsigned* status;
  long long* trace;        // nullable diagnostic buffer: 16 clock samples per CTA
};

// Grouped GEMM (MoE experts; Discussion, "Extension to MoE and Sparse Architectures"): the problems of one launch.  Group g multiplies the token rows
// [off[g], off[g] + m[g]) of x against expert expert[g]'s weight [N, K]; all groups share N, K and the kernel's tile shapes.
constexpr int kMaxGroups = 64;
struct GemmW8Groups {
  int n;                      // groups in this launch (0: not a grouped launch)
  int tiles_per_group;        // ceil(N / 128)
  int xq2_row0;               // row of the stacked-components buffer where the second components start
  int expert[kMaxGroups], off[kMaxGroups], m[kMaxGroups];
};

struct GemmW8NoGroups {};      // what the ungrouped instantiations take in its place: no parameter bytes to copy per launch
template <bool kGrouped> struct GroupArg { using type = GemmW8NoGroups; };
template <> struct GroupArg<true> { using type = GemmW8Groups; };

__device__ __forceinline__ void trace_mark(const GemmW8Params& p, int slot) {
  if (p.trace) p.trace[blockIdx.x * 16 + slot] = clock64();
}

__device__ __forceinline__ long long range_begin(long long cta, long long total, long long grid) {
  // 32-bit division when the product fits (every realistic size): the 64-bit one costs hundreds of cycles at kernel start
  if ((cta + 1) * total < (1LL << 32)) return static_cast<unsigned>(cta * total) / static_cast<unsigned>(grid);
  return cta * total / grid;
}
__device__ __forceinline__ long long block_owner(long long blk, long long total, long long grid) {
  return ((blk + 1) * grid - 1) / total;
}

// One chunk of W accumulator columns (= W tokens) of the final epilogue.  The sums come from TMEM (tile finished by this
// CTA alone) or from the split-K meeting place in global memory (which is read and left zeroed for the next call).
// A thread owns one weight row n, so its W results belong to W different rows of y; they are transposed through a
// 16 KB shared-memory buffer [W][128] and leave as full 16-byte vectors along n (2-byte scattered stores were the
// slowest part of the kernel at large M).  Called by the 128 epilogue threads together.
// Mode 2: where the partial sums of the other CTAs of the cluster were delivered in this CTA's shared memory.
// Slot s (from cluster rank s) holds [pass][token group of 4][128 weight rows][4 tokens] sums for this CTA's token
// range [t0, t0 + T): a warp's 16-byte accesses (one weight row per lane) cover 512 contiguous bytes, which is what
// both the remote stores and the local loads want.
struct RecvInfo {
  const int32_t* base;     // nullptr: nothing to add
  int S, self, slot_words, T, t0;
};

template <bool kBase, bool kBf16, int W>
__device__ __forceinline__ void epilogue_chunk(const GemmW8Params& p, uint32_t t_row, int32_t* acc_tile, int c0, int r, int n,
                                               bool row_ok, float sw, const float* s_alpha, const float* s_beta,
                                               uint8_t* stage_buf, int et, int n0, int rows_valid, const RecvInfo& rv,
                                               int m_valid, long long y_row0) {
  using OutT = typename std::conditional<kBf16, __nv_bfloat16, float>::type;
  constexpr int kEsz = static_cast<int>(sizeof(OutT));
  uint32_t a[W], b[W];
  float al[kBase ? 1 : W], be[kBase ? 1 : W];
  if (acc_tile == nullptr) {
    tmem_ldw<W>(t_row + c0, a);
    if constexpr (!kBase) tmem_ldw<W>(t_row + p.Mp + c0, b);
  }
  if constexpr (!kBase) {
    // the per-token scales of the chunk, fetched as vectors up front: read one by one inside the loop below they
    // would each wait for the preceding shared-memory store (possible aliasing) with nothing to hide the latency
#pragma unroll
    for (int j = 0; j < W; j += 4) {
      const float4 va = *reinterpret_cast<const float4*>(s_alpha + c0 + j);
      const float4 vb = *reinterpret_cast<const float4*>(s_beta + c0 + j);
      al[j] = va.x; al[j + 1] = va.y; al[j + 2] = va.z; al[j + 3] = va.w;
      be[j] = vb.x; be[j + 1] = vb.y; be[j + 2] = vb.z; be[j + 3] = vb.w;
    }
  }
  if (acc_tile == nullptr) {
    tmem_ld_wait();
    if (rv.base != nullptr) {
      // the other K slices of this tile, in cluster-rank order (a fixed order: the FP32 sums of the comparison
      // path come out the same on every run)
      for (int s = 0; s < rv.S; ++s) {
        if (s == rv.self) continue;
        const int32_t* q = rv.base + (s < rv.self ? s : s - 1) * rv.slot_words + ((c0 - rv.t0) >> 2) * (kTileN * 4) + r * 4;
#pragma unroll
        for (int j = 0; j < W; j += 4) {
          const int4 va = *reinterpret_cast<const int4*>(q + (j >> 2) * (kTileN * 4));
          if constexpr (kBase) {
            a[j] = __float_as_uint(__uint_as_float(a[j]) + __int_as_float(va.x));
            a[j + 1] = __float_as_uint(__uint_as_float(a[j + 1]) + __int_as_float(va.y));
            a[j + 2] = __float_as_uint(__uint_as_float(a[j + 2]) + __int_as_float(va.z));
            a[j + 3] = __float_as_uint(__uint_as_float(a[j + 3]) + __int_as_float(va.w));
          } else {
            const int4 vb = *reinterpret_cast<const int4*>(q + rv.T * kTileN + (j >> 2) * (kTileN * 4));
            a[j] += static_cast<uint32_t>(va.x); a[j + 1] += static_cast<uint32_t>(va.y);
            a[j + 2] += static_cast<uint32_t>(va.z); a[j + 3] += static_cast<uint32_t>(va.w);
            b[j] += static_cast<uint32_t>(vb.x); b[j + 1] += static_cast<uint32_t>(vb.y);
            b[j + 2] += static_cast<uint32_t>(vb.z); b[j + 3] += static_cast<uint32_t>(vb.w);
          }
        }
      }
    }
  } else {
#pragma unroll
    for (int j = 0; j < W; ++j) {
      a[j] = static_cast<uint32_t>(__ldcg(acc_tile + (c0 + j) * kTileN + r));
      if constexpr (!kBase) b[j] = static_cast<uint32_t>(__ldcg(acc_tile + (p.Mp + c0 + j) * kTileN + r));
    }
#pragma unroll
    for (int j = 0; j < W; ++j) {
      __stcg(acc_tile + (c0 + j) * kTileN + r, 0);
      if constexpr (!kBase) __stcg(acc_tile + (p.Mp + c0 + j) * kTileN + r, 0);
    }
  }
  OutT* stage = reinterpret_cast<OutT*>(stage_buf);
#pragma unroll
  for (int j = 0; j < W; ++j) {
    float v;
    if constexpr (kBase) {
      v = __uint_as_float(a[j]);
    } else {
      const int32_t ya = static_cast<int32_t>(a[j]), yb = static_cast<int32_t>(b[j]);
      // y = s_W * (alpha * Y1 + beta * Y2)   (Alg. 1 line 8)
      v = sw * __fmaf_rn(al[j], static_cast<float>(ya), be[j] * static_cast<float>(yb));
    }
    if constexpr (kBf16) stage[j * kTileN + r] = __float2bfloat16_rn(v);
    else stage[j * kTileN + r] = v;
  }
  if constexpr (!kBase) {
    if (p.acc_dbg && row_ok) {
#pragma unroll
      for (int j = 0; j < W; ++j) {
        const int i = c0 + j;
        if (i < p.M) {
          const long long idx = static_cast<long long>(i) * p.N + n;
          p.acc_dbg[idx] = static_cast<int32_t>(a[j]);
          p.acc_dbg[static_cast<long long>(p.M) * p.N + idx] = static_cast<int32_t>(b[j]);
        }
      }
    }
  }
  named_bar_sync(1, 128);
  const int wm = min(W, m_valid - c0);                           // tokens of this chunk that exist
  int nv = min(rows_valid, p.N - n0);                            // weight rows of this tile / band that exist
  if (nv < 0) nv = 0;
  OutT* y = static_cast<OutT*>(p.y);
  const bool vec_ok = ((static_cast<long long>(p.N) * kEsz) & 15) == 0 && ((static_cast<long long>(n0) * kEsz) & 15) == 0;
  if (vec_ok) {
    constexpr int kEpv = 16 / kEsz, kSegs = kTileN / kEpv;
    const int sg = et % kSegs, nf = sg * kEpv;
    if (nf + kEpv <= nv) {
#pragma unroll 4
      for (int j = et / kSegs; j < wm; j += 128 / kSegs) {
        const uint4 val = *reinterpret_cast<const uint4*>(stage + j * kTileN + nf);
        *reinterpret_cast<uint4*>(y + (y_row0 + c0 + j) * p.N + n0 + nf) = val;
      }
    } else if (nf < nv) {
      for (int j = et / kSegs; j < wm; j += 128 / kSegs)
        for (int e = nf; e < nv; ++e) y[(y_row0 + c0 + j) * p.N + n0 + e] = stage[j * kTileN + e];
    }
  } else {
    if (et < nv)
      for (int j = 0; j < wm; ++j) y[(y_row0 + c0 + j) * p.N + n0 + et] = stage[j * kTileN + et];
  }
  named_bar_sync(1, 128);            // the buffer is free for the next chunk
}

// The token chunks [tok0, tok1) of one finished tile (both multiples of 8).
template <bool kBase, bool kBf16>
__device__ __forceinline__ void epilogue_tile(const GemmW8Params& p, uint32_t t_row, int32_t* acc_tile, int r, int n, bool row_ok,
                                              float sw, const float* s_alpha, const float* s_beta, uint8_t* stage_buf, int et,
                                              int n0, int rows_valid, int tok0, int tok1, const RecvInfo& rv, int m_valid,
                                              long long y_row0) {
  int c0 = tok0;
  if constexpr (kBase)
    for (; c0 + 32 <= tok1; c0 += 32)
      epilogue_chunk<kBase, kBf16, 32>(p, t_row, acc_tile, c0, r, n, row_ok, sw, s_alpha, s_beta, stage_buf, et, n0, rows_valid, rv, m_valid, y_row0);
  for (; c0 + 16 <= tok1; c0 += 16)      // 16 tokens at a time: two sums and two scales per token stay in registers
    epilogue_chunk<kBase, kBf16, 16>(p, t_row, acc_tile, c0, r, n, row_ok, sw, s_alpha, s_beta, stage_buf, et, n0, rows_valid, rv, m_valid, y_row0);
  for (; c0 + 8 <= tok1; c0 += 8)
    epilogue_chunk<kBase, kBf16, 8>(p, t_row, acc_tile, c0, r, n, row_ok, sw, s_alpha, s_beta, stage_buf, et, n0, rows_valid, rv, m_valid, y_row0);
}

// Adds W accumulator columns of a partial tile into the split-K meeting place (reductions without return value).
template <bool kBase, int W>
__device__ __forceinline__ void partial_chunk(uint32_t t_row, int32_t* acc_tile, int c0, int r) {
  uint32_t v[W];
  tmem_ldw<W>(t_row + c0, v);
  tmem_ld_wait();
#pragma unroll
  for (int j = 0; j < W; ++j) {
    if constexpr (kBase) atomicAdd(reinterpret_cast<float*>(acc_tile) + (c0 + j) * kTileN + r, __uint_as_float(v[j]));
    else atomicAdd(acc_tile + (c0 + j) * kTileN + r, static_cast<int32_t>(v[j]));
  }
}

// kBase = false: the MSD path (INT8 x INT8 -> INT32, stacked components, scale-combine epilogue).
// kBase = true : the comparison path the method replaces - the same pipeline on BF16 weights that a preceding kernel
//                dequantized into the workspace, BF16 x BF16 -> FP32, no decomposition and no scales in the epilogue.
// kGrouped: several (token rows, expert weight) problems in one stream-K launch; the group table travels as a kernel
//                parameter, weight tiles are addressed in the stacked [E*N, K] weight, the two components of a
//                group's rows come as two boxes of the component buffer.
template <bool kBase, bool kGrouped = false>
__global__ void __launch_bounds__(kGemmThreads, 1)
gemm_w8a16_kernel(const __grid_constant__ CUtensorMap tmap_w, const __grid_constant__ CUtensorMap tmap_w2,
                  const __grid_constant__ CUtensorMap tmap_x, const GemmW8Params p,
                  const __grid_constant__ typename GroupArg<kGrouped>::type grp) {
  extern __shared__ uint8_t smem_dyn[];
  __shared__ __align__(8) uint64_t full_bar[kMaxStages];
  __shared__ __align__(8) uint64_t empty_bar[kMaxStages];
  __shared__ __align__(8) uint64_t tfull_bar[2];
  __shared__ __align__(8) uint64_t tempty_bar[2];
  __shared__ __align__(8) uint64_t cfree_bar, crecv_bar, cdone_bar;
  __shared__ float s_red[4];      // mode 2: "pipelines of the cluster drained", "partials delivered"
  __shared__ uint32_t tmem_base_slot;
  __shared__ int abort_flag;
  __shared__ int is_last_flag;
  __shared__ __align__(16) float s_alpha[128], s_beta[128];

  const int warp = threadIdx.x >> 5;
  const int lane = threadIdx.x & 31;
  if (p.num_stages < 1 || p.kw < 1 || p.kblocks < 1) return;     // malformed plan: touch nothing
  // lets a decomposition kernel queued behind this GEMM become resident early (it still waits for this grid to finish)
  pdl_launch_dependents();
  if (threadIdx.x == 64) {       // first thing: the descriptor fetches are on the way to the first copy
    tma_prefetch_desc(&tmap_w);
    tma_prefetch_desc(&tmap_w2);
    tma_prefetch_desc(&tmap_x);
  }
  if (threadIdx.x == 0 && p.trace) {
    trace_mark(p, 0);
    unsigned long long g;
    asm volatile("mov.u64 %0, %globaltimer;" : "=l"(g));
    p.trace[blockIdx.x * 16 + 1] = static_cast<long long>(g);
  }
  uint8_t* smem = reinterpret_cast<uint8_t*>((reinterpret_cast<uintptr_t>(smem_dyn) + 1023) & ~static_cast<uintptr_t>(1023));
  uint8_t* epi_buf = smem + p.epi_off;             // 16 KB transpose buffer of the epilogue, after the pipeline stages
  const int x_chunk_bytes = p.NB * kBlockK;

  const long long grid = gridDim.x;
  // mode 0: this CTA's slice of the tile-major (tile, K block) sequence; mode 1: its row band and every K block
  long long blk_begin, blk_end;
  int band_row0 = 0, band_h = kTileN;
  if (p.mode == 0) {
    blk_begin = range_begin(blockIdx.x, p.total_blocks, grid);
    blk_end = range_begin(blockIdx.x + 1, p.total_blocks, grid);
  } else if (p.mode == 2) {
    // a cluster of csplit CTAs per weight tile, CTA `rank` of it takes the rank-th slice of the tile's K blocks
    const int tile2 = blockIdx.x / p.csplit, rank = blockIdx.x - tile2 * p.csplit;
    blk_begin = static_cast<long long>(tile2) * p.kblocks + rank * p.kblocks / p.csplit;
    blk_end = static_cast<long long>(tile2) * p.kblocks + (rank + 1) * p.kblocks / p.csplit;
  } else {
    const int g0 = static_cast<int>(range_begin(blockIdx.x, p.groups8, grid));
    const int g1 = static_cast<int>(range_begin(blockIdx.x + 1, p.groups8, grid));
    band_row0 = p.gran * g0;
    band_h = p.gran * (g1 - g0);
    blk_begin = 0;
    blk_end = p.kblocks;
  }
  // One weight box in shared memory: a 3-D box packs its kw chunks back to back at this CTA's own band height (a
  // multiple of 8 rows, so every chunk still starts on a 1 KB swizzle atom); 2-D boxes sit at the plan's stride.
  const int w_chunk = (p.tma3d && p.mode == 1) ? band_h * kBlockK : p.w_chunk_bytes;
  const int w_stage_bytes = p.kw * w_chunk;
  const int stage_bytes = w_stage_bytes + p.kw * x_chunk_bytes;
  // Mode 1: every CTA walks K from its own starting block so that concurrent requests of the CTAs spread over the
  // whole row instead of hitting the same 128-byte column of every row (integer sums do not depend on the order).
  const int kb_rot = (p.mode == 1) ? static_cast<int>((static_cast<long long>(blockIdx.x) * p.kb_rot_step) % p.kblocks) : 0;
  const CUtensorMap* wmap = (p.mode == 1 && band_h != p.hmax) ? &tmap_w2 : &tmap_w;
  const int tx_bytes = p.kw * ((p.mode == 0 ? kWStageBytes : band_h * kBlockK) + x_chunk_bytes);

  // the barriers of the pipeline stages one stage per lane of the producer warp, the others by its first lane
  if (warp == 0 && lane < p.num_stages) {
    mbar_init(&full_bar[lane], 1);
    mbar_init(&empty_bar[lane], 1);
  }
  if (threadIdx.x == 0) {
    for (int a = 0; a < 2; ++a) {
      mbar_init(&tfull_bar[a], 1);
      mbar_init(&tempty_bar[a], 4);      // one arrival per epilogue warp
    }
    if (p.mode == 2) {
      mbar_init(&cfree_bar, p.csplit);               // one arrival per CTA of the cluster
      mbar_init(&crecv_bar, 1);                      // this CTA's own arrival; the peers' copies count in bytes
      {
        // finishing CTAs this one sends to: each lets it know when its copy has landed
        const int G8i = p.Mp >> 3, Fi = p.csplit < G8i ? p.csplit : G8i;
        const int ranki = static_cast<int>(blockIdx.x) % p.csplit;
        const int n_to = Fi - (ranki < Fi ? 1 : 0);
        mbar_init(&cdone_bar, n_to > 0 ? n_to : 1);
      }
    }
    abort_flag = 0;
  }
  if (warp == 0) {
    mbar_init_fence();
    __syncwarp();
  }
  // ------------------------------ TMA producer, first part ------------------------------
  // Runs before the CTA-wide barrier below: the thread that initialised the mbarriers is in this warp, and the sooner
  // the first weight boxes are requested the sooner the stream from HBM starts.
  uint64_t pol_w = 0, pol_x = 0;
  bool w_lane = false, x_lane = false;
  int c = 0, x_half = 0, tile = 0, kbi = 0, kbr = 0, kbr0 = 0, pre = 0, pre0 = 0, tile_first = 0, kbi_first = 0;
  // first weight row of a tile in the weight tensor, and first row of its stacked components in the component buffer
  auto w_row = [&](int t) -> int {
    if constexpr (kGrouped) {
      const int g = t / grp.tiles_per_group;
      return grp.expert[g] * p.N + (t - g * grp.tiles_per_group) * kTileN;
    } else {
      return band_row0 + t * kTileN;
    }
  };
  auto x_row = [&](int t) -> int {
    if constexpr (kGrouped) return grp.off[t / grp.tiles_per_group] + x_half * grp.xq2_row0;
    else return 0;
  };
  const int x_half_bytes = kGrouped ? p.Mp * kBlockK : 0;
  auto advance = [&]() {
    if (++kbi == p.kblocks) { kbi = 0; ++tile; }
    if (++kbr == p.kblocks) kbr = 0;
  };
  // the weight box(es) / component box(es) of K block `kblk` (in units of stages) into stage memory at `dst`
  auto load_w = [&](uint8_t* dst, int kblk, int row, uint64_t* bar) {
    if (p.tma3d) tma_load_3d_hint(dst, wmap, 0, row, kblk * p.kw, bar, pol_w);
    else tma_load_2d_hint(dst + c * w_chunk, wmap, (kblk * p.kw + c) * kBlockK, row, bar, pol_w);
  };
  auto load_x = [&](uint8_t* dst, int kblk, int row, uint64_t* bar) {
    if (p.tma3d && !kGrouped) tma_load_3d_hint(dst + w_stage_bytes, &tmap_x, 0, row, kblk * p.kw, bar, pol_x);
    else tma_load_2d_hint(dst + w_stage_bytes + c * x_chunk_bytes + x_half * x_half_bytes, &tmap_x, (kblk * p.kw + c) * kBlockK, row, bar, pol_x);
  };
  if (warp == 0) {
    __syncwarp();
    // The whole warp takes part: lane 0 owns the barriers, lanes [0, kw) each issue one weight box of a stage and
    // lanes [kw, 2 kw) one box of the stacked components, so the copies of a stage are issued side by side instead
    // of one after another by a single thread.
    pol_w = policy_evict_first();    // weights are streamed once
    pol_x = policy_evict_last();      // the stacked components are re-read by every CTA
    w_lane = lane < (p.tma3d ? 1 : p.kw);
    x_lane = lane >= p.kw && lane < (kGrouped ? 3 : 2) * p.kw;     // grouped: one box per component
    if (p.tma3d && !kGrouped) x_lane = lane == p.kw;              // one 3-D box of the stacked components per stage
    c = w_lane ? lane : (lane - p.kw) % p.kw;
    x_half = w_lane ? 0 : (lane - p.kw) / p.kw;
    // (tile, K block) of the next block to load, advanced by one per stage; kbr = rotated K block
    const int tile0 = blk_begin < (1LL << 32) ? static_cast<int>(static_cast<unsigned>(blk_begin) / static_cast<unsigned>(p.kblocks))
                                              : static_cast<int>(blk_begin / p.kblocks);
    const int kbi0 = static_cast<int>(blk_begin - static_cast<long long>(tile0) * p.kblocks);
    tile = tile0; kbi = kbi0;
    tile_first = tile0; kbi_first = kbi0;
    kbr = kbi + kb_rot;
    if (kbr >= p.kblocks) kbr -= p.kblocks;
    kbr0 = kbr;
    // Weight tiles of the first stages do not depend on the decomposition kernel: issue them before waiting for it.
    const long long nblk = blk_end - blk_begin;
    pre = static_cast<int>(nblk < p.num_stages ? nblk : p.num_stages);
    pre0 = pre < p.pre_stages ? pre : p.pre_stages;
    if constexpr (kBase) pdl_wait_primary();     // here the weights themselves come from the preceding kernel
    for (int i = 0; i < pre0; ++i) {
      if (lane == 0) mbar_arrive_expect_tx(&full_bar[i], tx_bytes);
      __syncwarp();
      if (w_lane) load_w(smem + i * stage_bytes, kbr, w_row(tile), &full_bar[i]);
      advance();
    }
    if (lane == 0) trace_mark(p, 3);
  }
  if (warp == 1) tmem_alloc(&tmem_base_slot, p.tmem_cols);
  tc_fence_before();
  if (p.mode == 2) cluster_arrive_all();    // "my barriers are initialised": the epilogue warps wait for the peers' before their first remote arrive
  __syncthreads();
  tc_fence_after();
  const uint32_t tmem_base = tmem_base_slot;
  volatile int* abort = &abort_flag;
  if (threadIdx.x == 0) trace_mark(p, 2);

  if (warp == 0) {
    pdl_wait_primary();
    if (lane == 0) trace_mark(p, 4);
    {
      int kx = kbr0;
      for (int i = 0; i < pre; ++i) {
        if (i >= pre0) {     // weight boxes held back so that the wait above was not queued behind them
          if (lane == 0) mbar_arrive_expect_tx(&full_bar[i], tx_bytes);
          __syncwarp();
          if (w_lane) load_w(smem + i * stage_bytes, kbr, w_row(tile), &full_bar[i]);
          advance();
        }
        if (x_lane) load_x(smem + i * stage_bytes, kx, x_row(tile_first + (kbi_first + i) / p.kblocks), &full_bar[i]);
        if (++kx == p.kblocks) kx = 0;
      }
    }
    int stage = pre % p.num_stages;
    uint32_t phase = (pre == p.num_stages) ? 1 : 0;
    bool ok = true;
    for (long long blk = blk_begin + pre; blk < blk_end; ++blk) {
      if (lane == 0) {
        ok = wait_bounded(&empty_bar[stage], phase ^ 1, abort, p.status);
        if (ok) mbar_arrive_expect_tx(&full_bar[stage], tx_bytes);
      }
      ok = __shfl_sync(0xffffffffu, ok ? 1 : 0, 0) != 0;
      if (!ok) break;
      uint8_t* dst = smem + stage * stage_bytes;
      if (w_lane) load_w(dst, kbr, w_row(tile), &full_bar[stage]);
      else if (x_lane) load_x(dst, kbr, x_row(tile), &full_bar[stage]);
      advance();
      if (++stage == p.num_stages) { stage = 0; phase ^= 1; }
    }
    if (lane == 0) trace_mark(p, 5);
    if (!ok) {
      // give copies already in flight a bounded time to land before the CTA goes away
      const long long t0 = clock64();
      while (clock64() - t0 < 2000000LL) {}
    }
  } else if (warp == 1) {
    // ------------------------------ MMA issuer ------------------------------
    if (lane == 0) {
      const uint32_t idesc = kBase ? idesc_dense(/*D=F32*/ 1, /*A=BF16*/ 1, /*B=BF16*/ 1, 0, 0, kTileN, p.NB)
                                   : idesc_dense(/*D=S32*/ 2, /*A=S8*/ 1, /*B=S8*/ 1, 0, 0, kTileN, p.NB);
      int stage = 0;
      uint32_t phase = 0;
      int seg = 0;
      bool ok = true;
      long long blk = blk_begin;
      while (blk < blk_end && ok) {
        const int tile = static_cast<int>(blk / p.kblocks);
        const long long tile_end = static_cast<long long>(tile + 1) * p.kblocks;
        const long long seg_end = tile_end < blk_end ? tile_end : blk_end;
        const int acc = seg & 1;
        ok = wait_bounded(&tempty_bar[acc], ((seg >> 1) & 1) ^ 1, abort, p.status);
        if (!ok) break;
        tc_fence_after();
        const uint32_t d_tmem = tmem_base + acc * p.NB;
        for (long long b = blk; b < seg_end; ++b) {
          ok = wait_bounded(&full_bar[stage], phase, abort, p.status);
          if (!ok) break;
          if (b == blk_begin) trace_mark(p, 6);
          tc_fence_after();
          const uint32_t wa = smem_u32(smem + stage * stage_bytes);
          const uint32_t xa = wa + w_stage_bytes;     // the MMA reads 128 A rows; rows past the band are never used
          for (int c = 0; c < p.kw; ++c) {
#pragma unroll
            for (int k = 0; k < kBlockK / 32; ++k) {
              const uint64_t adesc = smem_desc(wa + c * w_chunk + k * 32, 16, 1024, kSwizzle128B);
              const uint64_t bdesc = smem_desc(xa + c * x_chunk_bytes + k * 32, 16, 1024, kSwizzle128B);
              const uint32_t accum = (b > blk || c > 0 || k > 0) ? 1u : 0u;
              if constexpr (kBase) mma_f16(d_tmem, adesc, bdesc, idesc, accum);
              else mma_i8(d_tmem, adesc, bdesc, idesc, accum);
            }
          }
          tc_commit(&empty_bar[stage]);          // frees the stage once these MMAs have read it
          if (++stage == p.num_stages) { stage = 0; phase ^= 1; }
        }
        if (!ok) break;
        tc_commit(&tfull_bar[acc]);              // accumulator of this segment complete
        ++seg;
        blk = seg_end;
      }
      trace_mark(p, 7);
    }
  } else {
    // ------------------------------ epilogue (warps 2..5) ------------------------------
    const int quad = warp & 3;                    // TMEM lane group this warp may read
    const int r = quad * 32 + lane;               // weight row within the tile == TMEM lane
    const int et = threadIdx.x - 64;              // 0..127
    if constexpr (!kBase) {
      pdl_wait_primary();
      if (!kGrouped && et < p.M) {
        s_alpha[et] = __ldcg(p.alpha + et);
        s_beta[et] = __ldcg(p.beta + et);
      }
    }
    named_bar_sync(1, 128);
    int seg = 0;
    int sent_to = 0;           // mode 2: finishing CTAs whose acknowledgement is outstanding
    bool ok = true;
    long long blk = blk_begin;
    while (blk < blk_end && ok) {
      const int tile = static_cast<int>(blk / p.kblocks);
      const long long tile_begin = static_cast<long long>(tile) * p.kblocks;
      const long long tile_end = tile_begin + p.kblocks;
      const long long seg_end = tile_end < blk_end ? tile_end : blk_end;
      const bool complete = (blk == tile_begin) && (seg_end == tile_end);
      const int acc = seg & 1;
      // weight row within its matrix; grouped: also which rows of x / y and which expert's scales this tile is about
      int n = band_row0 + tile * kTileN + r;
      int m_valid = p.M;
      long long y_row0 = 0, sw_row0 = 0;
      if constexpr (kGrouped) {
        const int g = tile / grp.tiles_per_group;
        n = (tile - g * grp.tiles_per_group) * kTileN + r;
        m_valid = grp.m[g];
        y_row0 = grp.off[g];
        sw_row0 = static_cast<long long>(grp.expert[g]) * p.N;
      }
      const bool row_ok = (r < band_h) && (n < p.N);
      // requested before the wait for the accumulator: a cold read of the scale array would otherwise be the call's tail
      const float sw = (!kBase && row_ok) ? __ldg(p.w_scale + sw_row0 + n) : 0.0f;
      ok = wait_bounded(&tfull_bar[acc], (seg >> 1) & 1, abort, p.status);
      if (!ok) break;
      if (et == 0) { if (seg == 0) trace_mark(p, 8); trace_mark(p, 9); }
      tc_fence_after();
      const uint32_t t_row = tmem_base + (static_cast<uint32_t>(quad * 32) << 16) + acc * p.NB;
      bool finish = complete;
      int32_t* acc_tile = nullptr;
      int tok0 = 0, tok1 = p.Mp;
      RecvInfo rv = {nullptr, 0, 0, 0, 0, 0};
      if (p.mode == 2 && p.csplit > 1) {
        // ---- split-K inside a cluster: partial sums travel through the peers' shared memory ----
        // Finishing is shared out as well: owner f < F completes the tokens of its groups of 8 for the whole tile.
        const int S = p.csplit, rank = static_cast<int>(blockIdx.x) - tile * S;
        const int G8 = p.Mp >> 3, F = S < G8 ? S : G8;
        const int tmax = 8 * ((G8 + F - 1) / F);
        const int passes = kBase ? 1 : 2;
        const int slot_words = passes * tmax * kTileN;
        // shared memory of the drained pipeline: S-1 incoming slots (one per peer), then the outgoing staging slots
        uint8_t* stage_out = smem + static_cast<size_t>(S - 1) * slot_words * 4;
        // 1. this CTA's own MMAs are complete, so it may overwrite its own buffers: stage what the others will finish
        int oi = 0;
        for (int f = 0; f < F; ++f) {
          if (f == rank) continue;
          const int ft0 = 8 * (f * G8 / F), ft1 = 8 * ((f + 1) * G8 / F), fT = ft1 - ft0;
          uint8_t* so = stage_out + static_cast<size_t>(oi) * slot_words * 4;
          for (int ps = 0; ps < passes; ++ps) {
            uint8_t* srow = so + static_cast<size_t>(ps * fT * kTileN + r * 4) * 4;
            for (int c = ft0; c < ft1; c += 32) {
              const int nc = ft1 - c < 32 ? ft1 - c : 32;     // up to 32 columns per round, their TMEM loads in flight together
              uint32_t v[4][8];
#pragma unroll
              for (int g = 0; g < 4; ++g)
                if (g * 8 < nc) tmem_ld8(t_row + ps * p.Mp + c + g * 8, v[g]);
              tmem_ld_wait();
#pragma unroll
              for (int g = 0; g < 4; ++g) {
                if (g * 8 < nc) {
                  uint8_t* d = srow + static_cast<size_t>(((c - ft0 + g * 8) >> 2) * (kTileN * 4)) * 4;
                  *reinterpret_cast<uint4*>(d) = make_uint4(v[g][0], v[g][1], v[g][2], v[g][3]);
                  *reinterpret_cast<uint4*>(d + kTileN * 16) = make_uint4(v[g][4], v[g][5], v[g][6], v[g][7]);
                }
              }
            }
          }
          ++oi;
        }
        fence_proxy_async_smem();               // the copy engine reads what these threads wrote
        finish = rank < F;
        if (finish) {
          tok0 = 8 * (rank * G8 / F);
          tok1 = 8 * ((rank + 1) * G8 / F);
          // bytes this CTA is going to receive (posted before any peer can start sending)
          if (et == 0) mbar_arrive_expect_tx(&crecv_bar, static_cast<uint32_t>((S - 1) * passes * (tok1 - tok0) * kTileN * 4));
        }
        named_bar_sync(1, 128);
        // 2. the pipelines of all CTAs of the cluster are drained: tell every CTA (itself included), wait for all
        cluster_wait_all();                     // every CTA of the cluster has initialised its barriers
        if (et < S) mbar_arrive_cluster(mapa_shared(smem_u32(&cfree_bar), et));
        ok = wait_bounded_cluster(&cfree_bar, 0, abort, p.status);
        if (!ok) break;
        // 3. one bulk copy per finishing peer, straight into its slot for this rank
        if (et == 0) {
          oi = 0;
          for (int f = 0; f < F; ++f) {
            if (f == rank) continue;
            const int fT = 8 * ((f + 1) * G8 / F) - 8 * (f * G8 / F);
            const int slot = rank < f ? rank : rank - 1;
            bulk_copy_to_peer(mapa_shared(smem_u32(smem) + static_cast<uint32_t>(slot * slot_words) * 4u, f),
                              stage_out + static_cast<size_t>(oi) * slot_words * 4,
                              static_cast<uint32_t>(passes * fT * kTileN * 4), mapa_shared(smem_u32(&crecv_bar), f));
            ++oi;
          }
        }
        if (finish) {
          ok = wait_bounded_cluster(&crecv_bar, 0, abort, p.status);
          if (!ok) break;
          // the senders may let go of their staging buffers (and exit)
          if (et < S && et != rank) mbar_arrive_cluster(mapa_shared(smem_u32(&cdone_bar), et));
          rv.base = reinterpret_cast<const int32_t*>(smem);
          rv.S = S; rv.self = rank; rv.slot_words = slot_words; rv.T = tok1 - tok0; rv.t0 = tok0;
        }
        sent_to = F - (rank < F ? 1 : 0);
      } else if (!complete) {
        // add this CTA's partial sums into the tile's meeting place, then find out whether it was the last contributor
        acc_tile = p.accum + static_cast<long long>(tile) * p.NB * kTileN;
        int c0 = 0;
        for (; c0 + 32 <= p.NB; c0 += 32) partial_chunk<kBase, 32>(t_row, acc_tile, c0, r);
        if (c0 + 16 <= p.NB) partial_chunk<kBase, 16>(t_row, acc_tile, c0, r);
        named_bar_sync(1, 128);
        if (et == 0) {
          const int c_lo = static_cast<int>(block_owner(tile_begin, p.total_blocks, grid));
          const int c_hi = static_cast<int>(block_owner(tile_end - 1, p.total_blocks, grid));
          __threadfence();     // cumulative: publishes the additions of all 128 threads ordered by the barrier above
          const unsigned prev = atomicAdd(&p.counters[tile], 1u);
          const int last = (prev == static_cast<unsigned>(c_hi - c_lo)) ? 1 : 0;
          if (last) p.counters[tile] = 0;          // leave the counter ready for the next call
          is_last_flag = last;
        }
        named_bar_sync(1, 128);
        finish = is_last_flag != 0;
        if (finish) __threadfence();
      }
      if (finish) {
        if constexpr (kGrouped) {
          // the scales of this group's token rows (the previous tile's epilogue has finished reading the old ones)
          named_bar_sync(1, 128);
          if (et < m_valid) {
            s_alpha[et] = __ldcg(p.alpha + y_row0 + et);
            s_beta[et] = __ldcg(p.beta + y_row0 + et);
          }
          named_bar_sync(1, 128);
        }
        if (p.ytype == MSD_OUT_BF16)
          epilogue_tile<kBase, true>(p, t_row, acc_tile, r, n, row_ok, sw, s_alpha, s_beta, epi_buf, et, n - r, band_h, tok0, tok1, rv,
                                             m_valid, y_row0);
        else
          epilogue_tile<kBase, false>(p, t_row, acc_tile, r, n, row_ok, sw, s_alpha, s_beta, epi_buf, et, n - r, band_h, tok0, tok1, rv,
                                              m_valid, y_row0);
      }
      tc_fence_before();
      __syncwarp();
      if (lane == 0) mbar_arrive(&tempty_bar[acc]);
      ++seg;
      blk = seg_end;
    }
    // mode 2: the staging buffers must outlive the copies that read them
    if (sent_to > 0 && ok) wait_bounded_cluster(&cdone_bar, 0, abort, p.status);
    if (et == 0) { trace_mark(p, 10); if (p.trace) p.trace[blockIdx.x * 16 + 11] = seg; }
  }

  tc_fence_before();
  __syncthreads();
  if (threadIdx.x == 0 && p.trace) {
    trace_mark(p, 12);
    unsigned long long g;
    asm volatile("mov.u64 %0, %globaltimer;" : "=l"(g));
    p.trace[blockIdx.x * 16 + 13] = static_cast<long long>(g);
  }
  if (warp == 1) {
    tc_fence_after();
    tmem_dealloc(tmem_base, p.tmem_cols);
  }
}

static long long* g_trace = nullptr;

static int pow2_at_least(int v) {
  int p = 32;
  while (p < v) p <<= 1;
  return p;
}

struct GemmW8Plan {
  int Mp, NB, kblocks, num_tiles, grid, stages, tmem_cols;
  int mode, groups8, gran, hmax, w_chunk_bytes, kw, epi_off, csplit;
  long long total_blocks;
  size_t off_q, off_alpha, off_beta, off_counters, off_slots, bytes;
  size_t smem_bytes;
};

// `base`: plan for the dequantize-to-BF16 comparison path (K counted in bytes of BF16, one operand row per token).
// How many clusters of S CTAs of the GEMM kernel the device can hold at once (cached per configuration); 0 on error.
static int max_resident_clusters(bool base, int S, size_t smem_bytes);

static GemmW8Plan plan_w8(int64_t M, int64_t N, int64_t K, bool base = false) {
  GemmW8Plan pl;
  pl.Mp = base ? static_cast<int>((M + 15) / 16 * 16) : static_cast<int>((M + 7) / 8 * 8);
  pl.NB = base ? pl.Mp : 2 * pl.Mp;
  const int64_t kbytes = base ? 2 * K : K;
  // K boxes per stage: wide stages read each weight row in runs of kw*128 bytes (good for DRAM page locality);
  // the operand tile of the stacked components grows with kw too, so wide activations get narrower stages.
  int kw = (pl.NB <= 64) ? 4 : 2;
  while (kw > 1 && static_cast<int64_t>(kw) * kBlockK > kbytes) kw >>= 1;
  pl.kw = kw;
  pl.kblocks = static_cast<int>((kbytes + static_cast<int64_t>(kw) * kBlockK - 1) / (static_cast<int64_t>(kw) * kBlockK));
  pl.num_tiles = static_cast<int>((N + kTileN - 1) / kTileN);
  pl.total_blocks = static_cast<long long>(pl.kblocks) * pl.num_tiles;
  // Row bands of mode 1 come in two heights that differ by one group.  Groups of 8 rows keep every band on a 16-byte
  // boundary of y (vector stores); balancing the bands to a single row measured no faster.
  pl.gran = 8;
  pl.groups8 = static_cast<int>((N + pl.gran - 1) / pl.gran);
  const int sms = sm_count();
  int grid = option(OPT_GEMM_CTAS);       // testing aid: a given number of CTAs
  if (grid < 1) grid = sms;
  if (grid > 256) grid = 256;
  // Row partition pays when every SM gets a band of at least 64 rows (the MMA always spans 128 rows, so shorter
  // bands waste tensor time and TMA rows on the shared activation tile) and the bands still fit one MMA.
  const int band_max = pl.gran * ((pl.groups8 + grid - 1) / grid);
  const int band_min = pl.gran * (pl.groups8 / grid);
  int mode = (band_min >= 64 && band_max <= kTileN) ? 1 : 0;
  const int mode_env = option(OPT_GEMM_MODE);            // testing aid: 0 / 1 / 2 force a schedule where it is feasible
  if (mode_env == 0 || mode_env == 1) mode = mode_env;
  if (mode_env == 2) mode = 0;
  if (mode == 1 && (band_max > kTileN || band_min < 8)) mode = 0;
  pl.mode = mode;
  if (mode == 1) {
    pl.hmax = band_max;
    pl.w_chunk_bytes = static_cast<int>(round_up(static_cast<size_t>(band_max) * kBlockK, 1024));
  } else {
    if (grid > pl.total_blocks) grid = static_cast<int>(pl.total_blocks);
    pl.hmax = kTileN;
    pl.w_chunk_bytes = kWStageBytes;
  }
  pl.grid = grid;
  const int tail_pad = kWStageBytes - pl.w_chunk_bytes;     // the MMA reads a full 128-row A tile from every box
  // at least two stages must fit: narrow the stage (and recount the K blocks) until they do
  int stage_bytes = pl.kw * (pl.w_chunk_bytes + pl.NB * kBlockK);
  while (pl.kw > 1 && (kSmemBudget - tail_pad) / stage_bytes < 2) {
    pl.kw >>= 1;
    stage_bytes = pl.kw * (pl.w_chunk_bytes + pl.NB * kBlockK);
  }
  pl.kblocks = static_cast<int>((kbytes + static_cast<int64_t>(pl.kw) * kBlockK - 1) / (static_cast<int64_t>(pl.kw) * kBlockK));
  pl.total_blocks = static_cast<long long>(pl.kblocks) * pl.num_tiles;
  if (mode == 0 && pl.grid > pl.total_blocks) pl.grid = static_cast<int>(pl.total_blocks);
  int stages = (kSmemBudget - tail_pad) / stage_bytes;
  if (stages > kMaxStages) stages = kMaxStages;
  if (stages < 1) stages = 1;      // cannot happen: one 128-byte box of the widest operands is 48 KB
  pl.stages = stages;
  pl.epi_off = static_cast<int>(round_up(static_cast<size_t>(stages) * stage_bytes + tail_pad, 1024));
  pl.smem_bytes = static_cast<size_t>(pl.epi_off) + kEpiBytes + 1024;
  // Few weight tiles (small N): instead of the stream-K split with its global atomics, a cluster of S CTAs per tile
  // splits K evenly and sums the partial tiles through distributed shared memory (mode 2).  Taken when the clusters
  // cover at least three quarters of the SMs, all of them are resident at once, and the partials fit the
  // pipeline buffers they are delivered into.
  pl.csplit = 1;
  if (mode == 0 && mode_env != 0 && pl.num_tiles > 0) {
    int S = grid / pl.num_tiles;
    if (S > 8) S = 8;
    if (S > pl.kblocks) S = pl.kblocks;
    for (; S >= 2; --S) {
      // S-1 incoming and S-1 outgoing slots of [passes][longest token range][128] sums live in the drained pipeline
      const int G8 = pl.Mp / 8, F = S < G8 ? S : G8;
      const size_t xfer = 2 * static_cast<size_t>(S - 1) * (base ? 1 : 2) * 8 * ((G8 + F - 1) / F) * kTileN * sizeof(int32_t);
      if (xfer <= static_cast<size_t>(pl.epi_off)) break;
    }
    if (S >= 2) {
      const bool covers = static_cast<long long>(pl.num_tiles) * S * 4 >= 3LL * grid;
      if ((covers || mode_env == 2) && max_resident_clusters(base, S, pl.smem_bytes) >= pl.num_tiles) {
        pl.mode = 2;
        pl.csplit = S;
        pl.grid = pl.num_tiles * S;
      }
    }
  }
  pl.tmem_cols = pow2_at_least(2 * pl.NB);
  size_t off = 0;
  pl.off_q = off;         off = round_up(off + (base ? static_cast<size_t>(N) * K * 2 : static_cast<size_t>(pl.NB) * K), 1024);
  pl.off_alpha = off;     off = round_up(off + 128 * sizeof(float), 256);
  pl.off_beta = off;      off = round_up(off + 128 * sizeof(float), 256);
  // one arrival counter per weight tile, then the two counters of the in-kernel decomposition
  pl.off_counters = off;  off = round_up(off + static_cast<size_t>(pl.num_tiles + 2) * sizeof(unsigned), 1024);
  // split-K meeting place: one [NB x 128] tile of sums per weight tile (used by the stream-K split only)
  pl.off_slots = off;     off = round_up(off + static_cast<size_t>(pl.num_tiles) * pl.NB * kTileN * sizeof(int32_t), 1024);
  pl.bytes = off;
  return pl;
}

static bool ensure_smem_attr() {
  static bool attr_done = false;
  if (!attr_done) {
    if (cudaFuncSetAttribute(gemm_w8a16_kernel<false>, cudaFuncAttributeMaxDynamicSharedMemorySize, 227 * 1024 - 2048) != cudaSuccess ||
        cudaFuncSetAttribute(gemm_w8a16_kernel<true>, cudaFuncAttributeMaxDynamicSharedMemorySize, 227 * 1024 - 2048) != cudaSuccess ||
        cudaFuncSetAttribute(gemm_w8a16_kernel<false, true>, cudaFuncAttributeMaxDynamicSharedMemorySize, 227 * 1024 - 2048) != cudaSuccess)
    {
      cudaGetLastError();
      return false;
    }
    attr_done = true;
  }
  return true;
}

static int max_resident_clusters(bool base, int S, size_t smem_bytes) {
  struct Entry { bool base; int S; size_t smem; int n; };
  static Entry cache[32];
  static int used = 0;
  for (int i = 0; i < used; ++i)
    if (cache[i].base == base && cache[i].S == S && cache[i].smem == smem_bytes) return cache[i].n;
  if (!ensure_smem_attr()) return 0;
  cudaLaunchConfig_t cfg = {};
  cfg.gridDim = dim3(static_cast<unsigned>(S) * 64);
  cfg.blockDim = dim3(kGemmThreads);
  cfg.dynamicSmemBytes = smem_bytes;
  cudaLaunchAttribute attr[1];
  attr[0].id = cudaLaunchAttributeClusterDimension;
  attr[0].val.clusterDim.x = static_cast<unsigned>(S);
  attr[0].val.clusterDim.y = 1;
  attr[0].val.clusterDim.z = 1;
  cfg.attrs = attr;
  cfg.numAttrs = 1;
  int n = 0;
  const cudaError_t e = base ? cudaOccupancyMaxActiveClusters(&n, gemm_w8a16_kernel<true>, &cfg)
                             : cudaOccupancyMaxActiveClusters(&n, gemm_w8a16_kernel<false>, &cfg);
  if (e != cudaSuccess) { cudaGetLastError(); n = 0; }
  if (used < 32) cache[used++] = Entry{base, S, smem_bytes, n};
  return n;
}

// The step MSD removes (Sec. 3.1, first equation): INT8 weights -> bf16(s_W * w), written back to memory.
__global__ void dequant_w8_to_bf16_kernel(const int8_t* __restrict__ w, const float* __restrict__ w_scale, int64_t N, int64_t K,
                                          __nv_bfloat16* __restrict__ out) {
  pdl_launch_dependents();
  const int64_t chunks_per_row = K >> 4;
  const int64_t total = N * chunks_per_row;
  for (int64_t i = static_cast<int64_t>(blockIdx.x) * blockDim.x + threadIdx.x; i < total;
       i += static_cast<int64_t>(gridDim.x) * blockDim.x) {
    const int64_t n = i / chunks_per_row;
    const float s = __ldg(w_scale + n);
    const uint4 v = __ldg(reinterpret_cast<const uint4*>(w) + i);
    const uint32_t wv[4] = {v.x, v.y, v.z, v.w};
    uint32_t o[8];
#pragma unroll
    for (int j = 0; j < 8; ++j) {
      const int b0 = static_cast<int8_t>((wv[j >> 1] >> (16 * (j & 1))) & 0xFF);
      const int b1 = static_cast<int8_t>((wv[j >> 1] >> (16 * (j & 1) + 8)) & 0xFF);
      const __nv_bfloat162 h = __floats2bfloat162_rn(s * static_cast<float>(b0), s * static_cast<float>(b1));
      o[j] = *reinterpret_cast<const uint32_t*>(&h);
    }
    uint4* dst = reinterpret_cast<uint4*>(out) + 2 * i;
    dst[0] = make_uint4(o[0], o[1], o[2], o[3]);
    dst[1] = make_uint4(o[4], o[5], o[6], o[7]);
  }
}

// Tensor map of a K-major byte matrix [rows, kbytes] for the GEMM's stages: with `t3` one 3-D box {128 B, box_rows, kw}
// (third dimension = the 128-byte K blocks of a row, stride 128 B) brings the kw chunks of a stage with one copy
// instruction; otherwise 2-D boxes of 128 B x box_rows.  t3 needs kbytes % 128 == 0 (a K block never straddles rows).
static bool encode_stage_map(CUtensorMap* out, const void* base, uint64_t kbytes, uint64_t rows, uint32_t box_rows, int kw, bool t3) {
  if (t3)
    return encode_tmap_3d(out, CU_TENSOR_MAP_DATA_TYPE_UINT8, base, kBlockK, rows, kbytes / kBlockK, kbytes, kBlockK, kBlockK, box_rows,
                          static_cast<uint32_t>(kw), CU_TENSOR_MAP_SWIZZLE_128B);
  return encode_tmap_2d(out, CU_TENSOR_MAP_DATA_TYPE_UINT8, base, kbytes, rows, kbytes, kBlockK, box_rows, CU_TENSOR_MAP_SWIZZLE_128B);
}

msd_status_t launch_dequant_w8_to_bf16(const int8_t* w, const float* w_scale, int64_t N, int64_t K, void* out_bf16, cudaStream_t s) {
  const int64_t total = N * (K >> 4);
  int64_t blocks = (total + 255) / 256;
  const int64_t cap = static_cast<int64_t>(sm_count()) * 16;
  if (blocks > cap) blocks = cap;
  dequant_w8_to_bf16_kernel<<<static_cast<unsigned>(blocks), 256, 0, s>>>(w, w_scale, N, K, static_cast<__nv_bfloat16*>(out_bf16));
  return cudaGetLastError() == cudaSuccess ? MSD_OK : MSD_ERR_CUDA;
}

constexpr int64_t kMaxExactK = 131072;

static msd_status_t check_w8_args(const void* x, const void* w, const void* ws, int64_t M, int64_t N, int64_t K,
                                  const void* y, int ytype, const void* workspace, int64_t max_m = 128) {
  if (M < 1 || M > max_m || N < 1 || K < 16 || K % 16 != 0 || N > (1 << 24) || K > (1 << 24)) return MSD_ERR_BAD_SHAPE;
  // the two sums of Alg. 1 are exact in INT32 only while 127 * 128 * K < 2^31
  if (K > kMaxExactK) return MSD_ERR_UNSUPPORTED;
  if (ytype != MSD_OUT_BF16 && ytype != MSD_OUT_FP32) return MSD_ERR_UNSUPPORTED;
  if (ytype == MSD_OUT_BF16 && N % 8 != 0) return MSD_ERR_BAD_SHAPE;
  if (!x || !w || !ws || !y || !workspace) return MSD_ERR_NULL_POINTER;
  if (!aligned(x, 16) || !aligned(w, 16) || !aligned(y, 16) || !aligned(ws, 4) || !aligned(workspace, 1024))
    return MSD_ERR_BAD_ALIGNMENT;
  return MSD_OK;
}

}  // namespace msd

extern "C" {

size_t msd_gemm_w8a16_workspace_bytes(int64_t M, int64_t N, int64_t K) {
  if (M < 1 || M > (1 << 24) || N < 1 || K < 16) return 0;
  if (M > 128) return msd::w8_prefill_workspace_bytes(M, N, K);
  return msd::plan_w8(M, N, K).bytes;
}

msd_status_t msd_gemm_w8a16(const void* x_bf16, const int8_t* w, const float* w_scale, int64_t M, int64_t N,
                            int64_t K, void* y, msd_out_t ytype, int32_t* acc_dbg, void* workspace,
                            size_t workspace_bytes, void* stream) {
  return msd_gemm_w8a16_ex(x_bf16, w, w_scale, M, N, K, y, ytype, acc_dbg, MSD_SCALING_DEFAULT, workspace, workspace_bytes, stream);
}

msd_status_t msd_gemm_w8a16_ex(const void* x_bf16, const int8_t* w, const float* w_scale, int64_t M, int64_t N,
                               int64_t K, void* y, msd_out_t ytype, int32_t* acc_dbg, msd_scaling_t scaling,
                               void* workspace, size_t workspace_bytes, void* stream) {
  using namespace msd;
  if (scaling != MSD_SCALING_DEFAULT && scaling != MSD_SCALING_FRACTIONAL) return MSD_ERR_UNSUPPORTED;
  msd_status_t st = check_w8_args(x_bf16, w, w_scale, M, N, K, y, ytype, workspace, 1 << 24);
  if (st != MSD_OK) return st;
  if (M > 128) {
    // many rows: tokens on the MMA M axis, both components against the same weight tile (gemm_w8a16_prefill.cu)
    if (ytype == MSD_OUT_FP32 && N % 4 != 0) return MSD_ERR_BAD_SHAPE;     // the output rows are written by TMA stores
    return w8_prefill_launch(x_bf16, w, w_scale, M, N, K, y, ytype, acc_dbg, scaling_c1(scaling), scaling_c2(scaling), workspace,
                             workspace_bytes, static_cast<cudaStream_t>(stream));
  }
  const GemmW8Plan pl = plan_w8(M, N, K);
  if (workspace_bytes < pl.bytes) return MSD_ERR_WORKSPACE_TOO_SMALL;
  unsigned* status = device_status_ptr();
  if (!status) return MSD_ERR_CUDA;
  cudaStream_t s = static_cast<cudaStream_t>(stream);
  uint8_t* ws = static_cast<uint8_t*>(workspace);
  int8_t* q = reinterpret_cast<int8_t*>(ws + pl.off_q);
  float* alpha = reinterpret_cast<float*>(ws + pl.off_alpha);
  float* beta = reinterpret_cast<float*>(ws + pl.off_beta);

  // a1-a3: the decomposition kernel writes the stacked operand: rows [0, M) hold Q1, rows [Mp, Mp+M) hold Q2; the padding
  // rows are never read back.  (Decomposing inside the GEMM kernel - by extra quantiser warps, or by its first CTAs
  // behind a counter - was built and measured slower at every M: the row maximum then waits behind the weight prefetch.)
  st = launch_decompose_int8(x_bf16, M, K, K, q, q + static_cast<size_t>(pl.Mp) * K, alpha, beta, scaling_c1(scaling),
                             scaling_c2(scaling), s);
  if (st != MSD_OK) return st;

  CUtensorMap tmap_w, tmap_w2, tmap_x;
  const uint32_t box2 = (pl.mode == 1 && pl.hmax > pl.gran) ? pl.hmax - pl.gran : pl.hmax;
  const bool t3 = K % kBlockK == 0;
  if (!encode_stage_map(&tmap_w, w, K, N, pl.hmax, pl.kw, t3) || !encode_stage_map(&tmap_w2, w, K, N, box2, pl.kw, t3) ||
      !encode_stage_map(&tmap_x, q, K, pl.NB, pl.NB, pl.kw, t3))
    return MSD_ERR_CUDA;

  GemmW8Params p;
  p.tma3d = t3 ? 1 : 0;
  p.M = static_cast<int>(M); p.Mp = pl.Mp; p.NB = pl.NB; p.N = static_cast<int>(N); p.K = static_cast<int>(K);
  p.kb_rot_step = 5;
  p.pre_stages = 64;
  p.mode = pl.mode; p.groups8 = pl.groups8; p.gran = pl.gran; p.hmax = pl.hmax; p.w_chunk_bytes = pl.w_chunk_bytes; p.kw = pl.kw; p.epi_off = pl.epi_off; p.csplit = pl.csplit;
  p.kblocks = pl.kblocks; p.num_tiles = pl.num_tiles; p.total_blocks = pl.total_blocks;
  p.num_stages = pl.stages; p.tmem_cols = pl.tmem_cols; p.ytype = ytype;
  p.w_scale = w_scale; p.alpha = alpha; p.beta = beta; p.y = y; p.acc_dbg = acc_dbg;
  p.accum = reinterpret_cast<int32_t*>(ws + pl.off_slots);
  p.counters = reinterpret_cast<unsigned*>(ws + pl.off_counters);
  p.status = status;
  p.trace = g_trace;

  if (!ensure_smem_attr()) return MSD_ERR_CUDA;
  GemmW8NoGroups no_groups;
  const bool pdl = option(OPT_NO_PDL) <= 0;
  if (launch_pdl_cluster(gemm_w8a16_kernel<false>, dim3(pl.grid), dim3(kGemmThreads), pl.smem_bytes, s, pdl,
                         static_cast<unsigned>(pl.csplit), tmap_w, tmap_w2, tmap_x, p, no_groups) != cudaSuccess)
    return MSD_ERR_CUDA;
  return MSD_OK;
}

size_t msd_gemm_dequant_bf16_workspace_bytes(int64_t M, int64_t N, int64_t K) {
  if (M < 1 || M > (1 << 24) || N < 1 || K < 16) return 0;
  if (M > 128) return msd::w8_prefill_base_workspace_bytes(M, N, K);
  return msd::plan_w8(M, N, K, true).bytes;
}

msd_status_t msd_gemm_dequant_bf16(const void* x_bf16, const int8_t* w, const float* w_scale, int64_t M, int64_t N,
                                   int64_t K, void* y, msd_out_t ytype, void* workspace, size_t workspace_bytes,
                                   void* stream) {
  using namespace msd;
  msd_status_t st = check_w8_args(x_bf16, w, w_scale, M, N, K, y, ytype, workspace, 1 << 24);
  if (st != MSD_OK) return st;
  if (M > 128) {
    if (K % 64 != 0) return MSD_ERR_BAD_SHAPE;          // a K stage of the many-row kernel is 64 BF16 elements
    if (ytype == MSD_OUT_FP32 && N % 4 != 0) return MSD_ERR_BAD_SHAPE;
    return w8_prefill_base_launch(x_bf16, w, w_scale, M, N, K, y, ytype, workspace, workspace_bytes, static_cast<cudaStream_t>(stream));
  }
  const GemmW8Plan pl = plan_w8(M, N, K, true);
  if (workspace_bytes < pl.bytes) return MSD_ERR_WORKSPACE_TOO_SMALL;
  unsigned* status = device_status_ptr();
  if (!status) return MSD_ERR_CUDA;
  cudaStream_t s = static_cast<cudaStream_t>(stream);
  uint8_t* ws = static_cast<uint8_t*>(workspace);
  __nv_bfloat16* wbf = reinterpret_cast<__nv_bfloat16*>(ws + pl.off_q);
  st = launch_dequant_w8_to_bf16(w, w_scale, N, K, wbf, s);
  if (st != MSD_OK) return st;
  CUtensorMap tmap_w, tmap_w2, tmap_x;
  const uint64_t kb = static_cast<uint64_t>(2 * K);
  const uint32_t box2 = (pl.mode == 1 && pl.hmax > pl.gran) ? pl.hmax - pl.gran : pl.hmax;
  const bool t3 = kb % kBlockK == 0;
  if (!encode_stage_map(&tmap_w, wbf, kb, N, pl.hmax, pl.kw, t3) || !encode_stage_map(&tmap_w2, wbf, kb, N, box2, pl.kw, t3) ||
      !encode_stage_map(&tmap_x, x_bf16, kb, M, pl.NB, pl.kw, t3))
    return MSD_ERR_CUDA;
  GemmW8Params p;
  p.tma3d = t3 ? 1 : 0;
  p.M = static_cast<int>(M); p.Mp = pl.Mp; p.NB = pl.NB; p.N = static_cast<int>(N); p.K = static_cast<int>(K);
  p.kb_rot_step = 0;
  p.pre_stages = 64;
  p.mode = pl.mode; p.groups8 = pl.groups8; p.gran = pl.gran; p.hmax = pl.hmax; p.w_chunk_bytes = pl.w_chunk_bytes; p.kw = pl.kw; p.epi_off = pl.epi_off; p.csplit = pl.csplit;
  p.kblocks = pl.kblocks; p.num_tiles = pl.num_tiles; p.total_blocks = pl.total_blocks;
  p.num_stages = pl.stages; p.tmem_cols = pl.tmem_cols; p.ytype = ytype;
  p.w_scale = w_scale; p.alpha = nullptr; p.beta = nullptr; p.y = y; p.acc_dbg = nullptr;
  p.accum = reinterpret_cast<int32_t*>(ws + pl.off_slots);
  p.counters = reinterpret_cast<unsigned*>(ws + pl.off_counters);
  p.status = status;
  p.trace = nullptr;
  if (!ensure_smem_attr()) return MSD_ERR_CUDA;
  GemmW8NoGroups no_groups;
  const bool pdl = option(OPT_NO_PDL) <= 0;
  if (launch_pdl_cluster(gemm_w8a16_kernel<true>, dim3(pl.grid), dim3(kGemmThreads), pl.smem_bytes, s, pdl,
                         static_cast<unsigned>(pl.csplit), tmap_w, tmap_w2, tmap_x, p, no_groups) != cudaSuccess)
    return MSD_ERR_CUDA;
  return MSD_OK;
}

// ---------------------------------------------------------------------------------------------------------------------
// Grouped W8A16 layer (MoE experts; Discussion, "Extension to MoE and Sparse Architectures"): x rows sorted by expert, group g = rows [off_g, off_g + m_g) against
// expert e_g's weight.  One decomposition launch over all rows, then stream-K launches of up to kMaxGroups non-empty
// groups each; empty groups cost nothing (their weights are never read).
struct GroupedPlan {
  msd::GemmW8Plan base;       // tile shapes for the largest group
  int64_t mt_pad;             // rows reserved per component in the stacked buffer
  size_t off_q, off_alpha, off_beta, off_counters, off_slots, bytes;
};

static GroupedPlan plan_grouped(int64_t M_total, int max_group, int E, int64_t N, int64_t K) {
  using namespace msd;
  GroupedPlan g;
  g.base = plan_w8(max_group < 1 ? 1 : max_group, N, K);
  g.mt_pad = static_cast<int64_t>(round_up(static_cast<size_t>(M_total), 8)) + 128;     // a box may start at the last row
  const int groups_per_launch = E < kMaxGroups ? E : kMaxGroups;
  const size_t tiles = static_cast<size_t>(groups_per_launch) * g.base.num_tiles;
  size_t off = 0;
  g.off_q = off;        off = round_up(off + 2 * static_cast<size_t>(g.mt_pad) * K, 1024);
  g.off_alpha = off;    off = round_up(off + static_cast<size_t>(M_total + 1) * sizeof(float), 256);
  g.off_beta = off;     off = round_up(off + static_cast<size_t>(M_total + 1) * sizeof(float), 256);
  g.off_counters = off; off = round_up(off + (tiles + 2) * sizeof(unsigned), 1024);
  g.off_slots = off;    off = round_up(off + tiles * g.base.NB * kTileN * sizeof(int32_t), 1024);
  g.bytes = off;
  return g;
}

size_t msd_grouped_gemm_w8a16_workspace_bytes(int64_t M_total, int32_t max_group_size, int32_t E, int64_t N, int64_t K) {
  if (M_total < 0 || max_group_size < 0 || max_group_size > 128 || E < 1 || N < 1 || K < 16) return 0;
  return plan_grouped(M_total, max_group_size, E, N, K).bytes;
}

msd_status_t msd_grouped_gemm_w8a16(const void* x_bf16, const int8_t* w, const float* w_scale, const int32_t* group_sizes_host,
                                    int32_t E, int64_t N, int64_t K, void* y, msd_out_t ytype, void* workspace,
                                    size_t workspace_bytes, void* stream) {
  using namespace msd;
  if (E < 1 || N < 1 || K < 16 || K % 16 != 0 || N > (1 << 24) || K > (1 << 24)) return MSD_ERR_BAD_SHAPE;
  if (K > kMaxExactK) return MSD_ERR_UNSUPPORTED;       // INT32 sums would no longer be exact
  if (!group_sizes_host) return MSD_ERR_NULL_POINTER;
  if (ytype != MSD_OUT_BF16 && ytype != MSD_OUT_FP32) return MSD_ERR_UNSUPPORTED;
  if (ytype == MSD_OUT_BF16 && N % 8 != 0) return MSD_ERR_BAD_SHAPE;
  if (static_cast<int64_t>(E) * N > 0x7FFFFFFF) return MSD_ERR_BAD_SHAPE;
  int64_t M_total = 0;
  int max_group = 0;
  for (int e = 0; e < E; ++e) {
    if (group_sizes_host[e] < 0 || group_sizes_host[e] > 128) return MSD_ERR_BAD_SHAPE;      // decode regime per expert
    M_total += group_sizes_host[e];
    if (group_sizes_host[e] > max_group) max_group = group_sizes_host[e];
  }
  if (M_total == 0) return MSD_OK;
  if (!x_bf16 || !w || !w_scale || !y || !workspace) return MSD_ERR_NULL_POINTER;
  if (!aligned(x_bf16, 16) || !aligned(w, 16) || !aligned(y, 16) || !aligned(workspace, 1024)) return MSD_ERR_BAD_ALIGNMENT;
  const GroupedPlan gp = plan_grouped(M_total, max_group, E, N, K);
  if (workspace_bytes < gp.bytes) return MSD_ERR_WORKSPACE_TOO_SMALL;
  unsigned* status = device_status_ptr();
  if (!status) return MSD_ERR_CUDA;
  cudaStream_t s = static_cast<cudaStream_t>(stream);
  uint8_t* ws = static_cast<uint8_t*>(workspace);
  int8_t* q = reinterpret_cast<int8_t*>(ws + gp.off_q);
  float* alpha = reinterpret_cast<float*>(ws + gp.off_alpha);
  float* beta = reinterpret_cast<float*>(ws + gp.off_beta);
  msd_status_t st = launch_decompose_int8(x_bf16, M_total, K, K, q, q + static_cast<size_t>(gp.mt_pad) * K, alpha, beta, 127.0f,
                                          254.0f, s);
  if (st != MSD_OK) return st;

  const GemmW8Plan& pl = gp.base;
  const int kw = pl.kw;
  const int kblocks = pl.kblocks;
  CUtensorMap tmap_w, tmap_x;
  const bool t3 = K % kBlockK == 0;        // the weight stages as 3-D boxes; the two component boxes of a group stay 2-D
  if (!encode_stage_map(&tmap_w, w, K, static_cast<uint64_t>(E) * N, kTileN, kw, t3) ||
      !encode_tmap_2d(&tmap_x, CU_TENSOR_MAP_DATA_TYPE_UINT8, q, K, 2 * static_cast<uint64_t>(gp.mt_pad), K, kBlockK, pl.Mp,
                      CU_TENSOR_MAP_SWIZZLE_128B))
    return MSD_ERR_CUDA;
  if (!ensure_smem_attr()) return MSD_ERR_CUDA;

  GemmW8Params p;
  p.M = pl.Mp; p.Mp = pl.Mp; p.NB = pl.NB; p.N = static_cast<int>(N); p.K = static_cast<int>(K);
  p.kb_rot_step = 0; p.pre_stages = 64;
  p.mode = 0; p.groups8 = 1; p.gran = 8; p.hmax = kTileN; p.w_chunk_bytes = kWStageBytes; p.kw = kw; p.csplit = 1;
  p.tma3d = t3 ? 1 : 0;
  p.kblocks = kblocks; p.num_stages = pl.stages; p.tmem_cols = pl.tmem_cols; p.ytype = ytype;
  // the planner laid the stages out for row bands when N is large; stream-K always stages full 128-row weight boxes
  {
    const int stage_bytes = kw * (kWStageBytes + pl.NB * kBlockK);
    int stages = kSmemBudget / stage_bytes;
    if (stages > kMaxStages) stages = kMaxStages;
    if (stages < 1) return MSD_ERR_UNSUPPORTED;
    p.num_stages = stages;
    p.epi_off = static_cast<int>(round_up(static_cast<size_t>(stages) * stage_bytes, 1024));
  }
  const size_t smem_bytes = static_cast<size_t>(p.epi_off) + kEpiBytes + 1024;
  p.w_scale = w_scale; p.alpha = alpha; p.beta = beta; p.y = y; p.acc_dbg = nullptr;
  p.accum = reinterpret_cast<int32_t*>(ws + gp.off_slots);
  p.counters = reinterpret_cast<unsigned*>(ws + gp.off_counters);
  p.status = status; p.trace = nullptr;

  const bool pdl = option(OPT_NO_PDL) <= 0;
  int e = 0;
  int64_t off = 0;
  while (e < E) {
    GemmW8Groups g;
    g.n = 0; g.tiles_per_group = pl.num_tiles; g.xq2_row0 = static_cast<int>(gp.mt_pad);
    while (e < E && g.n < kMaxGroups) {
      const int m = group_sizes_host[e];
      if (m > 0) {
        g.expert[g.n] = e; g.off[g.n] = static_cast<int>(off); g.m[g.n] = m;
        ++g.n;
      }
      off += m;
      ++e;
    }
    if (g.n == 0) break;
    p.num_tiles = g.n * pl.num_tiles;
    p.total_blocks = static_cast<long long>(p.num_tiles) * kblocks;
    int grid = sm_count();
    if (grid > p.total_blocks) grid = static_cast<int>(p.total_blocks);
    if (launch_pdl(gemm_w8a16_kernel<false, true>, dim3(grid), dim3(kGemmThreads), smem_bytes, s, pdl, tmap_w, tmap_w, tmap_x, p, g) !=
        cudaSuccess)
      return MSD_ERR_CUDA;
  }
  return MSD_OK;
}

// ---------------------------------------------------------------------------------------------------------------------
}  // extern "C"

// ---------------------------------------------------------------------------------------------------------------------
// Entry point for callers that cannot allocate device memory (see msd.h).  The scratch the GEMM needs lives in this
// file-scope device array, which every GPU that loads the library holds until the process exits.
// ---------------------------------------------------------------------------------------------------------------------
namespace msd {
constexpr int64_t kStaticMaxM = 16;
constexpr int64_t kStaticMaxN = 16384;
constexpr int64_t kStaticMaxK = 16384;
constexpr size_t kStaticScratchBytes = 3u << 20;      // covers the workspace of M<=16, N<=16384, K<=16384 (about 2.6 MB)
static __device__ __align__(256) unsigned char g_static_scratch[kStaticScratchBytes + 1024];

// Device address of the scratch array on the current device (resolved once per device); NULL on failure.
// In host code `g_static_scratch` is only a handle for the runtime, not an address a kernel could use.
static unsigned char* static_scratch_ptr() {
  static std::mutex mu;
  static unsigned char* cache[64] = {};
  int dev = 0;
  if (cudaGetDevice(&dev) != cudaSuccess || dev < 0 || dev >= 64) return nullptr;
  std::lock_guard<std::mutex> lock(mu);
  if (!cache[dev]) {
    unsigned char* ptr = nullptr;
    if (cudaGetSymbolAddress(reinterpret_cast<void**>(&ptr), g_static_scratch) != cudaSuccess || !ptr) return nullptr;
    cache[dev] = ptr;
  }
  return cache[dev];
}
}  // namespace msd

extern "C" {

msd_status_t msd_gemm_w8a16_noalloc(const void* x_bf16, const int8_t* w, const float* w_scale, int64_t M, int64_t N,
                                    int64_t K, void* y, msd_out_t ytype, void* stream) {
  using namespace msd;
  if (M < 1 || N < 1 || K < 16) return MSD_ERR_BAD_SHAPE;
  if (M > kStaticMaxM || N > kStaticMaxN || K > kStaticMaxK) return MSD_ERR_UNSUPPORTED;   // beyond the built-in scratch
  unsigned char* raw = static_scratch_ptr();
  if (!raw) return MSD_ERR_CUDA;
  unsigned char* ws = reinterpret_cast<unsigned char*>((reinterpret_cast<uintptr_t>(raw) + 1023) & ~static_cast<uintptr_t>(1023));
  const size_t avail = kStaticScratchBytes + 1024 - static_cast<size_t>(ws - raw);
  const GemmW8Plan pl = plan_w8(M, N, K);
  if (pl.bytes > avail) return MSD_ERR_UNSUPPORTED;
  // every host-detectable problem is reported before anything is enqueued (the scratch stands in for the workspace)
  const msd_status_t st = check_w8_args(x_bf16, w, w_scale, M, N, K, y, ytype, ws);
  if (st != MSD_OK) return st;
  // The array keeps whatever the previous call left.  The arrival counters (and, for the stream-K split only, the
  // meeting place of the partial sums) must start at zero; a completed call leaves them so, but a call that gave up on
  // a wait may not have, so they are cleared every time.  The other work splits never touch the meeting place.
  const size_t clear_bytes = (pl.mode == 0 ? pl.bytes : pl.off_slots) - pl.off_counters;
  if (cudaMemsetAsync(ws + pl.off_counters, 0, clear_bytes, static_cast<cudaStream_t>(stream)) != cudaSuccess)
    return MSD_ERR_CUDA;
  return msd_gemm_w8a16(x_bf16, w, w_scale, M, N, K, y, ytype, nullptr, ws, avail, stream);
}

void msd_debug_set_trace(void* device_buffer) { msd::g_trace = static_cast<long long*>(device_buffer); }

size_t msd_gemm_w8a16_host_workspace_bytes(int64_t M, int64_t N, int64_t K) {
  if (M < 1 || M > 128 || N < 1 || K < 16) return 0;
  return msd::plan_w8(M, N, K).bytes + msd::round_up(static_cast<size_t>(M) * K * 2, 1024) +
         msd::round_up(static_cast<size_t>(M) * N * 4, 1024);
}

msd_status_t msd_gemm_w8a16_host(const void* x_bf16_host, const int8_t* w, const float* w_scale, int64_t M,
                                 int64_t N, int64_t K, void* y_host, msd_out_t ytype, void* workspace,
                                 size_t workspace_bytes, void* stream) {
  using namespace msd;
  if (M < 1 || M > 128 || N < 1 || K < 16 || K % 16 != 0) return MSD_ERR_BAD_SHAPE;
  if (!x_bf16_host || !y_host || !workspace) return MSD_ERR_NULL_POINTER;
  if (!aligned(workspace, 1024)) return MSD_ERR_BAD_ALIGNMENT;
  if (workspace_bytes < msd_gemm_w8a16_host_workspace_bytes(M, N, K)) return MSD_ERR_WORKSPACE_TOO_SMALL;
  const size_t inner = plan_w8(M, N, K).bytes;
  uint8_t* ws = static_cast<uint8_t*>(workspace);
  uint8_t* x_dev = ws + inner;
  uint8_t* y_dev = x_dev + round_up(static_cast<size_t>(M) * K * 2, 1024);
  cudaStream_t s = static_cast<cudaStream_t>(stream);
  const size_t ybytes = static_cast<size_t>(M) * N * (ytype == MSD_OUT_BF16 ? 2 : 4);
  if (cudaMemcpyAsync(x_dev, x_bf16_host, static_cast<size_t>(M) * K * 2, cudaMemcpyHostToDevice, s) != cudaSuccess)
    return MSD_ERR_CUDA;
  msd_status_t st = msd_gemm_w8a16(x_dev, w, w_scale, M, N, K, y_dev, ytype, nullptr, workspace, inner, stream);
  if (st != MSD_OK) return st;
  if (cudaMemcpyAsync(y_host, y_dev, ybytes, cudaMemcpyDeviceToHost, s) != cudaSuccess) return MSD_ERR_CUDA;
  return MSD_OK;
}

}  // extern "C"

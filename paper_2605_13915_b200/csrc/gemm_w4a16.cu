// W4A16 MSD linear layer (Sec. 3.2.1, Alg. 2; Tab. mxfp4-compute): both MXFP4 components of the activation are
// multiplied against the MXFP4 weight by block-scaled FP4 MMAs (tcgen05.mma kind::mxf4, E8M0 scale per 32 K) that
// accumulate into the SAME FP32 tile in TMEM, so the "one add" of the two passes costs nothing and each weight tile
// is read once for both passes.
//
// Tile: 128 activation rows x 224 (default) or 256 weight rows, K walked in stages of 256 elements (128 packed bytes =
// one 128-byte swizzle row).  Per stage TMA brings the A1, A2 (up to 128 x 128 B) and B (224/256 x 128 B) tiles and
// bulk copies bring the scale blocks (512-byte blocks of 128 rows x 4 scales); four warps move the scales from shared
// memory into TMEM (tcgen05.st), one thread issues 4 K-steps x 2 passes of MMAs.  Persistent CTAs walk the work items
// (token tile, weight tile, K split) in an order chosen by which operand stays in L2.
//
// Warps: 0 = operand producer, 1 = MMA issuer + TMEM owner, 2..5 = epilogue (TMEM -> BF16/FP32 -> swizzled staging
// buffer -> TMA store), 6..9 = scale warps, 10 = scale producer.  The same kernel serves the grouped
// (mixture-of-experts) entry point: group g is token tile g.  gemm_w4a16_pair_kernel is the opt-in cta_group::2 variant.
#include <cuda_bf16.h>

#include <cstdlib>

#include "host_common.h"
#include "sm100.cuh"

namespace msd {

constexpr int kW4TileM = 128;
constexpr int kW4BlockK = 256;                                  // elements per stage (128 packed bytes)
constexpr int kW4ThreadsSf = 352;      // producer, MMA, four epilogue warps, four warps that write the scales into TMEM, scale producer
constexpr int kW4PairThreads = 352;    // the CTA-pair kernel has the same warp roles
constexpr int kW4ABytes = kW4TileM * 128;                       // 16 KB
constexpr int kW4SfBytes = 1024 + 1024 + 2048;                  // SFA1, SFA2 (2 k-groups each), SFB (2 row tiles x 2 k-groups)
constexpr int kW4Stages = 3;
constexpr int kW4StoreBytes = 2048;                              // one epilogue chunk: 32 rows x 64 bytes
constexpr int kW4TmemCols = 512;

struct GemmW4Params {
  int M, N, K;
  int m_tiles, n_tiles, kstages;
  int sf_kgroups;               // 128-element K groups per row of the blocked scale arrays (even)
  const uint8_t* sfa1;
  const uint8_t* sfa2;
  const uint8_t* sfb;
  void* y;
  int ytype;
  int ksplit, kper;             // K splits per output tile and K stages per split (1, kstages: no split)
  int part_rows;                // ksplit > 1: rows per split of the partial-sum buffer the tiles are written to
  int nstages;                  // pipeline stages that fit with a_rows rows per component tile
  int a_rows;                   // rows of a token tile that are loaded (the box of the component tensor maps): 128, or
                                // fewer when no group of a grouped launch is longer; the MMA reads stale rows beyond them,
                                // whose results are never stored
  int n_fastest;                // tile index -> (token tile, weight tile): weight tile fastest (1) or token tile fastest (0)
  unsigned* status;
};

// Mixture-of-experts launch: token tile g holds the rows of group g (at most 128), which multiply the weights of expert
// expert[g]; the rows of the result go to y rows off[g] ...
struct GemmW4Groups {
  int n;
  int expert[kMaxRowGroups], off[kMaxRowGroups + 1];
};
struct GemmW4NoGroups {};
template <bool kGrouped> struct W4GroupArg { using type = GemmW4NoGroups; };
template <> struct W4GroupArg<true> { using type = GemmW4Groups; };

// Sum of the K-split partial tiles, split 0 first (fixed order: the same inputs give the same bits), rounded once.
__global__ void __launch_bounds__(256)
ksplit_reduce_kernel(const float* __restrict__ part, int ksplit, int64_t part_stride, int64_t M, int64_t N, void* __restrict__ y,
                        int ytype) {
  pdl_wait_primary();
  const int64_t total = M * N / 4;                     // N is a multiple of 8
  for (int64_t i = static_cast<int64_t>(blockIdx.x) * blockDim.x + threadIdx.x; i < total; i += static_cast<int64_t>(gridDim.x) * blockDim.x) {
    float4 acc = __ldg(reinterpret_cast<const float4*>(part) + i);
    for (int s = 1; s < ksplit; ++s) {
      const float4 v = __ldg(reinterpret_cast<const float4*>(part + s * part_stride) + i);
      acc.x += v.x; acc.y += v.y; acc.z += v.z; acc.w += v.w;
    }
    if (ytype == MSD_OUT_BF16) {
      const __nv_bfloat162 h0 = __floats2bfloat162_rn(acc.x, acc.y), h1 = __floats2bfloat162_rn(acc.z, acc.w);
      reinterpret_cast<uint2*>(y)[i] = make_uint2(*reinterpret_cast<const uint32_t*>(&h0), *reinterpret_cast<const uint32_t*>(&h1));
    } else {
      reinterpret_cast<float4*>(y)[i] = acc;
    }
  }
}

msd_status_t launch_ksplit_reduce(const float* part, int ksplit, int64_t part_stride, int64_t M, int64_t N, void* y, int ytype,
                                  cudaStream_t s, bool pdl) {
  const int64_t quads = M * N / 4;
  int64_t blocks = (quads + 255) / 256;
  if (blocks > 4LL * sm_count()) blocks = 4LL * sm_count();
  if (blocks < 1) blocks = 1;
  return launch_pdl(ksplit_reduce_kernel, dim3(static_cast<unsigned>(blocks)), dim3(256), 0, s, pdl, part, ksplit, part_stride, M, N, y, ytype) == cudaSuccess
             ? MSD_OK : MSD_ERR_CUDA;
}


// kTN = weight rows per tile: 256 (one accumulator) or 224 (two accumulators of 224 columns + the two sets of scale
// columns fill the 512 TMEM columns exactly, so the epilogue of a tile overlaps the MMAs of the next).
template <int kTN, bool kGrouped = false>
__global__ void __launch_bounds__(kW4ThreadsSf, 1)
gemm_w4a16_kernel(const __grid_constant__ CUtensorMap tmap_a1, const __grid_constant__ CUtensorMap tmap_a2,
                  const __grid_constant__ CUtensorMap tmap_b, const __grid_constant__ CUtensorMap tmap_y,
                  const GemmW4Params p, const typename W4GroupArg<kGrouped>::type grp) {
  constexpr int kBBytes = kTN * 128;
  // Shared-memory stage: the two component tiles, the weight tile, the scale blocks.  Launches with few rows (one
  // token tile of M < 128 rows, short groups) load only a_rows <= 128 rows per component (whole 1 KB swizzle atoms), pack the stage accordingly and use the room for more
  // stages: their weight tiles come from HBM, not L2, and a freed stage takes twice as long to fill.  The MMA still
  // reads 128 rows from where a component tile starts: whatever follows it there, results never stored.
  constexpr int kMaxStages = 8;
  const int a_bytes = p.a_rows * 128;
  const int kStageBytes = 2 * a_bytes + kBBytes + kW4SfBytes;
  const int nstages = p.nstages;
  constexpr int kAcc = (2 * kTN + 64 <= kW4TmemCols) ? 2 : 1;       // accumulators that fit beside 2 x 32 scale columns
  constexpr int kSfCol = kAcc * kTN;
  extern __shared__ uint8_t smem_dyn[];
  __shared__ __align__(8) uint64_t full_bar[kMaxStages], empty_bar[kMaxStages], tfull_bar[2], tempty_bar[2];
  // the two sets of scale columns in TMEM: written by warps 6..9 (sf_ready), read by the MMAs of a stage (sf_free)
  __shared__ __align__(8) uint64_t sf_ready[2], sf_free[2];
  __shared__ uint32_t tmem_base_slot;
  __shared__ int abort_flag;

  const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
  uint8_t* smem = reinterpret_cast<uint8_t*>((reinterpret_cast<uintptr_t>(smem_dyn) + 1023) & ~static_cast<uintptr_t>(1023));

  if (threadIdx.x == 0) {
    for (int s = 0; s < nstages; ++s) { mbar_init(&full_bar[s], 1); mbar_init(&empty_bar[s], 1); }
    for (int a = 0; a < 2; ++a) { mbar_init(&tfull_bar[a], 1); mbar_init(&tempty_bar[a], 4); }
    for (int a = 0; a < 2; ++a) { mbar_init(&sf_ready[a], 4); mbar_init(&sf_free[a], 1); }
    abort_flag = 0;
    mbar_init_fence();
    tma_prefetch_desc(&tmap_a1);
    tma_prefetch_desc(&tmap_a2);
    tma_prefetch_desc(&tmap_b);
  }
  if (warp == 1) tmem_alloc(&tmem_base_slot, kW4TmemCols);
  tc_fence_before();
  __syncthreads();
  tc_fence_after();
  const uint32_t tmem_base = tmem_base_slot;
  volatile int* abort = &abort_flag;
  // Work items: (token tile, weight tile, K split).  With ksplit > 1 (few tiles, long K: decode shapes) every item
  // covers kper K stages and its FP32 partial tile goes to rows [split * part_rows, ...) of a partial-sum buffer that a
  // second kernel adds up in a fixed order.
  const int total_tiles = p.m_tiles * p.n_tiles * p.ksplit;

  if (warp == 0 || warp == 10) {
    // Two producer threads: issuing a bulk copy costs its thread 50-100 ns, and the time a freed stage waits for its
    // refill to be requested is part of the pipeline's round trip.  Warp 0 requests the operand tiles, warp 10 the
    // scale blocks (their bytes may be counted before warp 0's arrival announces them: the phase cannot end without it).
    if (lane == 0) {
      // components and blocked scales come from the kernel launched just before
      bool ok = true;
      pdl_wait_primary();
      int stage = 0; uint32_t phase = 0;
      for (int tile = blockIdx.x; tile < total_tiles && ok; tile += gridDim.x) {
        const int split = tile % p.ksplit, tile_mn = tile / p.ksplit;
        const int mt = p.n_fastest ? tile_mn / p.n_tiles : tile_mn % p.m_tiles, nt = p.n_fastest ? tile_mn % p.n_tiles : tile_mn / p.m_tiles;
        const int ks0 = split * p.kper, ks1 = ks0 + p.kper < p.kstages ? ks0 + p.kper : p.kstages;
        for (int ks = ks0; ks < ks1; ++ks) {
          ok = wait_bounded(&empty_bar[stage], phase ^ 1, abort, p.status);
          if (!ok) break;
          uint8_t* dst = smem + stage * kStageBytes;
          if (warp == 0) {
            mbar_arrive_expect_tx(&full_bar[stage], kStageBytes);
            tma_load_2d(dst, &tmap_a1, ks * 128, mt * kW4TileM, &full_bar[stage]);
            tma_load_2d(dst + a_bytes, &tmap_a2, ks * 128, mt * kW4TileM, &full_bar[stage]);
            int b_row = nt * kTN;
            if constexpr (kGrouped) b_row += grp.expert[mt] * p.N;          // the weights of the group's expert
            tma_load_2d(dst + 2 * a_bytes, &tmap_b, ks * 128, b_row, &full_bar[stage]);
          } else {
            uint8_t* sf = dst + 2 * a_bytes + kBBytes;
            const size_t a_off = (static_cast<size_t>(mt) * p.sf_kgroups + 2 * ks) * 512;
            bulk_load(sf, p.sfa1 + a_off, 1024, &full_bar[stage]);
            bulk_load(sf + 1024, p.sfa2 + a_off, 1024, &full_bar[stage]);
            size_t sfb_blk = static_cast<size_t>(2 * nt);
            if constexpr (kGrouped) sfb_blk += static_cast<size_t>(grp.expert[mt]) * 2 * p.n_tiles;
            bulk_load(sf + 2048, p.sfb + (sfb_blk * p.sf_kgroups + 2 * ks) * 512, 1024, &full_bar[stage]);
            bulk_load(sf + 3072, p.sfb + ((sfb_blk + 1) * p.sf_kgroups + 2 * ks) * 512, 1024, &full_bar[stage]);
          }
          if (++stage == nstages) { stage = 0; phase ^= 1; }
        }
      }
    }
  } else if (warp == 1) {
    if (lane == 0) {
      int stage = 0; uint32_t phase = 0;
      int it = 0;
      bool ok = true;
      uint32_t sfpar = 0;
      int nstage = 0;                                                   // stages issued so far (all tiles)
      const uint64_t op_desc = smem_desc(0, 16, 1024, kSwizzle128B);    // 128-byte-swizzled K-major operand tile
      const uint32_t idesc_lo = idesc_block_scaled(/*E2M1*/ 1, 1, kW4TileM, kTN, 0, 0);
      const uint32_t idesc_hi = idesc_block_scaled(/*E2M1*/ 1, 1, kW4TileM, kTN, 2, 2);
      for (int tile = blockIdx.x; tile < total_tiles && ok; tile += gridDim.x, ++it) {
        const int acc = (kAcc == 2) ? (it & 1) : 0;
        const uint32_t tphase = (kAcc == 2) ? ((it >> 1) & 1) : (it & 1);
        const uint32_t d_tmem = tmem_base + acc * kTN;
        ok = wait_bounded(&tempty_bar[acc], tphase ^ 1, abort, p.status);      // epilogue has drained this accumulator
        if (!ok) break;
        tc_fence_after();
        const int ks0 = (tile % p.ksplit) * p.kper, ks1 = ks0 + p.kper < p.kstages ? ks0 + p.kper : p.kstages;
        for (int ks = ks0; ks < ks1; ++ks) {
          ok = wait_bounded(&full_bar[stage], phase, abort, p.status);
          if (!ok) break;
          tc_fence_after();
          // Descriptors differ from the templates only in the 16-byte-granular address field (bits 0-13; shared
          // memory is far below its range), so every operand costs one 64-bit add: this single thread's instruction
          // count per stage, not the tensor pipe, was what paced the kernel.
          const uint64_t enc = static_cast<uint64_t>(smem_u32(smem + stage * kStageBytes) >> 4);
          const uint64_t a1d = op_desc + enc, a2d = a1d + (a_bytes >> 4), bd = a1d + (2 * a_bytes >> 4);
          const uint32_t sfa1_t = tmem_base + kSfCol + 32 * sfpar;     // 2 k-groups x 4 columns; the two sets alternate
          const uint32_t sfa2_t = sfa1_t + 8;
          const uint32_t sfb_t = sfa1_t + 16;                            // 2 k-groups x 8 columns (256 weight rows)
          // the scale columns of this stage were written by warps 6..9 (tcgen05.cp copies issued by this thread run in
          // order with the MMAs in the tensor pipe and cost a sixth of its time)
          ok = wait_bounded(&sf_ready[sfpar], (nstage >> 1) & 1, abort, p.status);
          if (!ok) break;
          tc_fence_after();
#pragma unroll
          for (int kk = 0; kk < 4; ++kk) {                    // 64 elements (32 bytes) per MMA
            const int g = kk >> 1;
            const uint32_t idesc = (kk & 1) ? idesc_hi : idesc_lo;   // which pair of scale bytes of the 4-scale column
            mma_mxf4(d_tmem, a1d + 2 * kk, bd + 2 * kk, idesc, sfa1_t + 4 * g, sfb_t + 8 * g, (ks > ks0 || kk > 0) ? 1u : 0u);
            mma_mxf4(d_tmem, a2d + 2 * kk, bd + 2 * kk, idesc, sfa2_t + 4 * g, sfb_t + 8 * g, 1u);
          }
          tc_commit(&sf_free[sfpar]);                // this set of scale columns may be rewritten once these MMAs are done
          sfpar ^= 1;
          ++nstage;
          tc_commit(&empty_bar[stage]);
          if (++stage == nstages) { stage = 0; phase ^= 1; }
        }
        if (!ok) break;
        tc_commit(&tfull_bar[acc]);
      }
    }
  } else if (warp >= 6) {      // (warp 10 went the producers' way above)
    // Scale warps.  A 512-byte scale block holds, for 128 rows and one 128-element K group, 32 rows of 16 bytes: row l
    // carries the four scales of rows l, l+32, l+64, l+96, and every 32-lane quadrant of TMEM wants the same four
    // 32-bit columns.  Each warp reads the stage's eight blocks (one 16-byte row per lane and block) and stores them as
    // 32 columns of its own quadrant.
    const int quad = warp & 3;
    int stage = 0; uint32_t phase = 0;
    int n = 0;
    bool ok = true;
    for (int tile = blockIdx.x; tile < total_tiles && ok; tile += gridDim.x) {
      const int ks0 = (tile % p.ksplit) * p.kper, ks1 = ks0 + p.kper < p.kstages ? ks0 + p.kper : p.kstages;
      for (int ks = ks0; ks < ks1; ++ks, ++n) {
        const int set = n & 1;
        ok = wait_bounded(&full_bar[stage], phase, abort, p.status);
        if (!ok) break;
        if (n >= 2) {                        // the MMAs that read this set two stages ago are done
          ok = wait_bounded(&sf_free[set], ((n >> 1) - 1) & 1, abort, p.status);
          if (!ok) break;
          tc_fence_after();
        }
        const uint4* sf = reinterpret_cast<const uint4*>(smem + stage * kStageBytes + 2 * a_bytes + kBBytes) + lane;
        uint32_t v[32];
        // column order of a set: sfa1 (g0, g1), sfa2 (g0, g1), then per K group the two halves of the weight tile
        constexpr int kBlk[8] = {0, 1, 2, 3, 4, 6, 5, 7};
#pragma unroll
        for (int j = 0; j < 8; ++j) {
          const uint4 q = sf[kBlk[j] * 32];
          v[4 * j] = q.x; v[4 * j + 1] = q.y; v[4 * j + 2] = q.z; v[4 * j + 3] = q.w;
        }
        tmem_st32(tmem_base + (static_cast<uint32_t>(quad * 32) << 16) + kSfCol + 32 * set, v);
        tmem_st_wait();
        tc_fence_before();
        __syncwarp();
        if (lane == 0) mbar_arrive(&sf_ready[set]);
        if (++stage == nstages) { stage = 0; phase ^= 1; }
      }
    }
  } else {
    // Epilogue: TMEM -> registers -> (BF16) -> this warp's staging buffer in shared memory -> TMA store.  A chunk is
    // 64 bytes of every row of the warp's 32 rows (32 BF16 or 16 FP32 columns), laid out with the 64-byte swizzle of
    // the output tensor map so that the 16-byte stores of the 32 lanes spread over all banks; two buffers per warp,
    // the store of one chunk in flight while the next is converted.  Rows past M and columns past N are clipped by
    // the store itself.
    const int quad = warp & 3;
    uint8_t* stage_buf = smem + nstages * kStageBytes + quad * (2 * kW4StoreBytes);
    const int ccols = (p.ytype == MSD_OUT_BF16) ? 32 : 16;
    const uint32_t swz = static_cast<uint32_t>((lane >> 1) & 3);
    int it = 0, buf = 0;
    bool ok = true;
    for (int tile = blockIdx.x; tile < total_tiles && ok; tile += gridDim.x, ++it) {
      const int split = tile % p.ksplit, tile_mn = tile / p.ksplit;
      const int mt = p.n_fastest ? tile_mn / p.n_tiles : tile_mn % p.m_tiles, nt = p.n_fastest ? tile_mn % p.n_tiles : tile_mn / p.m_tiles;
      const int acc = (kAcc == 2) ? (it & 1) : 0;
      const uint32_t tphase = (kAcc == 2) ? ((it >> 1) & 1) : (it & 1);
      ok = wait_bounded(&tfull_bar[acc], tphase, abort, p.status);
      if (!ok) break;
      tc_fence_after();
      int row0 = mt * kW4TileM + quad * 32;              // first output row of this warp
      int rows_end = p.M;                                // output rows at or past it belong to nobody (or somebody else)
      if constexpr (kGrouped) {
        row0 = grp.off[mt] + quad * 32;
        rows_end = grp.off[mt + 1];
      }
      const uint32_t trow = tmem_base + (static_cast<uint32_t>(quad * 32) << 16) + acc * kTN;
      // columns of this tile inside the matrix (a warp whose rows are all past M has nothing to store); chunks
      // beyond them are skipped altogether, so every pass through the loop commits exactly one store group
      const int cols_here = p.N - nt * kTN < kTN ? p.N - nt * kTN : kTN;
      const int cend = row0 < rows_end ? cols_here : 0;
      if (cend == 0) {
        tc_fence_before();
        __syncwarp();
        if (lane == 0) mbar_arrive(&tempty_bar[acc]);
      }
      for (int c0 = 0; c0 < cend; c0 += ccols, buf ^= 1) {
        uint32_t o[16];
        if (p.ytype == MSD_OUT_BF16) {
          uint32_t v[32];
          tmem_ld32(trow + c0, v);
          tmem_ld_wait();
#pragma unroll
          for (int j = 0; j < 16; ++j) {
            const __nv_bfloat162 h = __floats2bfloat162_rn(__uint_as_float(v[2 * j]), __uint_as_float(v[2 * j + 1]));
            o[j] = *reinterpret_cast<const uint32_t*>(&h);
          }
        } else {
          tmem_ld16(trow + c0, o);
          tmem_ld_wait();
        }
        if (c0 + ccols >= cend) {                   // all that is needed of this accumulator is in registers: the MMAs may have it back
          tc_fence_before();
          __syncwarp();
          if (lane == 0) mbar_arrive(&tempty_bar[acc]);
        }
        uint8_t* sb = stage_buf + buf * kW4StoreBytes;
        // the store that read this buffer two chunks ago is done with it (grouped launches may skip a commit when a
        // group ends inside the warp's rows, so there all earlier stores are waited for)
        if (lane == 0) { if constexpr (kGrouped) bulk_wait_group_read<0>(); else bulk_wait_group_read<1>(); }
        __syncwarp();
        uint8_t* srow = sb + lane * 64;
#pragma unroll
        for (int j = 0; j < 4; ++j)
          *reinterpret_cast<uint4*>(srow + ((static_cast<uint32_t>(j) ^ swz) << 4)) = make_uint4(o[4 * j], o[4 * j + 1], o[4 * j + 2], o[4 * j + 3]);
        fence_proxy_async_smem();
        __syncwarp();
        if (!kGrouped || row0 + 32 <= rows_end) {
          if (lane == 0) {
            tma_store_2d(&tmap_y, nt * kTN + c0, row0 + split * p.part_rows, sb);
            bulk_commit_group();
          }
        } else {
          // the group ends inside this warp's 32 rows: the rows below belong to the next group, so the box store
          // is replaced by 16-byte stores of the group's own rows (lane -> row lane / 4 + 8 i, 16-byte piece lane % 4)
          const int esize = (p.ytype == MSD_OUT_BF16) ? 2 : 4;
          const int col = nt * kTN + c0, piece = lane & 3;
          if ((col + (piece + 1) * (16 / esize)) <= p.N) {
#pragma unroll
            for (int i = 0; i < 4; ++i) {
              const int r = (lane >> 2) + 8 * i;
              if (row0 + r < rows_end) {
                const uint4 v = *reinterpret_cast<const uint4*>(sb + r * 64 + ((static_cast<uint32_t>(piece) ^ static_cast<uint32_t>((r >> 1) & 3)) << 4));
                *reinterpret_cast<uint4*>(static_cast<uint8_t*>(p.y) + (static_cast<size_t>(row0 + r) * p.N + col) * esize + piece * 16) = v;
              }
            }
          }
          __syncwarp();
        }
      }
    }
    if (lane == 0) bulk_wait_group<0>();            // every store has been written before the CTA goes away
  }

  tc_fence_before();
  __syncthreads();
  if (warp == 1) {
    tc_fence_after();
    tmem_dealloc(tmem_base, kW4TmemCols);
  }
}

// ---------------------------------------------------------------------------------------------------------------------
// CTA-pair kernel: two CTAs of a cluster share one 256 x kTN tile.  Each CTA loads its own 128 activation rows (both
// components) and HALF of the weight tile; one tcgen05.mma.cta_group::2 per K step, issued by the even CTA, multiplies
// all 256 rows against all kTN weight rows, each CTA's accumulator (its 128 rows x kTN columns) staying in its own
// TMEM.  Why: the single-CTA kernel is bound by the round trip of its shared-memory pipeline (a freed stage is refilled
// from L2 about 1.9 us later; three 64 KB stages in flight feed 80 GB/s per SM where the tensor pipe wants 116).  A
// pair needs 46 KB of operands for the same tensor time and holds four stages.
//
// Barriers.  Operand tiles of both CTAs complete on the LEADER's full_bar; the scale blocks complete on each CTA's own
// sf_full (its scale warps read them); the scale warps of both CTAs arrive on the leader's sf_ready (8 arrivals); the
// leader's commits (empty_bar, sf_free, tfull_bar) are multicast to both CTAs; both epilogues arrive on the leader's
// tempty_bar.
constexpr int kW4PairStages = 4;

template <int kTN>
__global__ void __launch_bounds__(kW4PairThreads, 1)
gemm_w4a16_pair_kernel(const __grid_constant__ CUtensorMap tmap_a1, const __grid_constant__ CUtensorMap tmap_a2,
                       const __grid_constant__ CUtensorMap tmap_bh, const __grid_constant__ CUtensorMap tmap_y,
                       const GemmW4Params p) {
  constexpr int kBHalfBytes = (kTN / 2) * 128;
  constexpr int kOpBytes = 2 * kW4ABytes + kBHalfBytes;             // operand bytes per CTA and stage
  constexpr int kStageBytes = kOpBytes + kW4SfBytes;
  constexpr int kAcc = (2 * kTN + 64 <= kW4TmemCols) ? 2 : 1;
  constexpr int kSfCol = kAcc * kTN;
  extern __shared__ uint8_t smem_dyn[];
  __shared__ __align__(8) uint64_t full_bar[kW4PairStages], empty_bar[kW4PairStages], sf_full[kW4PairStages];
  __shared__ __align__(8) uint64_t tfull_bar[2], tempty_bar[2], sf_ready[2], sf_free[2];
  __shared__ uint32_t tmem_base_slot;
  __shared__ int abort_flag;

  const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
  const uint32_t rank = cluster_ctarank();          // 0 = leader of the pair
  uint8_t* smem = reinterpret_cast<uint8_t*>((reinterpret_cast<uintptr_t>(smem_dyn) + 1023) & ~static_cast<uintptr_t>(1023));

  if (threadIdx.x == 0) {
    for (int s = 0; s < kW4PairStages; ++s) { mbar_init(&full_bar[s], 1); mbar_init(&empty_bar[s], 1); mbar_init(&sf_full[s], 1); }
    for (int a = 0; a < 2; ++a) {
      mbar_init(&tfull_bar[a], 1);
      mbar_init(&tempty_bar[a], 8);     // four epilogue warps in each CTA of the pair (used in the leader only)
      mbar_init(&sf_ready[a], 8);       // four scale warps in each CTA (used in the leader only)
      mbar_init(&sf_free[a], 1);
    }
    abort_flag = 0;
    mbar_init_fence();
    tma_prefetch_desc(&tmap_a1);
    tma_prefetch_desc(&tmap_a2);
    tma_prefetch_desc(&tmap_bh);
  }
  if (warp == 1) tmem_alloc_pair(&tmem_base_slot, kW4TmemCols);
  tc_fence_before();
  cluster_arrive_all();        // both CTAs' barriers exist before either signals the other's
  cluster_wait_all();
  tc_fence_after();
  const uint32_t tmem_base = tmem_base_slot;
  volatile int* abort = &abort_flag;
  const int m_pairs = (p.m_tiles + 1) >> 1;
  const int total_tiles = m_pairs * p.n_tiles;
  const int cluster_id = blockIdx.x >> 1, n_clusters = gridDim.x >> 1;

  if (warp == 0 || warp == 10) {
    // two producer threads per CTA: warp 0 the operand tiles, warp 10 the scale blocks (see the single-CTA kernel)
    if (lane == 0) {
      pdl_wait_primary();           // components and blocked scales come from the kernels launched just before
      int stage = 0; uint32_t phase = 0;
      bool ok = true;
      for (int tile = cluster_id; tile < total_tiles && ok; tile += n_clusters) {
        const int mt = 2 * (p.n_fastest ? tile / p.n_tiles : tile % m_pairs) + static_cast<int>(rank), nt = p.n_fastest ? tile % p.n_tiles : tile / m_pairs;
        const int mt_sf = mt < p.m_tiles ? mt : p.m_tiles - 1;       // the odd last pair: rows past M are zero-filled anyway
        for (int ks = 0; ks < p.kstages; ++ks) {
          ok = wait_bounded(&empty_bar[stage], phase ^ 1, abort, p.status);
          if (!ok) break;
          uint8_t* dst = smem + stage * kStageBytes;
          if (warp == 0) {
            // the leader's barrier counts the operand bytes of both CTAs
            if (rank == 0) mbar_arrive_expect_tx(&full_bar[stage], 2 * kOpBytes);
            const uint32_t bar = mapa_shared(smem_u32(&full_bar[stage]), 0);
            tma_load_2d_pair(dst, &tmap_a1, ks * 128, mt * kW4TileM, bar);
            tma_load_2d_pair(dst + kW4ABytes, &tmap_a2, ks * 128, mt * kW4TileM, bar);
            tma_load_2d_pair(dst + 2 * kW4ABytes, &tmap_bh, ks * 128, nt * kTN + static_cast<int>(rank) * (kTN / 2), bar);
          } else {
            uint8_t* sf = dst + kOpBytes;
            mbar_arrive_expect_tx(&sf_full[stage], kW4SfBytes);
            const size_t a_off = (static_cast<size_t>(mt_sf) * p.sf_kgroups + 2 * ks) * 512;
            bulk_load(sf, p.sfa1 + a_off, 1024, &sf_full[stage]);
            bulk_load(sf + 1024, p.sfa2 + a_off, 1024, &sf_full[stage]);
            bulk_load(sf + 2048, p.sfb + (static_cast<size_t>(2 * nt) * p.sf_kgroups + 2 * ks) * 512, 1024, &sf_full[stage]);
            bulk_load(sf + 3072, p.sfb + (static_cast<size_t>(2 * nt + 1) * p.sf_kgroups + 2 * ks) * 512, 1024, &sf_full[stage]);
          }
          if (++stage == kW4PairStages) { stage = 0; phase ^= 1; }
        }
      }
    }
  } else if (warp == 1) {
    if (lane == 0 && rank == 0) {
      int stage = 0; uint32_t phase = 0;
      int it = 0, nstage = 0;
      bool ok = true;
      const uint64_t op_desc = smem_desc(0, 16, 1024, kSwizzle128B);    // 128-byte-swizzled K-major operand tile
      const uint32_t idesc_lo = idesc_block_scaled(/*E2M1*/ 1, 1, 2 * kW4TileM, kTN, 0, 0);
      const uint32_t idesc_hi = idesc_block_scaled(/*E2M1*/ 1, 1, 2 * kW4TileM, kTN, 2, 2);
      for (int tile = cluster_id; tile < total_tiles && ok; tile += n_clusters, ++it) {
        const int acc = (kAcc == 2) ? (it & 1) : 0;
        const uint32_t tphase = (kAcc == 2) ? ((it >> 1) & 1) : (it & 1);
        const uint32_t d_tmem = tmem_base + acc * kTN;
        ok = wait_bounded(&tempty_bar[acc], tphase ^ 1, abort, p.status);   // both epilogues have drained this accumulator
        if (!ok) break;
        tc_fence_after();
        for (int ks = 0; ks < p.kstages; ++ks, ++nstage) {
          const int set = nstage & 1;
          ok = wait_bounded(&full_bar[stage], phase, abort, p.status);
          if (!ok) break;
          ok = wait_bounded(&sf_ready[set], (nstage >> 1) & 1, abort, p.status);
          if (!ok) break;
          tc_fence_after();
          const uint64_t enc = static_cast<uint64_t>(smem_u32(smem + stage * kStageBytes) >> 4);
          const uint64_t a1d = op_desc + enc, a2d = a1d + (kW4ABytes >> 4), bd = a1d + (2 * kW4ABytes >> 4);
          const uint32_t sfa1_t = tmem_base + kSfCol + 32 * set;        // 2 k-groups x 4 columns; the two sets alternate
          const uint32_t sfa2_t = sfa1_t + 8;
          const uint32_t sfb_t = sfa1_t + 16;                            // 2 k-groups x 8 columns (256 weight rows)
#pragma unroll
          for (int kk = 0; kk < 4; ++kk) {                    // 64 elements (32 bytes) per MMA
            const int g = kk >> 1;
            const uint32_t idesc = (kk & 1) ? idesc_hi : idesc_lo;   // which pair of scale bytes of the 4-scale column
            mma_mxf4_pair(d_tmem, a1d + 2 * kk, bd + 2 * kk, idesc, sfa1_t + 4 * g, sfb_t + 8 * g, (ks > 0 || kk > 0) ? 1u : 0u);
            mma_mxf4_pair(d_tmem, a2d + 2 * kk, bd + 2 * kk, idesc, sfa2_t + 4 * g, sfb_t + 8 * g, 1u);
          }
          tc_commit_pair(&sf_free[set], 3);         // this set of scale columns may be rewritten in both CTAs
          tc_commit_pair(&empty_bar[stage], 3);     // frees the stage in both CTAs
          if (++stage == kW4PairStages) { stage = 0; phase ^= 1; }
        }
        if (!ok) break;
        tc_commit_pair(&tfull_bar[acc], 3);
      }
    }
  } else if (warp >= 6) {      // (warp 10 went the producers' way above)
    // Scale warps: each CTA writes its own TMEM (its activation rows' scales and all of the weight tile's).
    const int quad = warp & 3;
    const uint32_t leader_ready[2] = {mapa_shared(smem_u32(&sf_ready[0]), 0), mapa_shared(smem_u32(&sf_ready[1]), 0)};
    int stage = 0; uint32_t phase = 0;
    int n = 0;
    bool ok = true;
    for (int tile = cluster_id; tile < total_tiles && ok; tile += n_clusters) {
      for (int ks = 0; ks < p.kstages; ++ks, ++n) {
        const int set = n & 1;
        ok = wait_bounded(&sf_full[stage], phase, abort, p.status);
        if (!ok) break;
        if (n >= 2) {                        // the MMAs that read this set two stages ago are done
          ok = wait_bounded(&sf_free[set], ((n >> 1) - 1) & 1, abort, p.status);
          if (!ok) break;
          tc_fence_after();
        }
        const uint4* sf = reinterpret_cast<const uint4*>(smem + stage * kStageBytes + kOpBytes) + lane;
        uint32_t v[32];
        constexpr int kBlk[8] = {0, 1, 2, 3, 4, 6, 5, 7};     // column order: sfa1 (g0, g1), sfa2 (g0, g1), then per K group the two weight-row blocks
#pragma unroll
        for (int j = 0; j < 8; ++j) {
          const uint4 q = sf[kBlk[j] * 32];
          v[4 * j] = q.x; v[4 * j + 1] = q.y; v[4 * j + 2] = q.z; v[4 * j + 3] = q.w;
        }
        tmem_st32(tmem_base + (static_cast<uint32_t>(quad * 32) << 16) + kSfCol + 32 * set, v);
        tmem_st_wait();
        tc_fence_before();
        __syncwarp();
        if (lane == 0) mbar_arrive_remote(leader_ready[set]);
        if (++stage == kW4PairStages) { stage = 0; phase ^= 1; }
      }
    }
  } else {
    // Epilogue as in the single-CTA kernel: TMEM -> registers -> (BF16) -> swizzled staging buffer -> TMA store.
    const int quad = warp & 3;
    uint8_t* stage_buf = smem + kW4PairStages * kStageBytes + quad * (2 * kW4StoreBytes);
    const uint32_t swz = static_cast<uint32_t>((lane >> 1) & 3);
    int it = 0, buf = 0;
    bool ok = true;
    const uint32_t leader_tempty[2] = {mapa_shared(smem_u32(&tempty_bar[0]), 0), mapa_shared(smem_u32(&tempty_bar[1]), 0)};
    for (int tile = cluster_id; tile < total_tiles && ok; tile += n_clusters, ++it) {
      const int mt = 2 * (p.n_fastest ? tile / p.n_tiles : tile % m_pairs) + static_cast<int>(rank), nt = p.n_fastest ? tile % p.n_tiles : tile / m_pairs;
      const int acc = (kAcc == 2) ? (it & 1) : 0;
      const uint32_t tphase = (kAcc == 2) ? ((it >> 1) & 1) : (it & 1);
      ok = wait_bounded(&tfull_bar[acc], tphase, abort, p.status);
      if (!ok) break;
      tc_fence_after();
      const int row0 = mt * kW4TileM + quad * 32;
      const uint32_t trow = tmem_base + (static_cast<uint32_t>(quad * 32) << 16) + acc * kTN;
      const int cols_here = p.N - nt * kTN < kTN ? p.N - nt * kTN : kTN;
      const int cend = row0 < p.M ? cols_here : 0;
      if (cend == 0) {
        tc_fence_before();
        __syncwarp();
        if (lane == 0) mbar_arrive_remote(leader_tempty[acc]);
      }
      auto release_acc = [&]() {                    // all that is needed of this accumulator is in registers
        tc_fence_before();
        __syncwarp();
        if (lane == 0) mbar_arrive_remote(leader_tempty[acc]);
      };
      auto store_chunk = [&](const uint32_t (&o)[16], int c0) {
        uint8_t* sb = stage_buf + buf * kW4StoreBytes;
        if (lane == 0) bulk_wait_group_read<1>();    // the store that read this buffer two chunks ago is done with it
        __syncwarp();
        uint8_t* srow = sb + lane * 64;
#pragma unroll
        for (int j = 0; j < 4; ++j)
          *reinterpret_cast<uint4*>(srow + ((static_cast<uint32_t>(j) ^ swz) << 4)) = make_uint4(o[4 * j], o[4 * j + 1], o[4 * j + 2], o[4 * j + 3]);
        fence_proxy_async_smem();
        __syncwarp();
        if (lane == 0) {
          tma_store_2d(&tmap_y, nt * kTN + c0, row0, sb);
          bulk_commit_group();
        }
        buf ^= 1;
      };
      if (p.ytype == MSD_OUT_BF16) {
        // The load of the next 32 columns is in flight while a chunk is converted and stored: a TMEM load takes about
        // 450 cycles, and with one accumulator no MMA runs while the tile drains.
        auto bf16_chunk = [&](const uint32_t (&v)[32], int c0) {
          uint32_t o[16];
#pragma unroll
          for (int j = 0; j < 16; ++j) {
            const __nv_bfloat162 h = __floats2bfloat162_rn(__uint_as_float(v[2 * j]), __uint_as_float(v[2 * j + 1]));
            o[j] = *reinterpret_cast<const uint32_t*>(&h);
          }
          store_chunk(o, c0);
        };
        uint32_t va[32], vb[32];
        if (cend > 0) {
          tmem_ld32(trow, va);
          tmem_ld_wait_for(va);
        }
        for (int c0 = 0; c0 < cend; c0 += 64) {
          const bool more_b = c0 + 32 < cend;
          if (more_b) tmem_ld32(trow + c0 + 32, vb); else release_acc();
          bf16_chunk(va, c0);
          if (!more_b) break;
          tmem_ld_wait_for(vb);
          const bool more_a = c0 + 64 < cend;
          if (more_a) tmem_ld32(trow + c0 + 64, va); else release_acc();
          bf16_chunk(vb, c0 + 32);
          if (more_a) tmem_ld_wait_for(va);
        }
      } else {
        for (int c0 = 0; c0 < cend; c0 += 16) {
          uint32_t o[16];
          tmem_ld16(trow + c0, o);
          tmem_ld_wait();
          if (c0 + 16 >= cend) release_acc();
          store_chunk(o, c0);
        }
      }
    }
    if (lane == 0) bulk_wait_group<0>();            // every store has been written before the CTA goes away
  }

  // Neither CTA leaves while the other may still signal its barriers or (through the pair MMAs) read its shared memory.
  tc_fence_before();
  __syncthreads();
  cluster_arrive_all();
  cluster_wait_all();
  if (warp == 1) {
    tc_fence_after();
    tmem_dealloc_pair(tmem_base, kW4TmemCols);
  }
}

struct GemmW4Plan {
  int m_tiles, n_tiles, kstages, sf_kgroups, grid, tile_n;
  int ksplit, kper, a_rows, nstages;
  size_t off_q1, off_q2, off_sfa1, off_sfa2, off_sfb, off_part, bytes;
};

// The CTA-pair kernel (256 tokens x 256 weight rows per pair of CTAs: half the weight tile per CTA, so less shared-memory
// traffic per MMA, and four stages) takes the shapes on which its tiles fill the GPU about as well as the single-CTA
// kernel's: at equal rounds x tile width it is 5-15 % faster, and where the 128 x 224 tiles need an extra round
// (M = 2048, N = 4096) by a quarter.  Not where the single-CTA kernel would split K (few tiles).
// MSD_W4_PAIR=0/1 forces the choice.
static bool w4_use_pair(int64_t M, int64_t N, int64_t K) {
  (void)K;
  if (const int forced = option(OPT_W4_PAIR); forced >= 0) return forced != 0;     // testing aid
  const int64_t m_tiles = (M + kW4TileM - 1) / kW4TileM, n_tiles = (N + 255) / 256;
  const int64_t clusters = sm_count() / 2, pair_tiles = (m_tiles + 1) / 2 * n_tiles, single_tiles = m_tiles * ((N + 223) / 224);
  // an odd number of token tiles leaves the last pair's second CTA without rows: only where that is a small share
  if (!(m_tiles >= 2 && (m_tiles % 2 == 0 || m_tiles >= 9) && 2 * single_tiles > sm_count())) return false;
  // rounds x tile width of either kernel (a pair tile takes a pair as long as a 128 x 256 tile takes a CTA)
  const int64_t cost_pair = (pair_tiles + clusters - 1) / clusters * 256, cost_single = (single_tiles + sm_count() - 1) / sm_count() * 224;
  return 100 * cost_pair <= 110 * cost_single;
}

// Weight rows per tile: MSD_W4_TILEN (224 or 256) if set; else 256 for the CTA-pair kernel (one accumulator) and 224 for
// the single-CTA kernel (two accumulators: the epilogue of a tile overlaps the MMAs of the next).
static int w4_tile_n(bool pair = false) {
  if (const int forced = option(OPT_W4_TILEN); forced >= 0) return forced == 256 ? 256 : 224;     // testing aid
  return pair ? 256 : 224;
}

static GemmW4Plan plan_w4(int64_t M, int64_t N, int64_t K) {
  GemmW4Plan pl;
  const int tile_n = w4_tile_n(w4_use_pair(M, N, K));
  pl.tile_n = tile_n;
  pl.m_tiles = static_cast<int>((M + kW4TileM - 1) / kW4TileM);
  pl.n_tiles = static_cast<int>((N + tile_n - 1) / tile_n);
  pl.kstages = static_cast<int>((K + kW4BlockK - 1) / kW4BlockK);
  pl.sf_kgroups = 2 * pl.kstages;
  const int tiles = pl.m_tiles * pl.n_tiles;
  // Few output tiles and a long K (decode shapes): split K so that there is about one work item per SM, each at
  // least four stages long; the FP32 partial tiles are added by a second kernel.
  pl.ksplit = 1;
  pl.kper = pl.kstages;
  {
    const int forced = option(OPT_W4_KSPLIT);     // testing aid
    int want = forced >= 0 ? forced : (2 * tiles <= sm_count() ? sm_count() / tiles : 1);
    if (want > pl.kstages / 4) want = pl.kstages / 4;
    if (want > 1) {
      pl.kper = (pl.kstages + want - 1) / want;
      pl.ksplit = (pl.kstages + pl.kper - 1) / pl.kper;
    }
  }
  const int items = tiles * pl.ksplit;
  int grid = sm_count();
  if (grid > items) grid = items;
  pl.grid = grid;
  // one token tile of fewer than 128 rows: only those rows are loaded and the stages are packed (more of them fit)
  pl.a_rows = pl.m_tiles == 1 ? static_cast<int>((M + 7) / 8 * 8) : kW4TileM;
  {
    const size_t stage_bytes = static_cast<size_t>(2 * pl.a_rows * 128 + tile_n * 128 + kW4SfBytes);
    int ns = static_cast<int>((227 * 1024 - 2048 - 8 * kW4StoreBytes - 1024) / stage_bytes);
    pl.nstages = ns > 8 ? 8 : ns;
  }
  size_t off = 0;
  pl.off_q1 = off;   off = round_up(off + static_cast<size_t>(M) * (K / 2), 1024);
  pl.off_q2 = off;   off = round_up(off + static_cast<size_t>(M) * (K / 2), 1024);
  pl.off_sfa1 = off; off = round_up(off + static_cast<size_t>(pl.m_tiles) * pl.sf_kgroups * 512, 1024);
  pl.off_sfa2 = off; off = round_up(off + static_cast<size_t>(pl.m_tiles) * pl.sf_kgroups * 512, 1024);
  pl.off_sfb = off;  off = round_up(off + static_cast<size_t>(2 * pl.n_tiles) * pl.sf_kgroups * 512, 1024);
  pl.off_part = off;
  if (pl.ksplit > 1) off = round_up(off + static_cast<size_t>(pl.ksplit) * pl.m_tiles * kW4TileM * N * sizeof(float), 1024);
  pl.bytes = off;
  return pl;
}

// ---- grouped (mixture of experts) ----------------------------------------------------------------------------------
// Workspace: components of up to 64 groups at a time as token tiles of 128 rows, their scale blocks, and the blocked
// scales of all experts' weights.
struct GroupedW4Plan {
  int n_tiles, kstages, sf_kgroups, tile_n;
  size_t off_q1, off_q2, off_sfa1, off_sfa2, off_sfb, bytes;
};
static GroupedW4Plan plan_grouped_w4(int32_t E, int64_t N, int64_t K, int groups) {
  GroupedW4Plan pl;
  // Tile width: the one whose tiles fill the SMs in fewer, or shorter, rounds (groups = non-empty groups of the first
  // launch; the workspace is sized for the wider layout of the blocked weight scales either way)
  if (const int forced = option(OPT_W4_TILEN); forced >= 0) {
    pl.tile_n = forced == 256 ? 256 : 224;
  } else {
    const long long g = groups < 1 ? 1 : (groups > kMaxRowGroups ? kMaxRowGroups : groups);
    const long long t224 = g * ((N + 223) / 224), t256 = g * ((N + 255) / 256);
    const long long c224 = (t224 + sm_count() - 1) / sm_count() * 224, c256 = (t256 + sm_count() - 1) / sm_count() * 256;
    pl.tile_n = c256 < c224 ? 256 : 224;
  }
  pl.n_tiles = static_cast<int>((N + pl.tile_n - 1) / pl.tile_n);
  pl.kstages = static_cast<int>((K + kW4BlockK - 1) / kW4BlockK);
  pl.sf_kgroups = 2 * pl.kstages;
  const size_t rows = static_cast<size_t>(kMaxRowGroups) * kW4TileM;
  size_t off = 0;
  pl.off_q1 = off;   off = round_up(off + rows * (K / 2), 1024);
  pl.off_q2 = off;   off = round_up(off + rows * (K / 2), 1024);
  pl.off_sfa1 = off; off = round_up(off + static_cast<size_t>(kMaxRowGroups) * pl.sf_kgroups * 512, 1024);
  pl.off_sfa2 = off; off = round_up(off + static_cast<size_t>(kMaxRowGroups) * pl.sf_kgroups * 512, 1024);
  // (N + 223) / 224 tiles is the larger count of the two widths
  pl.off_sfb = off;  off = round_up(off + static_cast<size_t>(E) * 2 * ((N + 223) / 224) * pl.sf_kgroups * 512, 1024);
  pl.bytes = off;
  return pl;
}

// Weight scales brought into the blocked layout once (msd_prepare_w4a16_scales): both tile widths' layouts back to
// back, each E matrices of 2 * ceil(N / width) row blocks x sf_kgroups blocks of 512 bytes.
struct PreparedScales {
  int sf_kgroups;
  size_t off224, off256, bytes;
};
static PreparedScales prepared_scales_layout(int32_t E, int64_t N, int64_t K) {
  PreparedScales ps;
  ps.sf_kgroups = 2 * static_cast<int>((K + kW4BlockK - 1) / kW4BlockK);
  ps.off224 = 0;
  ps.off256 = round_up(static_cast<size_t>(E) * 2 * ((N + 223) / 224) * ps.sf_kgroups * 512, 1024);
  ps.bytes = ps.off256 + round_up(static_cast<size_t>(E) * 2 * ((N + 255) / 256) * ps.sf_kgroups * 512, 1024);
  return ps;
}

__global__ void __launch_bounds__(256) sf_relayout_kernel(const SfRelayout rl) {
  __shared__ uint32_t sm_rl[kSfRelayoutSmemWords];
  sf_relayout(rl, static_cast<int>(blockIdx.x), static_cast<int>(gridDim.x), sm_rl);
}

static msd_status_t gemm_w4a16_impl(const void* x_bf16, const uint8_t* w_fp4, const uint8_t* w_e8m0, const uint8_t* prepared,
                                    int64_t M, int64_t N, int64_t K, void* y, msd_out_t ytype, void* workspace,
                                    size_t workspace_bytes, void* stream);
static msd_status_t grouped_gemm_w4a16_impl(const void* x_bf16, const uint8_t* w_fp4, const uint8_t* w_e8m0, const uint8_t* prepared,
                                            const int32_t* group_sizes_host, int32_t E, int64_t N, int64_t K, void* y,
                                            msd_out_t ytype, void* workspace, size_t workspace_bytes, void* stream);

}  // namespace msd

extern "C" {

size_t msd_w4a16_prepared_scales_bytes(int32_t E, int64_t N, int64_t K) {
  if (E < 1 || N < 1 || K < 128 || K % 128 != 0) return 0;
  return msd::prepared_scales_layout(E, N, K).bytes;
}

msd_status_t msd_prepare_w4a16_scales(const uint8_t* w_e8m0, int32_t E, int64_t N, int64_t K, uint8_t* prepared, void* stream) {
  using namespace msd;
  if (E < 1 || N < 1 || K < 128 || K % 128 != 0 || N > (1 << 24) || K > (1 << 24) || static_cast<int64_t>(E) * N > 0x7FFFFFFFLL)
    return MSD_ERR_BAD_SHAPE;
  if (!w_e8m0 || !prepared) return MSD_ERR_NULL_POINTER;
  if (!aligned(w_e8m0, 4) || !aligned(prepared, 1024)) return MSD_ERR_BAD_ALIGNMENT;
  const PreparedScales ps = prepared_scales_layout(E, N, K);
  for (int width = 224; width <= 256; width += 32) {
    SfRelayout rl = {};
    rl.src = w_e8m0; rl.dst = prepared + (width == 224 ? ps.off224 : ps.off256); rl.rows = N; rl.kblocks = static_cast<int>(K / 32);
    rl.sf_kgroups = ps.sf_kgroups; rl.tile_rows = width; rl.row_blocks = 2 * static_cast<int>((N + width - 1) / width);
    rl.matrices = E;
    const long long units = static_cast<long long>(E) * rl.row_blocks * ((ps.sf_kgroups + 31) / 32);
    const long long cap = static_cast<long long>(sm_count()) * 8;
    sf_relayout_kernel<<<static_cast<unsigned>(units < cap ? units : cap), 256, 0, static_cast<cudaStream_t>(stream)>>>(rl);
    if (cudaGetLastError() != cudaSuccess) return MSD_ERR_CUDA;
  }
  return MSD_OK;
}

size_t msd_gemm_w4a16_workspace_bytes(int64_t M, int64_t N, int64_t K) {
  if (M < 1 || N < 1 || K < 128 || K % 128 != 0) return 0;
  return msd::plan_w4(M, N, K).bytes;
}

msd_status_t msd_gemm_w4a16(const void* x_bf16, const uint8_t* w_fp4, const uint8_t* w_e8m0, int64_t M, int64_t N,
                            int64_t K, void* y, msd_out_t ytype, void* workspace, size_t workspace_bytes,
                            void* stream) {
  if (!w_e8m0) return MSD_ERR_NULL_POINTER;
  return msd::gemm_w4a16_impl(x_bf16, w_fp4, w_e8m0, nullptr, M, N, K, y, ytype, workspace, workspace_bytes, stream);
}

msd_status_t msd_gemm_w4a16_prepared(const void* x_bf16, const uint8_t* w_fp4, const uint8_t* prepared_scales, int64_t M,
                                     int64_t N, int64_t K, void* y, msd_out_t ytype, void* workspace,
                                     size_t workspace_bytes, void* stream) {
  if (!prepared_scales) return MSD_ERR_NULL_POINTER;
  return msd::gemm_w4a16_impl(x_bf16, w_fp4, nullptr, prepared_scales, M, N, K, y, ytype, workspace, workspace_bytes, stream);
}

}  // extern "C"

namespace msd {

static msd_status_t gemm_w4a16_impl(const void* x_bf16, const uint8_t* w_fp4, const uint8_t* w_e8m0, const uint8_t* prepared,
                                    int64_t M, int64_t N, int64_t K, void* y, msd_out_t ytype, void* workspace,
                                    size_t workspace_bytes, void* stream) {
  if (M < 1 || N < 1 || K < 128 || K % 128 != 0 || N % 8 != 0 || M > (1 << 24) || N > (1 << 24) || K > (1 << 24))
    return MSD_ERR_BAD_SHAPE;
  if (ytype != MSD_OUT_BF16 && ytype != MSD_OUT_FP32) return MSD_ERR_UNSUPPORTED;
  if (!x_bf16 || !w_fp4 || !y || !workspace) return MSD_ERR_NULL_POINTER;
  if (!aligned(x_bf16, 16) || !aligned(w_fp4, 16) || !aligned(w_e8m0, 4) || !aligned(prepared, 1024) || !aligned(y, 16) ||
      !aligned(workspace, 1024))
    return MSD_ERR_BAD_ALIGNMENT;     // the scale relayout reads the E8M0 rows as 32-bit words
  const GemmW4Plan pl = plan_w4(M, N, K);
  if (workspace_bytes < pl.bytes) return MSD_ERR_WORKSPACE_TOO_SMALL;
  unsigned* status = device_status_ptr();
  if (!status) return MSD_ERR_CUDA;
  cudaStream_t s = static_cast<cudaStream_t>(stream);
  uint8_t* ws = static_cast<uint8_t*>(workspace);
  uint8_t* q1 = ws + pl.off_q1;
  uint8_t* q2 = ws + pl.off_q2;

  // The weight scales go into the blocked layout in the same launch as the decomposition of x.  (Letting the GEMM start
  // on the first token tiles while the others are still being decomposed, behind per-tile progress counters, was built
  // and measured: the decomposition, held to two CTAs per SM so that both kernels fit, took twice as long and the GEMM
  // beside it lost what the earlier start gained.)
  const bool use_pair = w4_use_pair(M, N, K);
  const bool pdl = option(OPT_NO_PDL) <= 0;
  SfRelayout rl = {};
  rl.src = w_e8m0; rl.dst = ws + pl.off_sfb; rl.rows = N; rl.kblocks = static_cast<int>(K / 32);
  rl.sf_kgroups = pl.sf_kgroups; rl.tile_rows = pl.tile_n; rl.row_blocks = 2 * pl.n_tiles;
  // (scales prepared once by msd_prepare_w4a16_scales: nothing to bring into the blocked layout here)
  const uint8_t* sfb = ws + pl.off_sfb;
  if (prepared) {
    const PreparedScales ps = prepared_scales_layout(1, N, K);
    sfb = prepared + (pl.tile_n == 224 ? ps.off224 : ps.off256);
  }
  msd_status_t st = launch_decompose_mxfp4(x_bf16, M, K, K, q1, q2, ws + pl.off_sfa1, ws + pl.off_sfa2, pl.sf_kgroups, s,
                                           prepared ? nullptr : &rl);
  if (st != MSD_OK) return st;

  CUtensorMap tmap_a1, tmap_a2, tmap_b;
  const uint64_t kb = static_cast<uint64_t>(K / 2);
  if (!encode_tmap_2d(&tmap_a1, CU_TENSOR_MAP_DATA_TYPE_UINT8, q1, kb, M, kb, 128, static_cast<uint32_t>(use_pair ? kW4TileM : pl.a_rows), CU_TENSOR_MAP_SWIZZLE_128B) ||
      !encode_tmap_2d(&tmap_a2, CU_TENSOR_MAP_DATA_TYPE_UINT8, q2, kb, M, kb, 128, static_cast<uint32_t>(use_pair ? kW4TileM : pl.a_rows), CU_TENSOR_MAP_SWIZZLE_128B) ||
      !encode_tmap_2d(&tmap_b, CU_TENSOR_MAP_DATA_TYPE_UINT8, w_fp4, kb, N, kb, 128, static_cast<uint32_t>(pl.tile_n), CU_TENSOR_MAP_SWIZZLE_128B))
    return MSD_ERR_CUDA;

  GemmW4Params p;
  p.M = static_cast<int>(M); p.N = static_cast<int>(N); p.K = static_cast<int>(K);
  p.m_tiles = pl.m_tiles; p.n_tiles = pl.n_tiles; p.kstages = pl.kstages; p.sf_kgroups = pl.sf_kgroups;
  p.sfa1 = ws + pl.off_sfa1; p.sfa2 = ws + pl.off_sfa2; p.sfb = sfb;
  p.y = y; p.ytype = ytype; p.status = status;
  p.a_rows = kW4TileM; p.nstages = kW4Stages; p.ksplit = 1; p.kper = pl.kstages; p.part_rows = 0;
  {
    // Tile order.  A wave of CTAs either shares a few weight tiles and sweeps the token tiles (token tile fastest)
    // or the other way round; the operand that is swept should be the one that stays in L2 (40 MB assumed usable for
    // it).  Both components of x weigh M x K bytes, the weights N x K / 2.
    const double l2 = 40.0 * 1024 * 1024, a_bytes = static_cast<double>(M) * K, w_bytes = static_cast<double>(N) * K / 2;
    p.n_fastest = a_bytes <= l2 ? 0 : (w_bytes <= l2 ? 1 : (a_bytes > w_bytes ? 1 : 0));
  }

  // With a K split the kernel writes FP32 partial tiles (split s at rows s * part_rows ...) and a second kernel adds them.
  CUtensorMap tmap_y;
  const bool split = pl.ksplit > 1 && !use_pair;        // the CTA-pair kernel does not split K
  const bool ybf = !split && ytype == MSD_OUT_BF16;
  float* part = reinterpret_cast<float*>(ws + pl.off_part);
  const uint64_t part_rows = static_cast<uint64_t>(pl.m_tiles) * kW4TileM;
  if (!encode_tmap_2d(&tmap_y, ybf ? CU_TENSOR_MAP_DATA_TYPE_BFLOAT16 : CU_TENSOR_MAP_DATA_TYPE_FLOAT32, split ? static_cast<void*>(part) : y,
                      static_cast<uint64_t>(N), split ? part_rows * pl.ksplit : static_cast<uint64_t>(M),
                      static_cast<uint64_t>(N) * (ybf ? 2 : 4), ybf ? 32 : 16, 32, CU_TENSOR_MAP_SWIZZLE_64B))
    return MSD_ERR_CUDA;
  if (use_pair) {
    // CTA pairs: each CTA loads half of the weight tile's rows
    CUtensorMap tmap_bh;
    if (!encode_tmap_2d(&tmap_bh, CU_TENSOR_MAP_DATA_TYPE_UINT8, w_fp4, kb, N, kb, 128, static_cast<uint32_t>(pl.tile_n / 2),
                        CU_TENSOR_MAP_SWIZZLE_128B))
      return MSD_ERR_CUDA;
    const size_t smem_pair = static_cast<size_t>(kW4PairStages) * (2 * kW4ABytes + (pl.tile_n / 2) * 128 + kW4SfBytes) + 8 * kW4StoreBytes + 1024;
    static bool attr_pair_done = false;
    if (!attr_pair_done) {
      if (cudaFuncSetAttribute(gemm_w4a16_pair_kernel<256>, cudaFuncAttributeMaxDynamicSharedMemorySize, 227 * 1024 - 2048) != cudaSuccess ||
          cudaFuncSetAttribute(gemm_w4a16_pair_kernel<224>, cudaFuncAttributeMaxDynamicSharedMemorySize, 227 * 1024 - 2048) != cudaSuccess)
        return MSD_ERR_CUDA;
      attr_pair_done = true;
    }
    const int pair_tiles = ((pl.m_tiles + 1) / 2) * pl.n_tiles;
    int clusters = sm_count() / 2;
    if (clusters > pair_tiles) clusters = pair_tiles;
    const cudaError_t pe = pl.tile_n == 256
        ? launch_pdl_cluster(gemm_w4a16_pair_kernel<256>, dim3(2 * clusters), dim3(kW4PairThreads), smem_pair, s, pdl, 2u, tmap_a1, tmap_a2, tmap_bh, tmap_y, p)
        : launch_pdl_cluster(gemm_w4a16_pair_kernel<224>, dim3(2 * clusters), dim3(kW4PairThreads), smem_pair, s, pdl, 2u, tmap_a1, tmap_a2, tmap_bh, tmap_y, p);
    if (pe != cudaSuccess) return MSD_ERR_CUDA;
    return MSD_OK;
  }
  if (split) p.ytype = MSD_OUT_FP32;
  p.ksplit = pl.ksplit; p.kper = pl.kper; p.part_rows = static_cast<int>(part_rows);
  p.a_rows = pl.a_rows; p.nstages = pl.nstages;
  const size_t smem_bytes = static_cast<size_t>(pl.nstages) * (2 * pl.a_rows * 128 + pl.tile_n * 128 + kW4SfBytes) + 8 * kW4StoreBytes + 1024;
  static bool attr_done = false;
  if (!attr_done) {
    if (cudaFuncSetAttribute(gemm_w4a16_kernel<256, false>, cudaFuncAttributeMaxDynamicSharedMemorySize, 227 * 1024 - 2048) != cudaSuccess ||
        cudaFuncSetAttribute(gemm_w4a16_kernel<224, false>, cudaFuncAttributeMaxDynamicSharedMemorySize, 227 * 1024 - 2048) != cudaSuccess)
      return MSD_ERR_CUDA;
    attr_done = true;
  }
  const cudaError_t le = pl.tile_n == 256
      ? launch_pdl(gemm_w4a16_kernel<256, false>, dim3(pl.grid), dim3(kW4ThreadsSf), smem_bytes, s, pdl, tmap_a1, tmap_a2, tmap_b, tmap_y, p, GemmW4NoGroups())
      : launch_pdl(gemm_w4a16_kernel<224, false>, dim3(pl.grid), dim3(kW4ThreadsSf), smem_bytes, s, pdl, tmap_a1, tmap_a2, tmap_b, tmap_y, p, GemmW4NoGroups());
  if (le != cudaSuccess) return MSD_ERR_CUDA;
  if (split) {
    const msd_status_t rs = launch_ksplit_reduce(part, pl.ksplit, static_cast<int64_t>(part_rows) * N, M, N, y, static_cast<int>(ytype), s, pdl);
    if (rs != MSD_OK) return rs;
  }
  return MSD_OK;
}

}  // namespace msd

extern "C" {

size_t msd_grouped_gemm_w4a16_workspace_bytes(int32_t E, int64_t N, int64_t K) {
  if (E < 1 || N < 1 || K < 128 || K % 128 != 0) return 0;
  return msd::plan_grouped_w4(E, N, K, E).bytes;
}

msd_status_t msd_grouped_gemm_w4a16(const void* x_bf16, const uint8_t* w_fp4, const uint8_t* w_e8m0,
                                    const int32_t* group_sizes_host, int32_t E, int64_t N, int64_t K, void* y,
                                    msd_out_t ytype, void* workspace, size_t workspace_bytes, void* stream) {
  if (!w_e8m0) return MSD_ERR_NULL_POINTER;
  return msd::grouped_gemm_w4a16_impl(x_bf16, w_fp4, w_e8m0, nullptr, group_sizes_host, E, N, K, y, ytype, workspace, workspace_bytes, stream);
}

msd_status_t msd_grouped_gemm_w4a16_prepared(const void* x_bf16, const uint8_t* w_fp4, const uint8_t* prepared_scales,
                                             const int32_t* group_sizes_host, int32_t E, int64_t N, int64_t K, void* y,
                                             msd_out_t ytype, void* workspace, size_t workspace_bytes, void* stream) {
  if (!prepared_scales) return MSD_ERR_NULL_POINTER;
  return msd::grouped_gemm_w4a16_impl(x_bf16, w_fp4, nullptr, prepared_scales, group_sizes_host, E, N, K, y, ytype, workspace, workspace_bytes, stream);
}

}  // extern "C"

namespace msd {

static msd_status_t grouped_gemm_w4a16_impl(const void* x_bf16, const uint8_t* w_fp4, const uint8_t* w_e8m0, const uint8_t* prepared,
                                            const int32_t* group_sizes_host, int32_t E, int64_t N, int64_t K, void* y,
                                            msd_out_t ytype, void* workspace, size_t workspace_bytes, void* stream) {
  if (E < 1 || N < 1 || K < 128 || K % 128 != 0 || N % 8 != 0 || N > (1 << 24) || K > (1 << 24) ||
      static_cast<int64_t>(E) * N > 0x7FFFFFFFLL)
    return MSD_ERR_BAD_SHAPE;
  if (ytype != MSD_OUT_BF16 && ytype != MSD_OUT_FP32) return MSD_ERR_UNSUPPORTED;
  if (!x_bf16 || !w_fp4 || !group_sizes_host || !y || !workspace) return MSD_ERR_NULL_POINTER;
  if (!aligned(x_bf16, 16) || !aligned(w_fp4, 16) || !aligned(w_e8m0, 4) || !aligned(prepared, 1024) || !aligned(y, 16) ||
      !aligned(workspace, 1024))
    return MSD_ERR_BAD_ALIGNMENT;
  int64_t M_total = 0;
  int nonempty = 0, largest = 0;
  for (int e = 0; e < E; ++e) {
    if (group_sizes_host[e] < 0 || group_sizes_host[e] > kW4TileM) return MSD_ERR_BAD_SHAPE;     // decode regime per expert
    M_total += group_sizes_host[e];
    nonempty += group_sizes_host[e] > 0 ? 1 : 0;
    if (group_sizes_host[e] > largest) largest = group_sizes_host[e];
  }
  if (M_total > 0x7FFFFFFFLL) return MSD_ERR_BAD_SHAPE;
  const GroupedW4Plan pl = plan_grouped_w4(E, N, K, nonempty);
  const int a_rows = (largest + 7) / 8 * 8;             // rows of a token tile worth loading (whole 8-row swizzle atoms)
  if (workspace_bytes < pl.bytes) return MSD_ERR_WORKSPACE_TOO_SMALL;
  if (M_total == 0) return MSD_OK;
  unsigned* status = device_status_ptr();
  if (!status) return MSD_ERR_CUDA;
  cudaStream_t s = static_cast<cudaStream_t>(stream);
  uint8_t* ws = static_cast<uint8_t*>(workspace);
  uint8_t* q1 = ws + pl.off_q1;
  uint8_t* q2 = ws + pl.off_q2;
  const bool ybf = ytype == MSD_OUT_BF16;
  const uint64_t kb = static_cast<uint64_t>(K / 2);
  CUtensorMap tmap_a1, tmap_a2, tmap_b, tmap_y;
  if (!encode_tmap_2d(&tmap_a1, CU_TENSOR_MAP_DATA_TYPE_UINT8, q1, kb, static_cast<uint64_t>(kMaxRowGroups) * kW4TileM, kb, 128, static_cast<uint32_t>(a_rows), CU_TENSOR_MAP_SWIZZLE_128B) ||
      !encode_tmap_2d(&tmap_a2, CU_TENSOR_MAP_DATA_TYPE_UINT8, q2, kb, static_cast<uint64_t>(kMaxRowGroups) * kW4TileM, kb, 128, static_cast<uint32_t>(a_rows), CU_TENSOR_MAP_SWIZZLE_128B) ||
      !encode_tmap_2d(&tmap_b, CU_TENSOR_MAP_DATA_TYPE_UINT8, w_fp4, kb, static_cast<uint64_t>(E) * N, kb, 128, static_cast<uint32_t>(pl.tile_n), CU_TENSOR_MAP_SWIZZLE_128B) ||
      !encode_tmap_2d(&tmap_y, ybf ? CU_TENSOR_MAP_DATA_TYPE_BFLOAT16 : CU_TENSOR_MAP_DATA_TYPE_FLOAT32, y, static_cast<uint64_t>(N),
                      static_cast<uint64_t>(M_total), static_cast<uint64_t>(N) * (ybf ? 2 : 4), ybf ? 32 : 16, 32, CU_TENSOR_MAP_SWIZZLE_64B))
    return MSD_ERR_CUDA;
  const size_t stage_bytes = static_cast<size_t>(2 * a_rows * 128 + pl.tile_n * 128 + kW4SfBytes);
  int nstages = static_cast<int>((227 * 1024 - 2048 - 8 * kW4StoreBytes - 1024) / stage_bytes);
  if (nstages > 8) nstages = 8;
  const size_t smem_bytes = nstages * stage_bytes + 8 * kW4StoreBytes + 1024;
  static bool attr_done = false;
  if (!attr_done) {
    if (cudaFuncSetAttribute(gemm_w4a16_kernel<256, true>, cudaFuncAttributeMaxDynamicSharedMemorySize, 227 * 1024 - 2048) != cudaSuccess ||
        cudaFuncSetAttribute(gemm_w4a16_kernel<224, true>, cudaFuncAttributeMaxDynamicSharedMemorySize, 227 * 1024 - 2048) != cudaSuccess)
      return MSD_ERR_CUDA;
    attr_done = true;
  }
  const bool pdl = option(OPT_NO_PDL) <= 0;

  // up to 64 non-empty groups per pair of launches (decomposition + GEMM); the weight scales of all experts are brought
  // into the blocked layout by the first decomposition launch
  bool scales_done = prepared != nullptr;
  const uint8_t* sfb = ws + pl.off_sfb;
  if (prepared) {
    const PreparedScales ps = prepared_scales_layout(E, N, K);
    sfb = prepared + (pl.tile_n == 224 ? ps.off224 : ps.off256);
  }
  int e = 0;
  int64_t row = 0;
  while (e < E) {
    GemmW4Groups grp = {};
    RowGroups rg = {};
    const int64_t row_first = row;
    while (e < E && grp.n < kMaxRowGroups) {
      const int sz = group_sizes_host[e];
      if (sz > 0) {
        grp.expert[grp.n] = e;
        grp.off[grp.n] = static_cast<int>(row);
        rg.off[grp.n] = static_cast<int>(row - row_first);
        row += sz;
        ++grp.n;
      }
      ++e;
    }
    if (grp.n == 0) break;
    grp.off[grp.n] = static_cast<int>(row);
    rg.off[grp.n] = static_cast<int>(row - row_first);
    rg.n = grp.n;
    SfRelayout rl = {};
    rl.src = w_e8m0; rl.dst = ws + pl.off_sfb; rl.rows = N; rl.kblocks = static_cast<int>(K / 32);
    rl.sf_kgroups = pl.sf_kgroups; rl.tile_rows = pl.tile_n; rl.row_blocks = 2 * pl.n_tiles; rl.matrices = E;
    msd_status_t st = launch_decompose_mxfp4(static_cast<const uint16_t*>(x_bf16) + row_first * K, row - row_first, K, K, q1, q2,
                                             ws + pl.off_sfa1, ws + pl.off_sfa2, pl.sf_kgroups, s, scales_done ? nullptr : &rl, &rg);
    if (st != MSD_OK) return st;
    scales_done = true;

    GemmW4Params p;
    p.M = static_cast<int>(M_total); p.N = static_cast<int>(N); p.K = static_cast<int>(K);
    p.m_tiles = grp.n; p.n_tiles = pl.n_tiles; p.kstages = pl.kstages; p.sf_kgroups = pl.sf_kgroups;
    p.sfa1 = ws + pl.off_sfa1; p.sfa2 = ws + pl.off_sfa2; p.sfb = sfb;
    p.y = y; p.ytype = ytype; p.status = status;
    p.a_rows = a_rows; p.nstages = nstages;
    p.ksplit = 1; p.kper = pl.kstages; p.part_rows = 0;
    p.n_fastest = 1;              // the CTAs of a wave share a group's components; every expert's weights are read once
    {
    }
    const long long tiles = static_cast<long long>(grp.n) * pl.n_tiles;
    const int grid = static_cast<int>(tiles < sm_count() ? tiles : sm_count());
    const cudaError_t le = pl.tile_n == 256
        ? launch_pdl(gemm_w4a16_kernel<256, true>, dim3(grid), dim3(kW4ThreadsSf), smem_bytes, s, pdl, tmap_a1, tmap_a2, tmap_b, tmap_y, p, grp)
        : launch_pdl(gemm_w4a16_kernel<224, true>, dim3(grid), dim3(kW4ThreadsSf), smem_bytes, s, pdl, tmap_a1, tmap_a2, tmap_b, tmap_y, p, grp);
    if (le != cudaSuccess) return MSD_ERR_CUDA;
  }
  return MSD_OK;
}

}  // namespace msd

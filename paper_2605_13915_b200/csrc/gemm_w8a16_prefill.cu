// W8A16 MSD linear layer for many activation rows (prefill; Alg. 1 with the two passes kept as two INT32 accumulators):
//   y[i,n] = w_scale[n] * (alpha_i * sum_k q1[i,k] w[n,k] + beta_i * sum_k q2[i,k] w[n,k]).
// The decode kernel puts the weight rows on the MMA M axis and streams the weights once; here the tokens are many, so
// they sit on the M axis in tiles of 128, a tile of 256 weight rows is the N operand, and both components of the token
// tile are multiplied against the same weight tile in shared memory (tcgen05.mma kind::i8, S8 x S8 -> S32):
// accumulator D1 in TMEM columns [0,256), D2 in [256,512).  K stages of 128 elements (one 128-byte swizzle row per
// operand row): 16 + 16 + 32 KB, three stages.
//
// Persistent CTAs, 18 warps: 0 producer (TMA), 1 MMA issuer + TMEM owner, 2..17 epilogue (warp w reads TMEM lanes
// 32 (w % 4) .., columns 64 ((w - 2) / 4) .. of both accumulators, combines them with alpha_i, beta_i and w_scale[n]
// and writes them through a swizzled staging buffer with TMA stores).  The 512 TMEM columns hold one tile, so the
// epilogue of a tile does not overlap the MMAs of the next; sixteen warps keep it short.
//
// kPair: two CTAs of a cluster work on 256 tokens x 256 weight rows with tcgen05.mma.cta_group::2.  Each CTA loads its
// own 128 token rows of both components and half of the weight tile (48 instead of 64 KB per stage, four stages),
// all loads complete on the leader's barrier, the leader issues the MMAs and its commits reach both CTAs, each CTA's
// epilogue drains its own 128 accumulator rows and tells the leader.  Barrier operations between the CTAs use the
// default (CTA-scope) semantics: what is handed over is tensor memory, ordered by the tcgen05 fences.
#include <cuda_bf16.h>

#include <cstdlib>

#include "host_common.h"
#include "sm100.cuh"

namespace msd {

constexpr int kP8TileM = 128;
constexpr int kP8TileN = 256;
constexpr int kP8BlockK = 128;                                  // elements (= bytes) per stage and operand row
constexpr int kP8Threads = 576;                                 // producer, MMA, sixteen epilogue warps
constexpr int kP8ABytes = kP8TileM * kP8BlockK;                 // 16 KB
constexpr int kP8BBytes = kP8TileN * kP8BlockK;                 // 32 KB
constexpr int kP8StageBytes = 2 * kP8ABytes + kP8BBytes;        // 64 KB
constexpr int kP8Stages = 3;
constexpr int kP8PairStageBytes = 2 * kP8ABytes + kP8BBytes / 2;    // 48 KB per CTA of a pair
constexpr int kP8PairStages = 4;
constexpr int kP8StoreBytes = 2048;                             // one epilogue chunk: 32 rows x 64 bytes
constexpr int kP8TmemCols = 512;

struct GemmP8Params {
  int M, N, K;
  int m_tiles, n_tiles, kstages;
  int ksplit, kper;             // K splits per output tile and K stages per split (1, kstages: no split)
  int part_rows;                // ksplit > 1: rows per split of the FP32 partial-result buffer the tiles are written to
  int n_fastest;                // tile index -> (token tile, weight tile): weight tile fastest (1) or token tile fastest (0)
  const float* alpha;           // [M]
  const float* beta;            // [M]
  const float* w_scale;         // [N]
  int32_t* acc_dbg;             // nullable [2, M, N]
  int ytype;
  unsigned* status;
};

// kBase: the comparison path the method replaces (Sec. 3.1, first equation) on the same pipeline: tmap_a1 describes
// the BF16 activations and tmap_b the weights a preceding kernel dequantized to BF16 (both as byte matrices, a stage is
// 64 elements), one BF16 x BF16 -> FP32 accumulator, no second component and no scales in the epilogue.
template <bool kPair, bool kBase = false>
__global__ void __launch_bounds__(kP8Threads, 1)
gemm_w8a16_prefill_kernel(const __grid_constant__ CUtensorMap tmap_a1, const __grid_constant__ CUtensorMap tmap_a2,
                          const __grid_constant__ CUtensorMap tmap_b, const __grid_constant__ CUtensorMap tmap_y,
                          const GemmP8Params p) {
  constexpr int kStages = kPair ? kP8PairStages : kP8Stages;
  constexpr int kStageBytes = kPair ? kP8PairStageBytes : kP8StageBytes;
  extern __shared__ uint8_t smem_dyn[];
  __shared__ __align__(8) uint64_t full_bar[kStages], empty_bar[kStages], tfull_bar, tempty_bar;
  __shared__ uint32_t tmem_base_slot;
  __shared__ int abort_flag;

  const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
  const uint32_t rank = kPair ? cluster_ctarank() : 0u;     // 0 = leader of the pair
  uint8_t* smem = reinterpret_cast<uint8_t*>((reinterpret_cast<uintptr_t>(smem_dyn) + 1023) & ~static_cast<uintptr_t>(1023));

  if (threadIdx.x == 0) {
    for (int s = 0; s < kStages; ++s) { mbar_init(&full_bar[s], 1); mbar_init(&empty_bar[s], 1); }
    mbar_init(&tfull_bar, 1);
    mbar_init(&tempty_bar, kPair ? 32 : 16);      // a pair: the epilogue warps of both CTAs arrive on the leader's
    abort_flag = 0;
    mbar_init_fence();
    tma_prefetch_desc(&tmap_a1);
    if (!kBase) tma_prefetch_desc(&tmap_a2);
    tma_prefetch_desc(&tmap_b);
    tma_prefetch_desc(&tmap_y);
  }
  if (warp == 1) {
    if (kPair) tmem_alloc_pair(&tmem_base_slot, kP8TmemCols); else tmem_alloc(&tmem_base_slot, kP8TmemCols);
  }
  tc_fence_before();
  if (kPair) {               // both CTAs' barriers exist before either signals the other's
    cluster_arrive_all();
    cluster_wait_all();
  } else {
    __syncthreads();
  }
  tc_fence_after();
  const uint32_t tmem_base = tmem_base_slot;
  volatile int* abort = &abort_flag;
  // Work items: (token tile, weight tile, K split).  With ksplit > 1 (few output tiles, long K) an item covers kper K
  // stages and writes s_W (alpha D1 + beta D2) of its K range in FP32 to the partial buffer; a second kernel adds the
  // splits in a fixed order.
  // A pair takes two token tiles at once (no K split there); its CTAs stride over the pair tiles together.
  const int m_units = kPair ? (p.m_tiles + 1) >> 1 : p.m_tiles;
  const int total_tiles = m_units * p.n_tiles * p.ksplit;
  const int first = kPair ? blockIdx.x >> 1 : blockIdx.x, step = kPair ? gridDim.x >> 1 : gridDim.x;
  auto tile_of = [&](int tile_mn, int& mt, int& nt) {
    const int mu = p.n_fastest ? tile_mn / p.n_tiles : tile_mn % m_units;
    nt = p.n_fastest ? tile_mn % p.n_tiles : tile_mn / m_units;
    mt = kPair ? 2 * mu + static_cast<int>(rank) : mu;
  };

  if (warp == 0) {
    if (lane == 0) {
      pdl_wait_primary();           // the components and their scales come from the kernel launched just before
      int stage = 0; uint32_t phase = 0;
      bool ok = true;
      for (int tile = first; tile < total_tiles && ok; tile += step) {
        const int split = tile % p.ksplit, tile_mn = tile / p.ksplit;
        int mt, nt;
        tile_of(tile_mn, mt, nt);
        const int ks0 = split * p.kper, ks1 = ks0 + p.kper < p.kstages ? ks0 + p.kper : p.kstages;
        for (int ks = ks0; ks < ks1; ++ks) {
          ok = wait_bounded(&empty_bar[stage], phase ^ 1, abort, p.status);
          if (!ok) break;
          uint8_t* dst = smem + stage * kStageBytes;
          if (kPair) {
            // the leader's barrier counts the bytes of both CTAs; tmap_b's box is this CTA's half of the weight tile
            if (rank == 0) mbar_arrive_expect_tx(&full_bar[stage], 2 * (kStageBytes - (kBase ? kP8ABytes : 0)));
            const uint32_t bar = mapa_shared(smem_u32(&full_bar[stage]), 0);
            tma_load_2d_pair(dst, &tmap_a1, ks * kP8BlockK, mt * kP8TileM, bar);
            if (!kBase) tma_load_2d_pair(dst + kP8ABytes, &tmap_a2, ks * kP8BlockK, mt * kP8TileM, bar);
            tma_load_2d_pair(dst + 2 * kP8ABytes, &tmap_b, ks * kP8BlockK, nt * kP8TileN + static_cast<int>(rank) * (kP8TileN / 2), bar);
          } else {
            mbar_arrive_expect_tx(&full_bar[stage], kStageBytes - (kBase ? kP8ABytes : 0));
            tma_load_2d(dst, &tmap_a1, ks * kP8BlockK, mt * kP8TileM, &full_bar[stage]);
            if (!kBase) tma_load_2d(dst + kP8ABytes, &tmap_a2, ks * kP8BlockK, mt * kP8TileM, &full_bar[stage]);
            tma_load_2d(dst + 2 * kP8ABytes, &tmap_b, ks * kP8BlockK, nt * kP8TileN, &full_bar[stage]);
          }
          if (++stage == kStages) { stage = 0; phase ^= 1; }
        }
      }
    }
  } else if (warp == 1) {
    if (lane == 0 && rank == 0) {
      int stage = 0; uint32_t phase = 0;
      int it = 0;
      bool ok = true;
      const uint64_t op_desc = smem_desc(0, 16, 1024, kSwizzle128B);    // 128-byte-swizzled K-major operand tile
      const uint32_t idesc = kBase ? idesc_dense(/*D=F32*/ 1, /*A=BF16*/ 1, /*B=BF16*/ 1, 0, 0, kPair ? 2 * kP8TileM : kP8TileM, kP8TileN)
                                   : idesc_dense(/*D=S32*/ 2, /*A=S8*/ 1, /*B=S8*/ 1, 0, 0, kPair ? 2 * kP8TileM : kP8TileM, kP8TileN);
      for (int tile = first; tile < total_tiles && ok; tile += step, ++it) {
        ok = wait_bounded(&tempty_bar, (it & 1) ^ 1, abort, p.status);        // the epilogue has drained both accumulators
        if (!ok) break;
        tc_fence_after();
        const int ks0 = (tile % p.ksplit) * p.kper, ks1 = ks0 + p.kper < p.kstages ? ks0 + p.kper : p.kstages;
        for (int ks = ks0; ks < ks1; ++ks) {
          ok = wait_bounded(&full_bar[stage], phase, abort, p.status);
          if (!ok) break;
          tc_fence_after();
          const uint64_t enc = static_cast<uint64_t>(smem_u32(smem + stage * kStageBytes) >> 4);
          const uint64_t a1d = op_desc + enc, a2d = a1d + (kP8ABytes >> 4), bd = a1d + (2 * kP8ABytes >> 4);
#pragma unroll
          for (int kk = 0; kk < 4; ++kk) {                    // 32 elements (32 bytes) per MMA
            const uint32_t acc = (ks > ks0 || kk > 0) ? 1u : 0u;
            if constexpr (kBase) {              // 16 BF16 elements (32 bytes) per MMA
              if (kPair) mma_f16_pair(tmem_base, a1d + 2 * kk, bd + 2 * kk, idesc, acc);
              else mma_f16(tmem_base, a1d + 2 * kk, bd + 2 * kk, idesc, acc);
            } else if (kPair) {
              mma_i8_pair(tmem_base, a1d + 2 * kk, bd + 2 * kk, idesc, acc);
              mma_i8_pair(tmem_base + kP8TileN, a2d + 2 * kk, bd + 2 * kk, idesc, acc);
            } else {
              mma_i8(tmem_base, a1d + 2 * kk, bd + 2 * kk, idesc, acc);
              mma_i8(tmem_base + kP8TileN, a2d + 2 * kk, bd + 2 * kk, idesc, acc);
            }
          }
          if (kPair) tc_commit_pair(&empty_bar[stage], 3); else tc_commit(&empty_bar[stage]);    // frees the stage (in both CTAs)
          if (++stage == kStages) { stage = 0; phase ^= 1; }
        }
        if (!ok) break;
        if (kPair) tc_commit_pair(&tfull_bar, 3); else tc_commit(&tfull_bar);
      }
    }
  } else {
    // Epilogue (a5), sixteen warps: warp w reads TMEM lanes 32 (w % 4) .. and the 64 columns 64 ((w - 2) / 4) .. of both
    // accumulators, 16 columns at a time (a TMEM load takes several hundred cycles and a thread cannot wait for one
    // load while another is in flight, so the latency is hidden across warps: four per scheduler).  Results are staged
    // in chunks of 64 bytes per row (32 BF16 or 16 FP32 columns) in the 64-byte-swizzled layout of the output tensor
    // map and written by a TMA store; rows past M and columns past N are clipped by the store.
    const int quad = warp & 3, part = (warp - 2) >> 2;
    uint8_t* sb = smem + kStages * kStageBytes + (warp - 2) * kP8StoreBytes;
    const uint32_t leader_tempty = kPair ? mapa_shared(smem_u32(&tempty_bar), 0) : 0u;
    auto release_acc = [&]() {                      // all that is needed of the accumulators is in registers
      tc_fence_before();
      __syncwarp();
      if (lane == 0) {
        if (kPair) mbar_arrive_remote(leader_tempty); else mbar_arrive(&tempty_bar);
      }
    };
    const int ccols = (p.ytype == MSD_OUT_BF16) ? 32 : 16;
    const uint32_t swz = static_cast<uint32_t>((lane >> 1) & 3);
    int it = 0;
    bool ok = true;
    pdl_wait_primary();             // alpha and beta come from the decomposition kernel launched just before
    // Column scales: every lane needs the same scales of a chunk.  Lane l loads the scale of the chunk's l-th column
    // one chunk ahead and the lanes fetch them from one another by shuffles.
    for (int tile = first; tile < total_tiles && ok; tile += step, ++it) {
      const int split = tile % p.ksplit, tile_mn = tile / p.ksplit;
      int mt, nt;
      tile_of(tile_mn, mt, nt);
      const int row0 = mt * kP8TileM + quad * 32, row = row0 + lane;
      float a_i = 0.0f, b_i = 0.0f;
      if constexpr (!kBase) {
        if (row < p.M) { a_i = __ldg(p.alpha + row); b_i = __ldg(p.beta + row); }
      }
      const int col_base = nt * kP8TileN + part * 64;
      const int col_w = col_base + lane;
      float sw_next = (!kBase && lane < ccols && col_w < p.N) ? __ldg(p.w_scale + col_w) : 0.0f;
      ok = wait_bounded(&tfull_bar, it & 1, abort, p.status);
      if (!ok) break;
      tc_fence_after();
      const uint32_t trow = tmem_base + (static_cast<uint32_t>(quad * 32) << 16) + part * 64;
      // this warp's columns of the tile that lie inside the matrix; chunks beyond them are skipped altogether
      const int cols_here = p.N - col_base < 64 ? p.N - col_base : 64;
      const int cend = row0 < p.M ? (cols_here > 0 ? cols_here : 0) : 0;
      if (cend == 0) release_acc();
      for (int c0 = 0; c0 < cend; c0 += ccols) {
        uint32_t o[16];
        const int col = col_base + c0;
        const float sw_cur = sw_next;
        sw_next = (!kBase && lane < ccols && c0 + ccols < cend && col_w + c0 + ccols < p.N) ? __ldg(p.w_scale + col_w + c0 + ccols) : 0.0f;
#pragma unroll
        for (int hsub = 0; hsub < 2; ++hsub) {       // 16 accumulator columns per load
          if (hsub == 1 && p.ytype != MSD_OUT_BF16) break;
          uint32_t v1[16], v2[16];
          tmem_ld16(trow + c0 + 16 * hsub, v1);
          if constexpr (!kBase) tmem_ld16(trow + kP8TileN + c0 + 16 * hsub, v2);
          tmem_ld_wait();
          if constexpr (kBase) {
            // the FP32 sums as they are, rounded once to the output type
            if (p.ytype == MSD_OUT_BF16) {
#pragma unroll
              for (int j = 0; j < 8; ++j) {
                const __nv_bfloat162 h = __floats2bfloat162_rn(__uint_as_float(v1[2 * j]), __uint_as_float(v1[2 * j + 1]));
                o[8 * hsub + j] = *reinterpret_cast<const uint32_t*>(&h);
              }
            } else {
#pragma unroll
              for (int j = 0; j < 16; ++j) o[j] = v1[j];
            }
            continue;
          }
          if (p.acc_dbg && row < p.M) {
            for (int j = 0; j < 16 && col + 16 * hsub + j < p.N; ++j) {
              p.acc_dbg[static_cast<long long>(row) * p.N + col + 16 * hsub + j] = static_cast<int32_t>(v1[j]);
              p.acc_dbg[(static_cast<long long>(p.M) + row) * p.N + col + 16 * hsub + j] = static_cast<int32_t>(v2[j]);
            }
          }
          if (p.ytype == MSD_OUT_BF16) {
#pragma unroll
            for (int j = 0; j < 4; ++j) {
              const int cj = 16 * hsub + 4 * j;
              const float sx = __shfl_sync(0xffffffffu, sw_cur, cj), sy = __shfl_sync(0xffffffffu, sw_cur, cj + 1);
              const float sz = __shfl_sync(0xffffffffu, sw_cur, cj + 2), sw_ = __shfl_sync(0xffffffffu, sw_cur, cj + 3);
              const float y0 = sx * __fmaf_rn(a_i, static_cast<float>(static_cast<int32_t>(v1[4 * j])), b_i * static_cast<float>(static_cast<int32_t>(v2[4 * j])));
              const float y1 = sy * __fmaf_rn(a_i, static_cast<float>(static_cast<int32_t>(v1[4 * j + 1])), b_i * static_cast<float>(static_cast<int32_t>(v2[4 * j + 1])));
              const float y2 = sz * __fmaf_rn(a_i, static_cast<float>(static_cast<int32_t>(v1[4 * j + 2])), b_i * static_cast<float>(static_cast<int32_t>(v2[4 * j + 2])));
              const float y3 = sw_ * __fmaf_rn(a_i, static_cast<float>(static_cast<int32_t>(v1[4 * j + 3])), b_i * static_cast<float>(static_cast<int32_t>(v2[4 * j + 3])));
              const __nv_bfloat162 h0 = __floats2bfloat162_rn(y0, y1), h1 = __floats2bfloat162_rn(y2, y3);
              o[8 * hsub + 2 * j] = *reinterpret_cast<const uint32_t*>(&h0);
              o[8 * hsub + 2 * j + 1] = *reinterpret_cast<const uint32_t*>(&h1);
            }
          } else {
#pragma unroll
            for (int j = 0; j < 4; ++j) {
              const float sx = __shfl_sync(0xffffffffu, sw_cur, 4 * j), sy = __shfl_sync(0xffffffffu, sw_cur, 4 * j + 1);
              const float sz = __shfl_sync(0xffffffffu, sw_cur, 4 * j + 2), sw_ = __shfl_sync(0xffffffffu, sw_cur, 4 * j + 3);
              o[4 * j] = __float_as_uint(sx * __fmaf_rn(a_i, static_cast<float>(static_cast<int32_t>(v1[4 * j])), b_i * static_cast<float>(static_cast<int32_t>(v2[4 * j]))));
              o[4 * j + 1] = __float_as_uint(sy * __fmaf_rn(a_i, static_cast<float>(static_cast<int32_t>(v1[4 * j + 1])), b_i * static_cast<float>(static_cast<int32_t>(v2[4 * j + 1]))));
              o[4 * j + 2] = __float_as_uint(sz * __fmaf_rn(a_i, static_cast<float>(static_cast<int32_t>(v1[4 * j + 2])), b_i * static_cast<float>(static_cast<int32_t>(v2[4 * j + 2]))));
              o[4 * j + 3] = __float_as_uint(sw_ * __fmaf_rn(a_i, static_cast<float>(static_cast<int32_t>(v1[4 * j + 3])), b_i * static_cast<float>(static_cast<int32_t>(v2[4 * j + 3]))));
            }
          }
        }
        if (c0 + ccols >= cend) release_acc();
        if (lane == 0) bulk_wait_group_read<0>();    // the store of the previous chunk is done with the staging buffer
        __syncwarp();
        uint8_t* srow = sb + lane * 64;
#pragma unroll
        for (int j = 0; j < 4; ++j)
          *reinterpret_cast<uint4*>(srow + ((static_cast<uint32_t>(j) ^ swz) << 4)) = make_uint4(o[4 * j], o[4 * j + 1], o[4 * j + 2], o[4 * j + 3]);
        fence_proxy_async_smem();
        __syncwarp();
        if (lane == 0) {
          tma_store_2d(&tmap_y, col, row0 + split * p.part_rows, sb);
          bulk_commit_group();
        }
      }
    }
    if (lane == 0) bulk_wait_group<0>();            // every store has been written before the CTA goes away
  }

  tc_fence_before();
  __syncthreads();
  if (kPair) {       // neither CTA leaves while the other may still signal its barriers or read its shared memory
    cluster_arrive_all();
    cluster_wait_all();
  }
  if (warp == 1) {
    tc_fence_after();
    if (kPair) tmem_dealloc_pair(tmem_base, kP8TmemCols); else tmem_dealloc(tmem_base, kP8TmemCols);
  }
}

struct GemmP8Plan {
  int m_tiles, n_tiles, kstages, grid, ksplit, kper;
  size_t off_q1, off_q2, off_alpha, off_beta, off_part, bytes;
};

// base: the dequantize-to-BF16 comparison path (K counted in bytes of BF16; off_q1 holds the BF16 weights)
static GemmP8Plan plan_p8(int64_t M, int64_t N, int64_t K, bool base = false) {
  GemmP8Plan pl;
  pl.m_tiles = static_cast<int>((M + kP8TileM - 1) / kP8TileM);
  pl.n_tiles = static_cast<int>((N + kP8TileN - 1) / kP8TileN);
  pl.kstages = static_cast<int>(((base ? 2 * K : K) + kP8BlockK - 1) / kP8BlockK);
  const long long tiles = static_cast<long long>(pl.m_tiles) * pl.n_tiles;
  // Few output tiles and a long K (a few hundred rows on a narrow layer): split K so that there is about one work item
  // per SM, each at least eight stages long; the FP32 partial results are added by a second kernel.
  pl.ksplit = 1;
  pl.kper = pl.kstages;
  {
    const int forced = option(OPT_P8_KSPLIT);     // testing aid
    long long want = forced >= 0 ? forced : (2 * tiles <= sm_count() ? sm_count() / tiles : 1);
    if (want > pl.kstages / 8) want = pl.kstages / 8;
    if (want > 1) {
      pl.kper = static_cast<int>((pl.kstages + want - 1) / want);
      pl.ksplit = (pl.kstages + pl.kper - 1) / pl.kper;
    }
  }
  const long long items = tiles * pl.ksplit;
  pl.grid = static_cast<int>(items < sm_count() ? items : sm_count());
  size_t off = 0;
  pl.off_q1 = off;    off = round_up(off + (base ? static_cast<size_t>(N) * K * 2 : static_cast<size_t>(M) * K), 1024);
  pl.off_q2 = off;    off = round_up(off + (base ? 0 : static_cast<size_t>(M) * K), 1024);
  pl.off_alpha = off; off = round_up(off + static_cast<size_t>(M) * sizeof(float), 1024);
  pl.off_beta = off;  off = round_up(off + static_cast<size_t>(M) * sizeof(float), 1024);
  pl.off_part = off;
  if (pl.ksplit > 1) off = round_up(off + static_cast<size_t>(pl.ksplit) * pl.m_tiles * kP8TileM * N * sizeof(float), 1024);
  pl.bytes = off;
  return pl;
}

size_t w8_prefill_workspace_bytes(int64_t M, int64_t N, int64_t K) { return plan_p8(M, N, K).bytes; }
size_t w8_prefill_base_workspace_bytes(int64_t M, int64_t N, int64_t K) { return plan_p8(M, N, K, true).bytes; }

static msd_status_t p8_launch(bool base, const void* x_bf16, const int8_t* w, const float* w_scale, int64_t M, int64_t N, int64_t K,
                              void* y, int ytype, int32_t* acc_dbg, float c1, float c2, void* workspace, size_t workspace_bytes,
                              cudaStream_t s);

// Arguments already checked by the caller (msd_gemm_w8a16_ex); M > 128.
msd_status_t w8_prefill_launch(const void* x_bf16, const int8_t* w, const float* w_scale, int64_t M, int64_t N, int64_t K,
                               void* y, int ytype, int32_t* acc_dbg, float c1, float c2, void* workspace,
                               size_t workspace_bytes, cudaStream_t s) {
  return p8_launch(false, x_bf16, w, w_scale, M, N, K, y, ytype, acc_dbg, c1, c2, workspace, workspace_bytes, s);
}
// The comparison path for M > 128 (msd_gemm_dequant_bf16): weights dequantized to BF16 in the workspace, then the same
// pipeline as a BF16 GEMM with FP32 accumulation.
msd_status_t w8_prefill_base_launch(const void* x_bf16, const int8_t* w, const float* w_scale, int64_t M, int64_t N, int64_t K,
                                    void* y, int ytype, void* workspace, size_t workspace_bytes, cudaStream_t s) {
  return p8_launch(true, x_bf16, w, w_scale, M, N, K, y, ytype, nullptr, 0.0f, 0.0f, workspace, workspace_bytes, s);
}

static msd_status_t p8_launch(bool base, const void* x_bf16, const int8_t* w, const float* w_scale, int64_t M, int64_t N, int64_t K,
                              void* y, int ytype, int32_t* acc_dbg, float c1, float c2, void* workspace, size_t workspace_bytes,
                              cudaStream_t s) {
  if (static_cast<long long>((M + kP8TileM - 1) / kP8TileM) * ((N + kP8TileN - 1) / kP8TileN) > 0x7FFFFFFFLL) return MSD_ERR_BAD_SHAPE;
  const GemmP8Plan pl = plan_p8(M, N, K, base);
  if (workspace_bytes < pl.bytes) return MSD_ERR_WORKSPACE_TOO_SMALL;
  unsigned* status = device_status_ptr();
  if (!status) return MSD_ERR_CUDA;
  uint8_t* ws = static_cast<uint8_t*>(workspace);
  int8_t* q1 = reinterpret_cast<int8_t*>(ws + pl.off_q1);
  int8_t* q2 = reinterpret_cast<int8_t*>(ws + pl.off_q2);
  float* alpha = reinterpret_cast<float*>(ws + pl.off_alpha);
  float* beta = reinterpret_cast<float*>(ws + pl.off_beta);
  msd_status_t st = MSD_OK;
  if (base) st = launch_dequant_w8_to_bf16(w, w_scale, N, K, q1, s);
  else st = launch_decompose_int8(x_bf16, M, K, K, q1, q2, alpha, beta, c1, c2, s);
  if (st != MSD_OK) return st;
  // operand matrices as bytes: [M, kb] activations (components, or the BF16 x itself) and [N, kb] weights
  const uint64_t kb = static_cast<uint64_t>(base ? 2 * K : K);
  const void* a1_ptr = base ? x_bf16 : static_cast<const void*>(q1);
  const void* b_ptr = base ? static_cast<const void*>(q1) : static_cast<const void*>(w);

  // with a K split (not when the INT32 accumulators are asked for: they exist only unsplit) the kernel writes FP32
  // partial results, split s at rows s * part_rows ..., and the reduce kernel produces y
  const bool split = pl.ksplit > 1 && acc_dbg == nullptr;
  const int ksplit = split ? pl.ksplit : 1, kper = split ? pl.kper : pl.kstages;
  float* part = reinterpret_cast<float*>(ws + pl.off_part);
  const uint64_t part_rows = static_cast<uint64_t>(pl.m_tiles) * kP8TileM;
  CUtensorMap tmap_a1, tmap_a2, tmap_b, tmap_y;
  const bool ybf = !split && ytype == MSD_OUT_BF16;
  // CTA pairs (256 tokens x 256 weight rows per pair, half of the weight tile loaded by each CTA) where there is no K
  // split (the option MSD_P8_PAIR forces the choice).
  bool use_pair = false;
  {
    const int forced = option(OPT_P8_PAIR);       // testing aid
    const bool can = pl.ksplit == 1 && pl.m_tiles >= 2;
    // where the pair tiles need no more rounds on half as many units (an odd number of token tiles leaves a CTA idle)
    const long long tiles = static_cast<long long>(pl.m_tiles) * pl.n_tiles, pair_tiles = static_cast<long long>((pl.m_tiles + 1) / 2) * pl.n_tiles;
    const long long clusters = sm_count() / 2;
    const bool want = (pair_tiles + clusters - 1) / clusters <= (tiles + sm_count() - 1) / sm_count();
    use_pair = can && (forced >= 0 ? forced != 0 : want);
  }
  if (!encode_tmap_2d(&tmap_a1, CU_TENSOR_MAP_DATA_TYPE_UINT8, a1_ptr, kb, M, kb, kP8BlockK, kP8TileM, CU_TENSOR_MAP_SWIZZLE_128B) ||
      !encode_tmap_2d(&tmap_a2, CU_TENSOR_MAP_DATA_TYPE_UINT8, base ? a1_ptr : static_cast<const void*>(q2), kb, M, kb, kP8BlockK, kP8TileM, CU_TENSOR_MAP_SWIZZLE_128B) ||
      !encode_tmap_2d(&tmap_b, CU_TENSOR_MAP_DATA_TYPE_UINT8, b_ptr, kb, N, kb, kP8BlockK, use_pair ? kP8TileN / 2 : kP8TileN, CU_TENSOR_MAP_SWIZZLE_128B) ||
      !encode_tmap_2d(&tmap_y, ybf ? CU_TENSOR_MAP_DATA_TYPE_BFLOAT16 : CU_TENSOR_MAP_DATA_TYPE_FLOAT32, split ? static_cast<void*>(part) : y,
                      static_cast<uint64_t>(N), split ? part_rows * ksplit : static_cast<uint64_t>(M),
                      static_cast<uint64_t>(N) * (ybf ? 2 : 4), ybf ? 32 : 16, 32, CU_TENSOR_MAP_SWIZZLE_64B))
    return MSD_ERR_CUDA;

  GemmP8Params p;
  p.M = static_cast<int>(M); p.N = static_cast<int>(N); p.K = static_cast<int>(K);
  p.m_tiles = pl.m_tiles; p.n_tiles = pl.n_tiles; p.kstages = pl.kstages;
  p.alpha = alpha; p.beta = beta; p.w_scale = w_scale; p.acc_dbg = acc_dbg; p.ytype = split ? MSD_OUT_FP32 : ytype; p.status = status;
  p.ksplit = ksplit; p.kper = kper; p.part_rows = static_cast<int>(part_rows);
  {
    // A wave of CTAs either shares a few weight tiles and sweeps the token tiles (token tile fastest) or the other way
    // round; the operand that is swept should be the one that stays in L2 (40 MB assumed usable for it).
    const double l2 = 40.0 * 1024 * 1024, a_bytes = 2.0 * static_cast<double>(M) * K, w_bytes = (base ? 2.0 : 1.0) * static_cast<double>(N) * K;
    const bool n_fast = a_bytes <= l2 ? false : (w_bytes <= l2 ? true : a_bytes > w_bytes);
    p.n_fastest = n_fast;
  }
  const size_t smem_bytes = static_cast<size_t>(kP8Stages) * kP8StageBytes + 16 * kP8StoreBytes + 1024;
  const size_t smem_pair = static_cast<size_t>(kP8PairStages) * kP8PairStageBytes + 16 * kP8StoreBytes + 1024;
  static bool attr_done = false;
  if (!attr_done) {
    if (cudaFuncSetAttribute(gemm_w8a16_prefill_kernel<false>, cudaFuncAttributeMaxDynamicSharedMemorySize, static_cast<int>(smem_bytes)) != cudaSuccess ||
        cudaFuncSetAttribute(gemm_w8a16_prefill_kernel<true>, cudaFuncAttributeMaxDynamicSharedMemorySize, static_cast<int>(smem_pair)) != cudaSuccess ||
        cudaFuncSetAttribute(gemm_w8a16_prefill_kernel<false, true>, cudaFuncAttributeMaxDynamicSharedMemorySize, static_cast<int>(smem_bytes)) != cudaSuccess ||
        cudaFuncSetAttribute(gemm_w8a16_prefill_kernel<true, true>, cudaFuncAttributeMaxDynamicSharedMemorySize, static_cast<int>(smem_pair)) != cudaSuccess)
      return MSD_ERR_CUDA;
    attr_done = true;
  }
  const bool pdl = option(OPT_NO_PDL) <= 0;
  if (use_pair) {
    const long long pair_tiles = static_cast<long long>((pl.m_tiles + 1) / 2) * pl.n_tiles;
    const int clusters = static_cast<int>(pair_tiles < sm_count() / 2 ? pair_tiles : sm_count() / 2);
    const cudaError_t pe = base
        ? launch_pdl_cluster(gemm_w8a16_prefill_kernel<true, true>, dim3(2 * clusters), dim3(kP8Threads), smem_pair, s, pdl, 2u, tmap_a1, tmap_a2, tmap_b, tmap_y, p)
        : launch_pdl_cluster(gemm_w8a16_prefill_kernel<true>, dim3(2 * clusters), dim3(kP8Threads), smem_pair, s, pdl, 2u, tmap_a1, tmap_a2, tmap_b, tmap_y, p);
    if (pe != cudaSuccess) return MSD_ERR_CUDA;
    return MSD_OK;
  }
  const long long items = static_cast<long long>(pl.m_tiles) * pl.n_tiles * ksplit;
  const int grid = static_cast<int>(items < sm_count() ? items : sm_count());
  const cudaError_t le = base
      ? launch_pdl(gemm_w8a16_prefill_kernel<false, true>, dim3(grid), dim3(kP8Threads), smem_bytes, s, pdl, tmap_a1, tmap_a2, tmap_b, tmap_y, p)
      : launch_pdl(gemm_w8a16_prefill_kernel<false>, dim3(grid), dim3(kP8Threads), smem_bytes, s, pdl, tmap_a1, tmap_a2, tmap_b, tmap_y, p);
  if (le != cudaSuccess) return MSD_ERR_CUDA;
  if (split) return launch_ksplit_reduce(part, ksplit, static_cast<int64_t>(part_rows) * N, M, N, y, ytype, s, pdl);
  return MSD_OK;
}

}  // namespace msd

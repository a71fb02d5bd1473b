// W4A16 MSD with the paper-literal components (Sec. 3.2.1, Alg. 2; Tab. mxfp4-evolution, last row): both passes round
// onto the E1M2 grid {0, .25, ..., 1.75} with alpha = 2^ceil(log2(M_b / 1.859375)) and beta = alpha / 16 (error bound
// alpha / 64).  Block-scaled FP4 tensor cores multiply E2M1, not E1M2, but every E1M2 value is an E4M3 number, so the
// components travel as FP8 bytes and the product runs as tcgen05.mma kind::mxf8f6f4 (A = E4M3 components, B = the E2M1
// weights, UE8M0 scale per 32 elements on both) at the FP8 rate.  The packed 4-bit weights are expanded on the fly by
// the TMA engine (tensor-map type 16U4_ALIGN16B: 16 codes in 8 bytes followed by an 8-byte gap, one element per byte
// slot of shared memory, which is the layout this MMA kind reads for 4-bit operands).
//
// Tile 128 activation rows x 256 weight rows, K stages of 128 elements (one 128-byte swizzle row per operand row), both
// passes into the same FP32 accumulator.  Warps as in the E2M1 kernel: 0 operand producer, 1 MMA issuer + TMEM owner,
// 2..5 epilogue (TMA stores through swizzled staging buffers), 6..9 scale warps (shared memory -> TMEM by tcgen05.st),
// 10 scale producer.
#include <cuda_bf16.h>

#include <cstdlib>

#include "host_common.h"
#include "sm100.cuh"

namespace msd {

constexpr int kE1TileM = 128;
constexpr int kE1TileN = 256;
constexpr int kE1BlockK = 128;                                  // elements per stage
constexpr int kE1Threads = 352;
constexpr int kE1ABytes = kE1TileM * 128;                       // 16 KB (one byte per element)
constexpr int kE1BBytes = kE1TileN * 128;                       // 32 KB (one byte slot per 4-bit element)
constexpr int kE1SfBytes = 512 + 512 + 1024;                    // SFA1, SFA2, SFB (two row tiles): 4 scales per row each
constexpr int kE1StageBytes = 2 * kE1ABytes + kE1BBytes + kE1SfBytes;   // 67584 bytes of shared memory
// what the copies of a stage report to the barrier: the unpacking weight copy counts the 8 data bytes of every 16-byte
// slot group it fills (the packed size), not the gaps it leaves
constexpr int kE1StageTxBytes = 2 * kE1ABytes + kE1BBytes / 2 + kE1SfBytes;
constexpr int kE1Stages = 3;
constexpr int kE1TmemCols = 512;
constexpr int kE1SfCol = 256;
constexpr int kE1StoreBytes = 2048;                             // one epilogue chunk: 32 rows x 64 bytes

struct GemmE1Params {
  int M, N, K;
  int m_tiles, n_tiles, kstages;
  int sf_kgroups;               // K / 128
  const uint8_t* sfa1;
  const uint8_t* sfa2;
  const uint8_t* sfb;
  void* y;
  int ytype;
  unsigned* status;
};

// 2^e as an FP32 number for e in [-126, 127]
__device__ __forceinline__ float e1_pow2f(int e) { return __uint_as_float(static_cast<uint32_t>(e + 127) << 23); }

// E4M3 byte of the E1M2 value sign * k / 4, k = 0..7
__device__ __forceinline__ uint32_t e1m2_as_e4m3(int k, uint32_t sign) {
  // 0, .25, .5, .75, 1, 1.25, 1.5, 1.75 in E4M3 (bias 7, 3 mantissa bits)
  const uint64_t table = 0x3E3C3A3834302800ull;
  return static_cast<uint32_t>((table >> (8 * k)) & 0xFF) | (sign << 7);
}

// Alg. 2 on the E1M2 grid: one thread per 32-element block.  Components as E4M3 bytes [M, K]; scales as E8M0 bytes,
// row-major [M, K/32] (sf_kgroups == 0) or in 512-byte blocks of 128 rows x 4 scales.
__global__ void __launch_bounds__(256)
decompose_e1m2_kernel(const uint16_t* __restrict__ x, int64_t ldx, int64_t M, int K, uint8_t* __restrict__ q1,
                      uint8_t* __restrict__ q2, uint8_t* __restrict__ e1, uint8_t* __restrict__ e2, int sf_kgroups,
                      const SfRelayout rl) {
  pdl_launch_dependents();
  if (static_cast<int>(blockIdx.x) < rl.blocks) {          // the first CTAs bring the weight scales into the blocked layout
    __shared__ uint32_t sm_rl[kSfRelayoutSmemWords];
    sf_relayout(rl, blockIdx.x, rl.blocks, sm_rl);
    return;
  }
  const int kblocks = K >> 5;
  const int64_t nblocks = M * kblocks;
  for (int64_t b = static_cast<int64_t>(blockIdx.x - rl.blocks) * 256 + threadIdx.x; b < nblocks;
       b += static_cast<int64_t>(gridDim.x - rl.blocks) * 256) {
    const int64_t row = b / kblocks;
    const int kb = static_cast<int>(b - row * kblocks);
    const uint4* src = reinterpret_cast<const uint4*>(x + row * ldx + kb * 32);
    uint32_t w[16];
#pragma unroll
    for (int i = 0; i < 4; ++i) {
      const uint4 t = __ldg(src + i);
      w[4 * i] = t.x; w[4 * i + 1] = t.y; w[4 * i + 2] = t.z; w[4 * i + 3] = t.w;
    }
    uint32_t mbits = 0;    // maximum of |x| as BF16 bits (monotone in the value for finite inputs)
#pragma unroll
    for (int i = 0; i < 16; ++i) {
      mbits = max(mbits, w[i] & 0x7FFFu);
      mbits = max(mbits, (w[i] >> 16) & 0x7FFFu);
    }
    // alpha = smallest power of two with M_b <= 1.859375 alpha (= 238/128): M_b = (1 + f/128) 2^e -> e + (f > 110)
    const int expf = static_cast<int>(mbits >> 7);
    int a = -123;                                             // beta = alpha/16 must remain an E8M0 code
    if (expf > 0) a = max(-123, (expf - 127) + (((mbits & 0x7Fu) > 110u) ? 1 : 0));
    a = min(a, 127);
    const int bexp = a - 4;
    const int na = -a + 2, nb = -bexp + 2;                    // x / alpha * 4 and r / beta * 4: code index before rounding
    const float sa1 = e1_pow2f(na / 2), sa2 = e1_pow2f(na - na / 2);
    const float sb1 = e1_pow2f(nb / 2), sb2 = e1_pow2f(nb - nb / 2);
    const float alpha4 = e1_pow2f(a - 2);                     // alpha / 4: value of one code step
    uint32_t o1[8], o2[8];
#pragma unroll
    for (int i = 0; i < 8; ++i) { o1[i] = 0; o2[i] = 0; }
#pragma unroll
    for (int i = 0; i < 32; ++i) {
      const float v = (i & 1) ? __uint_as_float(w[i >> 1] & 0xFFFF0000u) : __uint_as_float(w[i >> 1] << 16);
      const float t1 = fminf(rintf(fabsf((v * sa1) * sa2)), 7.0f);          // round-half-to-even on the code, saturating
      const uint32_t s1 = __float_as_uint(v) >> 31;
      const float d1 = copysignf(t1, v) * alpha4;                           // alpha * q1
      const float r = v - d1;                                               // exact: both are multiples of alpha/4 scale units of x
      const float t2 = fminf(rintf(fabsf((r * sb1) * sb2)), 7.0f);
      const uint32_t s2 = __float_as_uint(r) >> 31;
      o1[i >> 2] |= e1m2_as_e4m3(static_cast<int>(t1), s1) << (8 * (i & 3));
      o2[i >> 2] |= e1m2_as_e4m3(static_cast<int>(t2), s2) << (8 * (i & 3));
    }
    uint4* d1p = reinterpret_cast<uint4*>(q1 + row * K + kb * 32);
    uint4* d2p = reinterpret_cast<uint4*>(q2 + row * K + kb * 32);
    d1p[0] = make_uint4(o1[0], o1[1], o1[2], o1[3]); d1p[1] = make_uint4(o1[4], o1[5], o1[6], o1[7]);
    d2p[0] = make_uint4(o2[0], o2[1], o2[2], o2[3]); d2p[1] = make_uint4(o2[4], o2[5], o2[6], o2[7]);
    const int64_t so = sf_kgroups == 0
                           ? row * kblocks + kb
                           : ((row >> 7) * sf_kgroups + (kb >> 2)) * 512 + (row & 31) * 16 + ((row >> 5) & 3) * 4 + (kb & 3);
    e1[so] = static_cast<uint8_t>(a + 127);
    e2[so] = static_cast<uint8_t>(bexp + 127);
  }
}

__device__ __forceinline__ void mma_mxf8f6f4(uint32_t d_tmem, uint64_t a_desc, uint64_t b_desc, uint32_t idesc,
                                             uint32_t sfa_tmem, uint32_t sfb_tmem, uint32_t accumulate) {
  asm volatile(
      "{\n\t.reg .pred p;\n\t"
      "setp.ne.b32 p, %6, 0;\n\t"
      "tcgen05.mma.cta_group::1.kind::mxf8f6f4.block_scale [%0], %1, %2, %3, [%4], [%5], p;\n\t}"
      ::"r"(d_tmem), "l"(a_desc), "l"(b_desc), "r"(idesc), "r"(sfa_tmem), "r"(sfb_tmem), "r"(accumulate)
      : "memory");
}

__global__ void __launch_bounds__(kE1Threads, 1)
gemm_w4a16_e1m2_kernel(const __grid_constant__ CUtensorMap tmap_a1, const __grid_constant__ CUtensorMap tmap_a2,
                       const __grid_constant__ CUtensorMap tmap_b, const __grid_constant__ CUtensorMap tmap_y,
                       const GemmE1Params p) {
  extern __shared__ uint8_t smem_dyn[];
  __shared__ __align__(8) uint64_t full_bar[kE1Stages], empty_bar[kE1Stages], tfull_bar, tempty_bar;
  // the two sets of scale columns in TMEM: written by warps 6..9 (sf_ready), read by the MMAs of a stage (sf_free)
  __shared__ __align__(8) uint64_t sf_ready[2], sf_free[2];
  __shared__ uint32_t tmem_base_slot;
  __shared__ int abort_flag;

  const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
  uint8_t* smem = reinterpret_cast<uint8_t*>((reinterpret_cast<uintptr_t>(smem_dyn) + 1023) & ~static_cast<uintptr_t>(1023));

  if (threadIdx.x == 0) {
    for (int s = 0; s < kE1Stages; ++s) { mbar_init(&full_bar[s], 1); mbar_init(&empty_bar[s], 1); }
    mbar_init(&tfull_bar, 1);
    mbar_init(&tempty_bar, 4);
    for (int a = 0; a < 2; ++a) { mbar_init(&sf_ready[a], 4); mbar_init(&sf_free[a], 1); }
    abort_flag = 0;
    mbar_init_fence();
    tma_prefetch_desc(&tmap_a1);
    tma_prefetch_desc(&tmap_a2);
    tma_prefetch_desc(&tmap_b);
  }
  if (warp == 1) tmem_alloc(&tmem_base_slot, kE1TmemCols);
  tc_fence_before();
  __syncthreads();
  tc_fence_after();
  const uint32_t tmem_base = tmem_base_slot;
  volatile int* abort = &abort_flag;
  const int total_tiles = p.m_tiles * p.n_tiles;

  if (warp == 0 || warp == 10) {
    // two producer threads (a bulk-copy instruction costs its thread 50-100 ns): warp 0 the operand tiles, warp 10 the scales
    if (lane == 0) {
      pdl_wait_primary();
      int stage = 0; uint32_t phase = 0;
      bool ok = true;
      for (int tile = blockIdx.x; tile < total_tiles && ok; tile += gridDim.x) {
        const int mt = tile % p.m_tiles, nt = tile / p.m_tiles;
        for (int ks = 0; ks < p.kstages; ++ks) {
          ok = wait_bounded(&empty_bar[stage], phase ^ 1, abort, p.status);
          if (!ok) break;
          uint8_t* dst = smem + stage * kE1StageBytes;
          if (warp == 0) {
            mbar_arrive_expect_tx(&full_bar[stage], kE1StageTxBytes);
            tma_load_2d(dst, &tmap_a1, ks * kE1BlockK, mt * kE1TileM, &full_bar[stage]);
            tma_load_2d(dst + kE1ABytes, &tmap_a2, ks * kE1BlockK, mt * kE1TileM, &full_bar[stage]);
            tma_load_2d(dst + 2 * kE1ABytes, &tmap_b, ks * kE1BlockK, nt * kE1TileN, &full_bar[stage]);   // coordinates in elements
          } else {
            uint8_t* sf = dst + 2 * kE1ABytes + kE1BBytes;
            const size_t a_off = (static_cast<size_t>(mt) * p.sf_kgroups + ks) * 512;
            bulk_load(sf, p.sfa1 + a_off, 512, &full_bar[stage]);
            bulk_load(sf + 512, p.sfa2 + a_off, 512, &full_bar[stage]);
            bulk_load(sf + 1024, p.sfb + (static_cast<size_t>(2 * nt) * p.sf_kgroups + ks) * 512, 512, &full_bar[stage]);
            bulk_load(sf + 1536, p.sfb + (static_cast<size_t>(2 * nt + 1) * p.sf_kgroups + ks) * 512, 512, &full_bar[stage]);
          }
          if (++stage == kE1Stages) { stage = 0; phase ^= 1; }
        }
      }
    }
  } else if (warp == 1) {
    if (lane == 0) {
      int stage = 0; uint32_t phase = 0;
      int it = 0;
      bool ok = true;
      int nstage = 0;                                                   // stages issued so far (all tiles)
      const uint64_t op_desc = smem_desc(0, 16, 1024, kSwizzle128B);
      for (int tile = blockIdx.x; tile < total_tiles && ok; tile += gridDim.x, ++it) {
        ok = wait_bounded(&tempty_bar, (it & 1) ^ 1, abort, p.status);
        if (!ok) break;
        tc_fence_after();
        for (int ks = 0; ks < p.kstages; ++ks) {
          ok = wait_bounded(&full_bar[stage], phase, abort, p.status);
          if (!ok) break;
          tc_fence_after();
          const uint64_t enc = static_cast<uint64_t>(smem_u32(smem + stage * kE1StageBytes) >> 4);
          const uint64_t a1d = op_desc + enc, a2d = a1d + (kE1ABytes >> 4), bd = a1d + (2 * kE1ABytes >> 4);
          const int set = nstage & 1;
          ok = wait_bounded(&sf_ready[set], (nstage >> 1) & 1, abort, p.status);      // warps 6..9 have written this stage's scales
          if (!ok) break;
          tc_fence_after();
          const uint32_t sfa1_t = tmem_base + kE1SfCol + 16 * set;        // 4 columns: 4 scales (K = 128) per row
          const uint32_t sfa2_t = sfa1_t + 4;
          const uint32_t sfb_t = sfa1_t + 8;                              // 8 columns: 256 weight rows
#pragma unroll
          for (int kk = 0; kk < 4; ++kk) {                    // 32 elements (32 byte slots) per MMA, scale byte kk of the column
            const uint32_t idesc = idesc_block_scaled(/*A: E4M3*/ 0, /*B: E2M1*/ 5, kE1TileM, kE1TileN, kk, kk);
            mma_mxf8f6f4(tmem_base, a1d + 2 * kk, bd + 2 * kk, idesc, sfa1_t, sfb_t, (ks > 0 || kk > 0) ? 1u : 0u);
            mma_mxf8f6f4(tmem_base, a2d + 2 * kk, bd + 2 * kk, idesc, sfa2_t, sfb_t, 1u);
          }
          tc_commit(&sf_free[set]);                  // this set of scale columns may be rewritten once these MMAs are done
          ++nstage;
          tc_commit(&empty_bar[stage]);
          if (++stage == kE1Stages) { stage = 0; phase ^= 1; }
        }
        if (!ok) break;
        tc_commit(&tfull_bar);
      }
    }
  } else if (warp >= 6) {
    // Scale warps: lane l of every 32-lane TMEM quadrant wants bytes 16 l .. 16 l + 15 of each 512-byte scale block as
    // four 32-bit columns; the stage's four blocks (SFA1, SFA2, SFB rows 0-127, SFB rows 128-255) make one set of 16.
    const int quad = warp & 3;
    int stage = 0; uint32_t phase = 0;
    int n = 0;
    bool ok = true;
    for (int tile = blockIdx.x; tile < total_tiles && ok; tile += gridDim.x) {
      for (int ks = 0; ks < p.kstages; ++ks, ++n) {
        const int set = n & 1;
        ok = wait_bounded(&full_bar[stage], phase, abort, p.status);
        if (!ok) break;
        if (n >= 2) {                        // the MMAs that read this set two stages ago are done
          ok = wait_bounded(&sf_free[set], ((n >> 1) - 1) & 1, abort, p.status);
          if (!ok) break;
          tc_fence_after();
        }
        const uint4* sf = reinterpret_cast<const uint4*>(smem + stage * kE1StageBytes + 2 * kE1ABytes + kE1BBytes) + lane;
        uint32_t v[16];
#pragma unroll
        for (int j = 0; j < 4; ++j) {
          const uint4 q = sf[j * 32];
          v[4 * j] = q.x; v[4 * j + 1] = q.y; v[4 * j + 2] = q.z; v[4 * j + 3] = q.w;
        }
        tmem_st16(tmem_base + (static_cast<uint32_t>(quad * 32) << 16) + kE1SfCol + 16 * set, v);
        tmem_st_wait();
        tc_fence_before();
        __syncwarp();
        if (lane == 0) mbar_arrive(&sf_ready[set]);
        if (++stage == kE1Stages) { stage = 0; phase ^= 1; }
      }
    }
  } else {
    // Epilogue: TMEM -> registers -> (BF16) -> this warp's staging buffer (64-byte-swizzled rows of 64 bytes) -> TMA
    // store; two buffers per warp; rows past M and columns past N are clipped by the store.
    const int quad = warp & 3;
    uint8_t* stage_buf = smem + kE1Stages * kE1StageBytes + quad * (2 * kE1StoreBytes);
    const int ccols = (p.ytype == MSD_OUT_BF16) ? 32 : 16;
    const uint32_t swz = static_cast<uint32_t>((lane >> 1) & 3);
    int it = 0, buf = 0;
    bool ok = true;
    for (int tile = blockIdx.x; tile < total_tiles && ok; tile += gridDim.x, ++it) {
      const int mt = tile % p.m_tiles, nt = tile / p.m_tiles;
      ok = wait_bounded(&tfull_bar, it & 1, abort, p.status);
      if (!ok) break;
      tc_fence_after();
      const int row0 = mt * kE1TileM + quad * 32;
      const uint32_t trow = tmem_base + (static_cast<uint32_t>(quad * 32) << 16);
      // chunks beyond the matrix are skipped altogether, so every pass through the loop commits exactly one store group
      const int cols_here = p.N - nt * kE1TileN < kE1TileN ? p.N - nt * kE1TileN : kE1TileN;
      const int cend = row0 < p.M ? cols_here : 0;
      if (cend == 0) {
        tc_fence_before();
        __syncwarp();
        if (lane == 0) mbar_arrive(&tempty_bar);
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
        if (c0 + ccols >= cend) {                   // all that is needed of the accumulator is in registers
          tc_fence_before();
          __syncwarp();
          if (lane == 0) mbar_arrive(&tempty_bar);
        }
        uint8_t* sb = stage_buf + buf * kE1StoreBytes;
        if (lane == 0) bulk_wait_group_read<1>();    // the store that read this buffer two chunks ago is done with it
        __syncwarp();
        uint8_t* srow = sb + lane * 64;
#pragma unroll
        for (int j = 0; j < 4; ++j)
          *reinterpret_cast<uint4*>(srow + ((static_cast<uint32_t>(j) ^ swz) << 4)) = make_uint4(o[4 * j], o[4 * j + 1], o[4 * j + 2], o[4 * j + 3]);
        fence_proxy_async_smem();
        __syncwarp();
        if (lane == 0) {
          tma_store_2d(&tmap_y, nt * kE1TileN + c0, row0, sb);
          bulk_commit_group();
        }
      }
    }
    if (lane == 0) bulk_wait_group<0>();            // every store has been written before the CTA goes away
  }

  tc_fence_before();
  __syncthreads();
  if (warp == 1) {
    tc_fence_after();
    tmem_dealloc(tmem_base, kE1TmemCols);
  }
}

struct GemmE1Plan {
  int m_tiles, n_tiles, kstages, sf_kgroups, grid;
  size_t off_q1, off_q2, off_sfa1, off_sfa2, off_sfb, bytes;
};

static GemmE1Plan plan_e1(int64_t M, int64_t N, int64_t K) {
  GemmE1Plan pl;
  pl.m_tiles = static_cast<int>((M + kE1TileM - 1) / kE1TileM);
  pl.n_tiles = static_cast<int>((N + kE1TileN - 1) / kE1TileN);
  pl.kstages = static_cast<int>(K / kE1BlockK);
  pl.sf_kgroups = pl.kstages;
  const int tiles = pl.m_tiles * pl.n_tiles;
  int grid = sm_count();
  if (grid > tiles) grid = tiles;
  pl.grid = grid;
  size_t off = 0;
  pl.off_q1 = off;   off = round_up(off + static_cast<size_t>(M) * K, 1024);
  pl.off_q2 = off;   off = round_up(off + static_cast<size_t>(M) * K, 1024);
  pl.off_sfa1 = off; off = round_up(off + static_cast<size_t>(pl.m_tiles) * pl.sf_kgroups * 512, 1024);
  pl.off_sfa2 = off; off = round_up(off + static_cast<size_t>(pl.m_tiles) * pl.sf_kgroups * 512, 1024);
  pl.off_sfb = off;  off = round_up(off + static_cast<size_t>(2 * pl.n_tiles) * pl.sf_kgroups * 512, 1024);
  pl.bytes = off;
  return pl;
}

static msd_status_t launch_decompose_e1m2(const void* x_bf16, int64_t M, int64_t K, int64_t ldx, uint8_t* q1, uint8_t* q2,
                                          uint8_t* e1, uint8_t* e2, int sf_kgroups, cudaStream_t stream,
                                          const SfRelayout* relayout = nullptr) {
  if (M == 0) return MSD_OK;
  SfRelayout rl = {};
  if (relayout) {
    rl = *relayout;
    const int64_t rb = static_cast<int64_t>(rl.row_blocks) * ((rl.sf_kgroups + 31) / 32);      // units of 128 rows x 32 K groups
    rl.blocks = static_cast<int>(rb < 4 * sm_count() ? rb : 4 * sm_count());
  }
  const int64_t nblocks = M * (K >> 5);
  const int64_t want = (nblocks + 255) / 256;
  const int64_t cap = static_cast<int64_t>(sm_count()) * 32;
  const unsigned grid = static_cast<unsigned>(want < cap ? want : cap) + static_cast<unsigned>(rl.blocks);
  decompose_e1m2_kernel<<<grid, 256, 0, stream>>>(static_cast<const uint16_t*>(x_bf16), ldx, M, static_cast<int>(K), q1, q2, e1, e2,
                                                  sf_kgroups, rl);
  return launch_status();
}

}  // namespace msd

extern "C" {

msd_status_t msd_decompose_mxfp4_e1m2(const void* x_bf16, int64_t M, int64_t K, int64_t ldx, uint8_t* q1_e4m3, uint8_t* q2_e4m3,
                                      uint8_t* e8m0_1, uint8_t* e8m0_2, void* stream) {
  if (M < 0 || K <= 0 || K % 32 != 0 || ldx < K || ldx % 8 != 0) return MSD_ERR_BAD_SHAPE;
  if (M == 0) return MSD_OK;
  if (!x_bf16 || !q1_e4m3 || !q2_e4m3 || !e8m0_1 || !e8m0_2) return MSD_ERR_NULL_POINTER;
  if (!msd::aligned(x_bf16, 16) || !msd::aligned(q1_e4m3, 16) || !msd::aligned(q2_e4m3, 16)) return MSD_ERR_BAD_ALIGNMENT;
  return msd::launch_decompose_e1m2(x_bf16, M, K, ldx, q1_e4m3, q2_e4m3, e8m0_1, e8m0_2, 0, static_cast<cudaStream_t>(stream));
}

size_t msd_gemm_w4a16_e1m2_workspace_bytes(int64_t M, int64_t N, int64_t K) {
  if (M < 1 || N < 1 || K < 128 || K % 128 != 0) return 0;
  return msd::plan_e1(M, N, K).bytes;
}

msd_status_t msd_gemm_w4a16_e1m2(const void* x_bf16, const uint8_t* w_fp4, const uint8_t* w_e8m0, int64_t M, int64_t N,
                                 int64_t K, void* y, msd_out_t ytype, void* workspace, size_t workspace_bytes, void* stream) {
  using namespace msd;
  if (M < 1 || N < 1 || K < 128 || K % 128 != 0 || N % 8 != 0 || M > (1 << 24) || N > (1 << 24) || K > (1 << 24))
    return MSD_ERR_BAD_SHAPE;
  if (ytype != MSD_OUT_BF16 && ytype != MSD_OUT_FP32) return MSD_ERR_UNSUPPORTED;
  if (!x_bf16 || !w_fp4 || !w_e8m0 || !y || !workspace) return MSD_ERR_NULL_POINTER;
  if (!aligned(x_bf16, 16) || !aligned(w_fp4, 32) || !aligned(w_e8m0, 4) || !aligned(y, 16) || !aligned(workspace, 1024))
    return MSD_ERR_BAD_ALIGNMENT;     // the scale relayout reads the E8M0 rows as 32-bit words
  const GemmE1Plan pl = plan_e1(M, N, K);
  if (workspace_bytes < pl.bytes) return MSD_ERR_WORKSPACE_TOO_SMALL;
  unsigned* status = device_status_ptr();
  if (!status) return MSD_ERR_CUDA;
  cudaStream_t s = static_cast<cudaStream_t>(stream);
  uint8_t* ws = static_cast<uint8_t*>(workspace);
  uint8_t* q1 = ws + pl.off_q1;
  uint8_t* q2 = ws + pl.off_q2;
  // the weight scales go into the blocked layout (two 128-row blocks per 256-row tile) in the decomposition launch
  SfRelayout rl = {};
  rl.src = w_e8m0; rl.dst = ws + pl.off_sfb; rl.rows = N; rl.kblocks = static_cast<int>(K / 32);
  rl.sf_kgroups = pl.sf_kgroups; rl.tile_rows = kE1TileN; rl.row_blocks = 2 * pl.n_tiles;
  msd_status_t st = launch_decompose_e1m2(x_bf16, M, K, K, q1, q2, ws + pl.off_sfa1, ws + pl.off_sfa2, pl.sf_kgroups, s, &rl);
  if (st != MSD_OK) return st;

  CUtensorMap tmap_a1, tmap_a2, tmap_b;
  if (!encode_tmap_2d(&tmap_a1, CU_TENSOR_MAP_DATA_TYPE_UINT8, q1, K, M, K, 128, kE1TileM, CU_TENSOR_MAP_SWIZZLE_128B) ||
      !encode_tmap_2d(&tmap_a2, CU_TENSOR_MAP_DATA_TYPE_UINT8, q2, K, M, K, 128, kE1TileM, CU_TENSOR_MAP_SWIZZLE_128B) ||
      // packed 4-bit codes in memory (K elements = K/2 bytes per row), one byte slot per code in shared memory
      !encode_tmap_2d(&tmap_b, CU_TENSOR_MAP_DATA_TYPE_16U4_ALIGN16B, w_fp4, K, N, K / 2, 128, kE1TileN, CU_TENSOR_MAP_SWIZZLE_128B))
    return MSD_ERR_CUDA;

  GemmE1Params p;
  p.M = static_cast<int>(M); p.N = static_cast<int>(N); p.K = static_cast<int>(K);
  p.m_tiles = pl.m_tiles; p.n_tiles = pl.n_tiles; p.kstages = pl.kstages; p.sf_kgroups = pl.sf_kgroups;
  p.sfa1 = ws + pl.off_sfa1; p.sfa2 = ws + pl.off_sfa2; p.sfb = ws + pl.off_sfb;
  p.y = y; p.ytype = ytype; p.status = status;
  CUtensorMap tmap_y;
  const bool ybf = ytype == MSD_OUT_BF16;
  if (!encode_tmap_2d(&tmap_y, ybf ? CU_TENSOR_MAP_DATA_TYPE_BFLOAT16 : CU_TENSOR_MAP_DATA_TYPE_FLOAT32, y, static_cast<uint64_t>(N),
                      static_cast<uint64_t>(M), static_cast<uint64_t>(N) * (ybf ? 2 : 4), ybf ? 32 : 16, 32, CU_TENSOR_MAP_SWIZZLE_64B))
    return MSD_ERR_CUDA;
  const size_t smem_bytes = static_cast<size_t>(kE1Stages) * kE1StageBytes + 8 * kE1StoreBytes + 1024;
  static bool attr_done = false;
  if (!attr_done) {
    if (cudaFuncSetAttribute(gemm_w4a16_e1m2_kernel, cudaFuncAttributeMaxDynamicSharedMemorySize, static_cast<int>(smem_bytes)) != cudaSuccess)
      return MSD_ERR_CUDA;
    attr_done = true;
  }
  const bool pdl = option(OPT_NO_PDL) <= 0;
  if (launch_pdl(gemm_w4a16_e1m2_kernel, dim3(pl.grid), dim3(kE1Threads), smem_bytes, s, pdl, tmap_a1, tmap_a2, tmap_b, tmap_y, p) != cudaSuccess)
    return MSD_ERR_CUDA;
  return MSD_OK;
}

}  // extern "C"

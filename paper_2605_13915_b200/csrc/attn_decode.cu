// Decode attention over an INT8 KV cache with MSD on Q and on the softmax probabilities (Sec. 4, Alg. 3; tiled
// form Sec. 4.3), split over the context (flash-decoding) and merged with the log-sum-exp rule.
//
// One CTA handles one (sequence, KV head, group of up to HG query heads, context split) and walks its tokens in
// tiles of 128.  Both GEMMs run on tcgen05 with the TOKENS on the MMA M axis / TMEM lanes:
//   S^T[128 tokens x Rp]  = K_tile[128 x D] (K-major, TMA, 128-byte swizzle)  x  Qstack[Rp x D]^T
//   O^T[128 dv x Rp]      = V_tile^T[dv x 128 tokens] (the same TMA layout read as an MN-major operand)  x  Pstack[Rp x 128]^T
// where Rp = 2*HG stacked rows: rows [0,HG) hold the first INT8 component of each head, rows [HG,2HG) the second,
// so one KV tile read from HBM serves both passes.  When v_cache is NULL the V operand aliases the first Dv bytes of
// the K rows already in shared memory (MLA latent cache) and nothing is loaded twice.
//
// Warps: 0 = TMA producer, 1 = MMA issuer + TMEM owner, 2..5 = softmax / merge (thread = token lane for the softmax,
// = dv lane for the merge).  The next tile's QK^T is issued while the current tile's softmax runs (S^T is double
// buffered in TMEM).  Every wait is bounded.
#include <cuda_bf16.h>

#include <algorithm>
#include <cmath>
#include <mutex>
#include <cstdlib>

#include "host_common.h"
#include "quant.cuh"
#include "sm100.cuh"

namespace msd {

constexpr int kTok = 128;           // tokens per tile
constexpr int kAttnThreads = 192;
constexpr int kChunk = 128;         // bytes of D / Dv per TMA box and per shared-memory operand chunk
constexpr int kChunkBytes = kTok * kChunk;
constexpr int kPartHdr = 4;         // words in front of a split's partial output row: reference maximum, sum of P, two unused

struct AttnParams {
  const uint16_t* q;      // [B,Hq,D] BF16 (read by attn_qstack_kernel only)
  // written by attn_qstack_kernel, one entry per (sequence, KV head, head group): the stacked INT8 operand exactly as
  // it lies in shared memory (DC chunks of [Rp x 128] bytes, 128-byte swizzle, unused slots zero) and alpha_Q[HG], beta_Q[HG]
  const uint8_t* q_img;
  const float* q_scales;
  const float* k_scale;   // [T,Hkv]
  const float* v_scale;   // [T,Hkv]
  const int32_t* cu;      // [B+1] token offsets of the sequences in a contiguous cache (unused when paged)
  // paged cache (block_table != nullptr): the cache is [num_blocks * page, Hkv, D]; logical token u of sequence b lives
  // in physical row block_table[b * max_blocks + u / page] * page + u % page; page is a power of two dividing the tile
  const int32_t* block_table;
  const int32_t* seqlens; // [B] (paged only)
  int page, page_shift, max_blocks;
  float* partial;         // [B,Hq,n_splits,4+Dv]: m, l, two unused words (O starts on a 16-byte boundary), O[Dv]
  int B, Hq, Hkv, D, Dv, G;   // with several query tokens per sequence Hq and G count (token, head) rows: Sq * real values
  // Speculative / multi-token decode (Sec. 4.4): Sq query tokens per sequence, the last Sq tokens of its cache.  The
  // Sq * Gr rows that share a KV head are laid out token-major: row r of a KV head = (token r / Gr, head r % Gr);
  // query token s sees the cache up to position L - Sq + s.
  int Sq, Gr;
  int HG, Rp, groups;     // heads per CTA, stacked rows, head groups per KV head
  int DC, DVT;            // 128-byte chunks of D / Dv
  int n_splits, stages, chunk;   // chunk: tokens per split (a multiple of the tile)
  // Balanced schedule (narrow head groups): the tiles of all sequences, in order, form one list that is cut into equal
  // runs (of at least q_min tiles), each walked by one CTA per (KV head, head group); a CTA writes one partial result
  // per sequence its run touches, into the slot that counts the runs which began on that sequence before it, and the
  // CTA that reaches a sequence's end records how many slots there are (n_slots, one per sequence, KV head, head group).
  int balanced, q_min;
  int32_t* n_slots;
  int v_alias;            // 1: V is the first Dv bytes of the K rows
  int kv_chunks;          // 128-byte chunks reserved per KV stage (>= DC, and >= DVT when V aliases the K rows)
  int tmem_cols;
  float scale;
  unsigned* status;
  long long* trace;       // nullable diagnostic buffer: 32 clock samples per CTA (first 1024 CTAs)
  // nullable debug dumps for bit-exact checks (Alg. 3 lines 1-4): the two INT8 components of every query row
  // [2][B*Sq*Hq][D], their scales [2][B*Sq*Hq] (alpha_Q, beta_Q), and the two INT32 score planes [2][Sq*Hq][dbg_T]
  // indexed by the token's row in the cache
  int8_t* q_dbg;
  float* qs_dbg;
  int32_t* s_dbg;
  long long dbg_T;
};

__device__ __forceinline__ void attn_mark(const AttnParams& p, int slot) {
  const int cta = blockIdx.y * gridDim.x + blockIdx.x;
  if (p.trace && cta < 1024) p.trace[cta * 32 + slot] = clock64();
}


// a read-only global load that stays where it is written (volatile: the compiler neither moves it nor issues it again
// later to save a register)
__device__ __forceinline__ float ldg_f32_pinned(const float* ptr) {
  float v;
  asm volatile("ld.global.nc.f32 %0, [%1];" : "=f"(v) : "l"(ptr));
  return v;
}

// 2^x for x <= 0 (flushes tiny results to zero): one MUFU instruction
__device__ __forceinline__ float ex2_approx(float x) {
  float y;
  asm("ex2.approx.ftz.f32 %0, %1;" : "=f"(y) : "f"(x));
  return y;
}

// c1 for one query row (one warp): head slot h of the group's stacked operand (rows h and HG + h of every 128-byte
// chunk at `img`, 128-byte swizzle) and its two scales.  `img` is shared memory in the attention kernel's own set-up
// and global memory in attn_qstack_kernel; same bit-exact rule as msd_decompose_int8.
// index of the query row behind head slot h of a group: row r of the KV head -> (query token, head of the group)
__device__ __forceinline__ long long attn_q_row_index(const AttnParams& p, int b, int hk, int grp, int h) {
  const int r_kv = grp * p.HG + h, sq = r_kv / p.Gr;
  return (static_cast<long long>(b) * p.Sq + sq) * (p.Hkv * p.Gr) + hk * p.Gr + (r_kv - sq * p.Gr);
}
__device__ __forceinline__ void prefetch_l2(const void* ptr) {
  asm volatile("prefetch.global.L2 [%0];" ::"l"(ptr));
}

__device__ __forceinline__ void attn_decompose_q_row(const AttnParams& p, int b, int hk, int grp, int h, int lane, uint8_t* img,
                                                     float* alpha_out, float* beta_out) {
  const long long q_row = attn_q_row_index(p, b, hk, grp, h);
  const uint4* qrow = reinterpret_cast<const uint4*>(p.q + q_row * p.D);
  const int nvec = p.D >> 3;                    // 8 BF16 values per 16-byte load (D % 16 == 0, D <= 640)
  uint4 qv[3];                                  // the whole row stays in registers between the two passes
  float m = 0.0f;
#pragma unroll
  for (int j = 0; j < 3; ++j) {
    const int i = lane + 32 * j;
    qv[j] = (i < nvec) ? __ldg(qrow + i) : make_uint4(0, 0, 0, 0);
  }
#pragma unroll
  for (int j = 0; j < 3; ++j) {
    const uint32_t w[4] = {qv[j].x, qv[j].y, qv[j].z, qv[j].w};
#pragma unroll
    for (int k = 0; k < 4; ++k) {
      m = fmaxf(m, fabsf(__uint_as_float(w[k] << 16)));
      m = fmaxf(m, fabsf(__uint_as_float(w[k] & 0xFFFF0000u)));
    }
  }
  m = warp_max(m);
  const float alpha = __fdiv_rn(m, 127.0f), beta = __fdiv_rn(alpha, 254.0f);
  const float inv_alpha = alpha > 0.0f ? __frcp_rn(alpha) : 0.0f, inv_beta = beta > 0.0f ? __frcp_rn(beta) : 0.0f;
  if (lane == 0) {
    *alpha_out = alpha; *beta_out = beta;
    if (p.qs_dbg) {
      p.qs_dbg[q_row] = alpha;
      p.qs_dbg[static_cast<long long>(p.B) * p.Hq + q_row] = beta;
    }
  }
#pragma unroll
  for (int j = 0; j < 3; ++j) {
    const int i = lane + 32 * j;
    if (i >= nvec) continue;
    const uint32_t w[4] = {qv[j].x, qv[j].y, qv[j].z, qv[j].w};
    uint32_t o1[2] = {0, 0}, o2[2] = {0, 0};
#pragma unroll
    for (int e = 0; e < 8; ++e) {
      const float x = (e & 1) ? __uint_as_float(w[e >> 1] & 0xFFFF0000u) : __uint_as_float(w[e >> 1] << 16);
      int c1 = 0, c2 = 0;
      if (alpha > 0.0f) {
        c1 = quant_i8(x, alpha, inv_alpha);
        const float r = __fmaf_rn(-alpha, static_cast<float>(c1), x);
        if (beta > 0.0f) c2 = quant_i8(r, beta, inv_beta);
      }
      o1[e >> 2] |= static_cast<uint32_t>(c1 & 0xFF) << (8 * (e & 3));
      o2[e >> 2] |= static_cast<uint32_t>(c2 & 0xFF) << (8 * (e & 3));
    }
    const int d = i << 3;                       // eight consecutive bytes stay inside one 16-byte swizzle chunk
    uint8_t* chunk = img + (d >> 7) * p.Rp * kChunk;
    *reinterpret_cast<uint2*>(chunk + swz_off(h, d & 127)) = make_uint2(o1[0], o1[1]);
    *reinterpret_cast<uint2*>(chunk + swz_off(p.HG + h, d & 127)) = make_uint2(o2[0], o2[1]);
    if (p.q_dbg) {
      *reinterpret_cast<uint2*>(p.q_dbg + q_row * p.D + d) = make_uint2(o1[0], o1[1]);
      *reinterpret_cast<uint2*>(p.q_dbg + (static_cast<long long>(p.B) * p.Hq + q_row) * p.D + d) = make_uint2(o2[0], o2[1]);
    }
  }
}

// Two rows of at most 128 values at once: lanes 0-15 take head slot h_a, lanes 16-31 head slot h_b (h_b < 0: none), 8
// values per lane; the same arithmetic per element as attn_decompose_q_row, the row maximum reduced over 16 lanes.
__device__ __forceinline__ void attn_decompose_q_pair(const AttnParams& p, int b, int hk, int grp, int h_a, int h_b, int lane, uint8_t* img,
                                                      float* alpha_out, float* beta_out) {
  const int h = (lane < 16) ? h_a : h_b;
  const int i = lane & 15;
  const int nvec = p.D >> 3;                    // <= 16
  const bool row = h >= 0, live = row && i < nvec;
  const long long q_row = row ? attn_q_row_index(p, b, hk, grp, h) : 0;
  uint4 qv = make_uint4(0, 0, 0, 0);
  if (live) qv = __ldg(reinterpret_cast<const uint4*>(p.q + q_row * p.D) + i);
  const uint32_t w[4] = {qv.x, qv.y, qv.z, qv.w};
  float m = 0.0f;
#pragma unroll
  for (int k = 0; k < 4; ++k) {
    m = fmaxf(m, fabsf(__uint_as_float(w[k] << 16)));
    m = fmaxf(m, fabsf(__uint_as_float(w[k] & 0xFFFF0000u)));
  }
#pragma unroll
  for (int o = 8; o > 0; o >>= 1) m = fmaxf(m, __shfl_xor_sync(0xffffffffu, m, o));      // stays inside the 16 lanes
  const float alpha = __fdiv_rn(m, 127.0f), beta = __fdiv_rn(alpha, 254.0f);
  const float inv_alpha = alpha > 0.0f ? __frcp_rn(alpha) : 0.0f, inv_beta = beta > 0.0f ? __frcp_rn(beta) : 0.0f;
  if (row && i == 0) {
    alpha_out[h] = alpha; beta_out[h] = beta;
    if (p.qs_dbg) {
      p.qs_dbg[q_row] = alpha;
      p.qs_dbg[static_cast<long long>(p.B) * p.Hq + q_row] = beta;
    }
  }
  if (!live) return;
  uint32_t o1[2] = {0, 0}, o2[2] = {0, 0};
#pragma unroll
  for (int e = 0; e < 8; ++e) {
    const float x = (e & 1) ? __uint_as_float(w[e >> 1] & 0xFFFF0000u) : __uint_as_float(w[e >> 1] << 16);
    int c1 = 0, c2 = 0;
    if (alpha > 0.0f) {
      c1 = quant_i8(x, alpha, inv_alpha);
      const float r = __fmaf_rn(-alpha, static_cast<float>(c1), x);
      if (beta > 0.0f) c2 = quant_i8(r, beta, inv_beta);
    }
    o1[e >> 2] |= static_cast<uint32_t>(c1 & 0xFF) << (8 * (e & 3));
    o2[e >> 2] |= static_cast<uint32_t>(c2 & 0xFF) << (8 * (e & 3));
  }
  const int d = i << 3;                         // < 128: the row's single chunk
  *reinterpret_cast<uint2*>(img + swz_off(h, d)) = make_uint2(o1[0], o1[1]);
  *reinterpret_cast<uint2*>(img + swz_off(p.HG + h, d)) = make_uint2(o2[0], o2[1]);
  if (p.q_dbg) {
    *reinterpret_cast<uint2*>(p.q_dbg + q_row * p.D + d) = make_uint2(o1[0], o1[1]);
    *reinterpret_cast<uint2*>(p.q_dbg + (static_cast<long long>(p.B) * p.Hq + q_row) * p.D + d) = make_uint2(o2[0], o2[1]);
  }
}

// Debug dump of one thread's raw QK^T sums (Alg. 3 lines 3-4): token `tok_row` (row of the cache), head slots
// [hs, hs + n) of head group `grp` of KV head `hk`; c1 / c2 are the two components' accumulators.
template <int N>
__device__ __forceinline__ void attn_dump_scores(const AttnParams& p, long long tok_row, int hk, int grp, int hs, int nh,
                                                 const uint32_t (&c1)[N], const uint32_t (&c2)[N]) {
#pragma unroll
  for (int h = 0; h < N; ++h) {
    if (hs + h < nh) {
      const int r_kv = grp * p.HG + hs + h, sq = r_kv / p.Gr;
      const long long row = static_cast<long long>(sq) * (p.Hkv * p.Gr) + hk * p.Gr + (r_kv - sq * p.Gr);
      p.s_dbg[row * p.dbg_T + tok_row] = static_cast<int32_t>(c1[h]);
      p.s_dbg[(static_cast<long long>(p.Hq) + row) * p.dbg_T + tok_row] = static_cast<int32_t>(c2[h]);
    }
  }
}

// A CTA's position in its run of tiles: sequence b (seq0: its first row in a contiguous cache, L: its tokens), tile t
// of the nb tiles of that sequence, the tiles the CTA still has to do, and the unit u (KV head * groups + head group)
// whose rows it computes throughout.
struct AttnWalk { int b, u, t, nb, left, seq0, L; };

__device__ __forceinline__ int attn_seq_tokens(const AttnParams& p, int b) {
  return p.block_table ? __ldg(p.seqlens + b) : __ldg(p.cu + b + 1) - __ldg(p.cu + b);
}
__device__ __forceinline__ int attn_seq_tiles(const AttnParams& p, int b) {
  const int L = attn_seq_tokens(p, b);
  return L > 0 ? (L + kTok - 1) / kTok : 0;
}
__device__ __forceinline__ void attn_walk_load(const AttnParams& p, AttnWalk& w) {      // L, nb, seq0 of sequence w.b
  w.seq0 = p.block_table ? 0 : __ldg(p.cu + w.b);
  w.L = max(attn_seq_tokens(p, w.b), 0);
  w.nb = (w.L + kTok - 1) / kTok;
}
// n tiles further (n never crosses the end of the sequence): on to the next sequence that has tokens
template <bool kBalanced>
__device__ __forceinline__ void attn_walk_advance(const AttnParams& p, AttnWalk& w, int n) {
  w.t += n;
  w.left -= n;
  if constexpr (!kBalanced) return;          // a fixed split never leaves its sequence
  if (w.t >= w.nb && w.left > 0) {
    w.t = 0;
    do {
      if (++w.b >= p.B) { w.left = 0; w.nb = 1; break; }     // cannot happen while the lengths stay what they were when the runs were cut
      attn_walk_load(p, w);
    } while (w.nb == 0);
  }
}

// Balanced schedule.  The tiles of all sequences, in order, form one list; it is cut into R equal runs, and run i is
// walked by the U = Hkv * groups consecutive CTAs [i U, (i+1) U), one per unit - so the CTAs that are dispatched
// together read the same token rows of the cache, one KV head each (whole DRAM pages between them), and every CTA
// has the same number of tiles.  Computes this CTA's run and the slot of its first partial result (the runs that
// began on the same sequence before it).  Called by all threads; false: nothing to do for this CTA.
__device__ __forceinline__ bool attn_walk_init(const AttnParams& p, int* s_scan, AttnWalk* w, int* slot0) {
  const int tid = threadIdx.x, lane = tid & 31;
  const int U = p.Hkv * p.groups;
  const int per = (p.B + kAttnThreads - 1) / kAttnThreads;
  int sum = 0;
  for (int b = tid * per; b < min(p.B, (tid + 1) * per); ++b) {
    const int n = attn_seq_tiles(p, b);
    sum += n;
    if (blockIdx.x < U && n == 0) p.n_slots[static_cast<long long>(b) * U + blockIdx.x] = 0;     // no tokens, no partial result
  }
  s_scan[tid] = sum;
  __syncthreads();
  // every warp for itself: lane l sums the entries of threads [6 l, 6 l + 6), then a scan over the lanes
  constexpr int kPerLane = kAttnThreads / 32;
  int v = 0;
#pragma unroll
  for (int j = 0; j < kPerLane; ++j) v += s_scan[lane * kPerLane + j];
  int incl = v;
#pragma unroll
  for (int o = 1; o < 32; o <<= 1) {
    const int n = __shfl_up_sync(0xffffffffu, incl, o);
    if (lane >= o) incl += n;
  }
  const int W = __shfl_sync(0xffffffffu, incl, 31);            // tiles in the list (< 2^24: the cache has < 2^31 rows)
  if (W == 0) return false;
  int R = min(W / p.q_min, static_cast<int>(gridDim.x) / U);   // runs: of at least q_min tiles, no more than fit the grid
  R = R < 1 ? 1 : R;
  const int ri = blockIdx.x / U;
  if (ri >= R) return false;
  const int lo = static_cast<int>(static_cast<long long>(ri) * W / R), hi = static_cast<int>(static_cast<long long>(ri + 1) * W / R);
  const unsigned bal = __ballot_sync(0xffffffffu, incl > lo);  // not 0: W > lo
  const int sel = __ffs(bal) - 1;
  int P = __shfl_sync(0xffffffffu, incl - v, sel);             // tiles of the sequences in front
  int idx = sel * kPerLane;
  while (idx < sel * kPerLane + kPerLane - 1 && P + s_scan[idx] <= lo) { P += s_scan[idx]; ++idx; }
  int b = idx * per, nb = 0;
  for (; b < p.B; ++b) {
    nb = attn_seq_tiles(p, b);
    if (P + nb > lo) break;
    P += nb;
  }
  if (b >= p.B || nb == 0) return false;     // (unreachable)
  w->b = b;
  attn_walk_load(p, *w);
  w->u = blockIdx.x - ri * U;
  w->t = lo - P;
  w->left = hi - lo;
  // the run that owns list position f is floor(((f + 1) R - 1) / W); the sequence began at position P
  *slot0 = (w->t > 0) ? ri - static_cast<int>((static_cast<long long>(P + 1) * R - 1) / W) : 0;
  return true;
}

// c1 (Alg. 3 lines 1-2) once per (sequence, KV head, head group) instead of once per context split: the query rows of
// the group's heads are decomposed into two INT8 components (same bit-exact rule as msd_decompose_int8) and written
// as the stacked operand image the attention CTAs copy into shared memory with one bulk copy per chunk.  One CTA per
// unit, one warp per head round robin.
__global__ void __launch_bounds__(1024)
attn_qstack_kernel(const AttnParams p, uint8_t* __restrict__ q_img, float* __restrict__ q_scales) {
  pdl_launch_dependents();
  const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
  int unit = blockIdx.x;
  const int grp = unit % p.groups; unit /= p.groups;
  const int hk = unit % p.Hkv;
  const int b = unit / p.Hkv;
  const int nh = min(p.HG, p.G - grp * p.HG);
  const int img_bytes = p.DC * p.Rp * kChunk;
  uint8_t* img = q_img + static_cast<size_t>(blockIdx.x) * img_bytes;
  float* sc = q_scales + static_cast<size_t>(blockIdx.x) * 2 * p.HG;
  // unused head slots and the padding of the last D chunk must be zero
  for (int i = threadIdx.x; i < img_bytes / 16; i += blockDim.x) reinterpret_cast<uint4*>(img)[i] = make_uint4(0, 0, 0, 0);
  for (int i = threadIdx.x; i < 2 * p.HG; i += blockDim.x) sc[i] = 0.0f;
  __syncthreads();
  for (int h = warp; h < nh; h += static_cast<int>(blockDim.x >> 5)) attn_decompose_q_row(p, b, hk, grp, h, lane, img, sc + h, sc + p.HG + h);
}

// Head groups of up to 8 query rows per KV head (GQA).  kMaxHG: head slots one softmax thread looks after (8; the code
// also compiles for 16, which the planner no longer picks);
// kNH: heads its code is unrolled for (<= kMaxHG); kMaxDVT: 128-wide tiles of Dv.
// kPaged: the cache is paged (block table); a template parameter so that the contiguous kernels carry none of it.
template <int kMaxHG, int kNH, int kMaxDVT, bool kPaged, bool kBalanced>
__global__ void __launch_bounds__(kAttnThreads, (kNH <= 8 && kMaxDVT == 1) ? 3 : 1)
attn_decode_kernel(const __grid_constant__ CUtensorMap tmap_k, const __grid_constant__ CUtensorMap tmap_v, const AttnParams p) {
  extern __shared__ uint8_t smem_dyn[];
  __shared__ __align__(8) uint64_t kv_full[4], kv_empty[4], v_full[4], v_empty[4], s_full[2], p_full[2], q_ready, o_full, o_empty;
  __shared__ uint32_t tmem_base_slot;
  __shared__ int abort_flag;
  // The CTA decomposes its few query rows itself (beside the other CTAs of the SM); wide head groups, where that
  // would be repeated by every context split, take them from attn_qstack_kernel instead (attn_decode_wide_kernel).
  constexpr int kSlots = kMaxHG;                   // head slots of the stacked operands: rows [0,kSlots) first
  constexpr int kNSW = 4;                          // component, rows [kSlots, 2*kSlots) second component
  __shared__ float s_aq[kSlots], s_bq[kSlots];
  __shared__ float red[2][4][kNH + 1];             // per-warp tile maxima, double buffered by tile parity
  // More than 4 heads per thread: what is the same in all threads of a warp and only read now and then - the query
  // scales, and the rescale factors a tile's softmax hands to its merge - stays in shared memory (per warp, by tile
  // parity), or the kernel does not fit the 96 registers that three CTAs per SM allow.
  constexpr bool kSmemState = kNH > 4;
  __shared__ float s_resc[kSmemState ? 2 : 1][4][kNH];
  __shared__ int s_scan[kAttnThreads];
  __shared__ AttnWalk s_walk;                      // the softmax warps' walk (kept here, not in registers, between segments)
  __shared__ int s_slot;

  const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
  const int U = p.Hkv * p.groups;
  // The CTA's tiles: a run of the list of all sequences' tiles (balanced schedule), or one context split of one
  // sequence (fixed splits: units along x, launched first, splits along y - the early splits of every sequence, which
  // are always full, start before the last, shorter ones); always for one unit.  Either way the run is walked sequence
  // by sequence ("segments"): all roles below step through the same AttnWalk, and tiles, buffers and barrier phases
  // are counted over the whole run, not per segment.
  AttnWalk w0;
  int slot0;
  if constexpr (kBalanced) {
    if (!attn_walk_init(p, s_scan, &w0, &slot0)) return;
  } else {
    const int split = blockIdx.y, b = blockIdx.x / U;
    const int L = attn_seq_tokens(p, b);
    const int t_begin = split * p.chunk;                       // every split covers the same number of tokens
    const int t_end = min(L, t_begin + p.chunk);
    const int ntiles = (t_end > t_begin) ? (t_end - t_begin + kTok - 1) / kTok : 0;
    if (ntiles == 0) {      // nothing in this split: neutral partials, before any barrier or TMEM use
      const int grp = blockIdx.x % p.groups, hk = (blockIdx.x / p.groups) % p.Hkv;
      const int h0 = hk * p.G + grp * p.HG, nh = min(p.HG, p.G - grp * p.HG);
      for (int i = threadIdx.x; i < nh * (p.Dv + kPartHdr); i += blockDim.x) {
        const int h = i / (p.Dv + kPartHdr), e = i % (p.Dv + kPartHdr);
        float* dst = p.partial + ((static_cast<long long>(b) * p.Hq + h0 + h) * p.n_splits + split) * (p.Dv + kPartHdr);
        dst[e] = (e == 0) ? -INFINITY : 0.0f;
      }
      return;
    }
    w0.b = b; w0.u = blockIdx.x % U; w0.t = t_begin / kTok; w0.left = ntiles;
    attn_walk_load(p, w0);
    slot0 = split;
  }
  const int total_tiles = w0.left;
  // The scales of the CTA's first tile, asked for as early as their address is known (softmax threads: one token each):
  // at the start everything is a cold read that queues behind the first KV tiles of every CTA of the grid.
  float ks_first = 0.0f, vs_first = 0.0f;
  if (threadIdx.x >= 64) {
    const int tok_rel = w0.t * kTok + (warp & 3) * 32 + lane;      // the thread's token lane (its warp's quarter of tensor memory)
    if (tok_rel < w0.L) {
      long long row = w0.seq0 + tok_rel;
      if constexpr (kPaged)
        row = static_cast<long long>(__ldg(p.block_table + static_cast<long long>(w0.b) * p.max_blocks + (tok_rel >> p.page_shift))) * p.page +
              (tok_rel & (p.page - 1));
      const long long sidx = row * p.Hkv + (blockIdx.x % U) / p.groups;
      ks_first = ldg_f32_pinned(p.k_scale + sidx);
      vs_first = ldg_f32_pinned(p.v_scale + sidx);
    }
  }
  if (threadIdx.x == 0 && p.trace) {
    attn_mark(p, 0);
    unsigned long long g;
    asm volatile("mov.u64 %0, %globaltimer;" : "=l"(g));
    const int cta = blockIdx.y * gridDim.x + blockIdx.x;
    if (cta < 1024) { p.trace[cta * 32 + 1] = static_cast<long long>(g); p.trace[cta * 32 + 2] = total_tiles; }
  }

  uint8_t* smem = reinterpret_cast<uint8_t*>((reinterpret_cast<uintptr_t>(smem_dyn) + 1023) & ~static_cast<uintptr_t>(1023));
  const int kv_stage_bytes = p.kv_chunks * kChunkBytes;
  uint8_t* sm_q = smem + p.stages * kv_stage_bytes;          // DC chunks of [Rp x 128]
  uint8_t* sm_p = sm_q + p.DC * p.Rp * kChunk;               // [Rp x 128]

  if (threadIdx.x == 0) {
    for (int s = 0; s < p.stages; ++s) {
      mbar_init(&kv_full[s], 1); mbar_init(&kv_empty[s], 1);
      mbar_init(&v_full[s], 1); mbar_init(&v_empty[s], 1);
    }
    mbar_init(&s_full[0], 1); mbar_init(&s_full[1], 1);
    // one P barrier per P buffer: the softmax may run one tile ahead of the PV issue, and a single barrier could then
    // be two phases past the one the MMA warp is testing, which a parity test cannot tell from "not yet"
    mbar_init(&p_full[0], kNSW); mbar_init(&p_full[1], kNSW); mbar_init(&q_ready, kNSW);
    mbar_init(&o_full, 1); mbar_init(&o_empty, kNSW);
    abort_flag = 0;
    for (int h = 0; h < kSlots; ++h) { s_aq[h] = 0.0f; s_bq[h] = 0.0f; }      // head slots without a head
    s_walk = w0;
    s_slot = slot0;
    mbar_init_fence();
    tma_prefetch_desc(&tmap_k);
    tma_prefetch_desc(&tmap_v);
  }
  if (warp == 1) tmem_alloc(&tmem_base_slot, p.tmem_cols);
  // zero the stacked Q operand (unused head slots and the padding of the last D chunk must be zero)
  for (int i = threadIdx.x; i < p.DC * p.Rp * kChunk / 16; i += blockDim.x) reinterpret_cast<uint4*>(sm_q)[i] = make_uint4(0, 0, 0, 0);
  tc_fence_before();
  __syncthreads();
  tc_fence_after();
  const uint32_t tmem_base = tmem_base_slot;
  const uint32_t tmem_o = tmem_base + 2 * p.Rp;             // O^T tiles after the two S^T buffers
  volatile int* abort = &abort_flag;

  if (warp == 0) {
    // ------------------------------ TMA producer: K (and V) tiles ------------------------------
    if (lane == 0) {
      // K tiles and (when V is a separate cache) V tiles travel in rings of their own: a K buffer is free again as
      // soon as QK^T has read it, long before the PV product of the same tile releases the V buffer, so the next K
      // tile can be fetched that much earlier.  With V aliased to the K rows there is only the K ring.
      const int k_bytes = p.DC * kChunkBytes, v_bytes = p.DVT * kChunkBytes;
      AttnWalk wk = w0, wv = w0;                 // where the next K / V tile comes from
      int kq = 0, vq = p.v_alias ? total_tiles : 0;
      // the tile at walk position w: chunks [0, nchunks) of the rows of KV head hk into dst
      const int hk = w0.u / p.groups;
      auto load_tile = [&](const AttnWalk& w, const CUtensorMap* tmap, int nchunks, uint8_t* dst, uint64_t* bar) {
        const int u0 = w.t * kTok;
        if constexpr (!kPaged) {
          mbar_arrive_expect_tx(bar, nchunks * kChunkBytes);
          for (int c = 0; c < nchunks; ++c) tma_load_3d(dst + c * kChunkBytes, tmap, c * kChunk, hk, w.seq0 + u0, bar);
        } else {
          // one box per page that holds tokens of the sequence; rows of the tile past them keep stale (finite) codes
          // and are masked like every token past the end
          const int32_t* bt = p.block_table + static_cast<long long>(w.b) * p.max_blocks;
          const int npg = min(kTok >> p.page_shift, (w.L - u0 + p.page - 1) >> p.page_shift);
          mbar_arrive_expect_tx(bar, nchunks * kChunk * p.page * npg);
          for (int pg = 0; pg < npg; ++pg) {
            const int tok = __ldg(bt + (u0 >> p.page_shift) + pg) * p.page;
            for (int c = 0; c < nchunks; ++c)
              tma_load_3d(dst + c * kChunkBytes + pg * p.page * kChunk, tmap, c * kChunk, hk, tok, bar);
          }
        }
      };
      long long t_idle = clock64();
      while (kq < total_tiles || vq < total_tiles) {
        bool progressed = false;
        if (kq < total_tiles && mbar_test_wait(&kv_empty[kq % p.stages], ((kq / p.stages) & 1) ^ 1)) {
          const int st = kq % p.stages;
          load_tile(wk, &tmap_k, p.DC, smem + st * kv_stage_bytes, &kv_full[st]);
          attn_walk_advance<kBalanced>(p, wk, 1);
          ++kq;
          progressed = true;
        }
        if (vq < total_tiles && mbar_test_wait(&v_empty[vq % p.stages], ((vq / p.stages) & 1) ^ 1)) {
          const int st = vq % p.stages;
          load_tile(wv, &tmap_v, p.DVT, smem + st * kv_stage_bytes + k_bytes, &v_full[st]);
          attn_walk_advance<kBalanced>(p, wv, 1);
          ++vq;
          progressed = true;
        }
        if (progressed) {
          t_idle = clock64();
        } else {
          if (*abort) break;
          if (clock64() - t_idle > kWaitBudgetCycles) {
            *abort = 1;
            atomicMax(p.status, kStatusTimeout);
            break;
          }
        }
      }
      (void)v_bytes;
    }
  } else if (warp == 1) {
    // ------------------------------ MMA issuer ------------------------------
    if (lane == 0) {
      const uint32_t idesc_qk = idesc_dense(2, 1, 1, 0, 0, kTok, p.Rp);     // S8 x S8 -> S32, both K-major
      const uint32_t idesc_pv = idesc_dense(2, 1, 1, 1, 0, kTok, p.Rp);     // A (V^T) MN-major
      bool ok = true;
      // Operand descriptors differ from three templates only in the 16-byte-granular address field (bits 0-13), so each
      // costs one 64-bit add: with 36 MMAs per MLA tile this thread's instruction count is on the critical path.
      const uint64_t dk = smem_desc(0, 16, 1024, kSwizzle128B);         // K-major tiles: K, stacked Q, P
      const uint64_t dvt = smem_desc(0, 16384, 1024, kSwizzle128B);     // V^T read MN-major from the token-major tile
      const uint64_t q_enc = dk + (smem_u32(sm_q) >> 4);
      const uint64_t p_enc = dk + (smem_u32(sm_p) >> 4);
      const uint32_t smem_enc = smem_u32(smem) >> 4;
      const uint32_t q_step = static_cast<uint32_t>(p.Rp * kChunk) >> 4, p_step = q_step;
      auto issue_qk = [&](int t) {
        const int st = t % p.stages;
        tc_fence_after();
        uint64_t ka = dk + smem_enc + static_cast<uint32_t>(st * (kv_stage_bytes >> 4));
        uint64_t qa = q_enc;
        const uint32_t d = tmem_base + (t & 1) * p.Rp;
        for (int c = 0; c < p.DC; ++c) {
#pragma unroll
          for (int k = 0; k < 4; ++k) mma_i8(d, ka + 2 * k, qa + 2 * k, idesc_qk, (c > 0 || k > 0) ? 1u : 0u);
          ka += kChunkBytes >> 4;
          qa += q_step;
        }
        tc_commit(&s_full[t & 1]);
        if (!p.v_alias) tc_commit(&kv_empty[st]);       // separate V: the K buffer is free once QK^T has read it
      };
      auto issue_pv = [&](int t) {
        tc_fence_after();
        const int st = t % p.stages;
        uint64_t va = dvt + smem_enc + static_cast<uint32_t>(st * (kv_stage_bytes >> 4)) +
                      (p.v_alias ? 0u : static_cast<uint32_t>(p.DC * (kChunkBytes >> 4)));
        const uint64_t pa = p_enc + (t & 1) * p_step;
        uint32_t d = tmem_o;
        for (int j = 0; j < p.DVT; ++j) {
#pragma unroll
          for (int k = 0; k < 4; ++k)        // 32 tokens per MMA: four 8-token groups of 1024 bytes
            mma_i8(d, va + k * (4096 >> 4), pa + 2 * k, idesc_pv, k > 0 ? 1u : 0u);
          va += kChunkBytes >> 4;
          d += p.Rp;
        }
        tc_commit(&o_full);
        tc_commit(p.v_alias ? &kv_empty[st] : &v_empty[st]);
      };
      // Two streams of work, each in tile order, issued as soon as their inputs are there (whichever comes first):
      //   QK^T(q) needs the KV tile q in shared memory, the score buffer q&1 drained (P of tile q-2 written) and, for
      //           the first tile of a segment, that segment's stacked Q operand (written once the previous segment's
      //           last merge is done, so every earlier QK^T has read the old one);
      //   PV(v)   needs P of tile v written, O^T of tile v-1 merged, and QK^T(v) already issued.
      // A QK^T that waits for its KV tile must not hold back a PV whose operands are ready, and vice versa.
      AttnWalk wq = w0;
      int q = 0, v = 0, seg = 0;                 // seg: segments whose stacked Q operand has been waited for
      bool q_first = true;                       // tile q is the first of its segment
      long long t_idle = clock64();
      while (ok && v < total_tiles) {
        bool progressed = false;
        if (q < total_tiles && q < v + 2 &&
            mbar_test_wait(&kv_full[q % p.stages], (q / p.stages) & 1) &&    // (q < v + 2 implies P of tile q-2 is written)
            (!q_first || mbar_test_wait(&q_ready, seg & 1))) {
          if (q_first) ++seg;
          issue_qk(q);
          attn_walk_advance<kBalanced>(p, wq, 1);
          q_first = kBalanced && wq.t == 0;
          ++q;
          progressed = true;
        }
        if (v < q && mbar_test_wait(&p_full[v & 1], (v >> 1) & 1) && (v == 0 || mbar_test_wait(&o_empty, (v - 1) & 1)) &&
            (p.v_alias || mbar_test_wait(&v_full[v % p.stages], (v / p.stages) & 1))) {
          issue_pv(v);
          ++v;
          progressed = true;
        }
        if (progressed) {
          t_idle = clock64();
        } else {
          if (*abort) { ok = false; break; }
          if (clock64() - t_idle > kWaitBudgetCycles) {
            *abort = 1;
            atomicMax(p.status, kStatusTimeout);
            ok = false;
          }
        }
      }
    }
  } else {
    // ------------------------------ softmax + merge warps ------------------------------
    const int quad = warp & 3;
    const int tl = quad * 32 + lane;                // token lane (softmax) / dv lane (merge)
    const int wi = warp - 2;                        // 0 .. 3
    const int wq = wi;
    constexpr int hs0 = 0;                          // first head slot of this warp
    const int bar_id = 1;
    constexpr int kRegState = kNH;
    const float kLog2e = 1.4426950408889634f;
    const float scale2 = p.scale * kLog2e;
    bool ok = true;
    int g0 = 0;                                     // tiles of the segments done so far
    // the CTA's unit: the same KV head and head group in every segment
    const int hk = (blockIdx.x % U) / p.groups, grp = (blockIdx.x % U) - hk * p.groups;
    const int nh = min(p.HG, p.G - grp * p.HG);                // heads actually present
    bool more = true;
    while (ok && more) {
      // ---- one segment: tiles [t, t + ntiles) of sequence b, from the walk in shared memory (it is advanced by one
      // thread between two barriers at the end of the segment; what the tile loop does not need is read again after it)
      const int ntiles = min(s_walk.left, s_walk.nb - s_walk.t);
      const int b = s_walk.b;
      const int32_t* bt = kPaged ? p.block_table + static_cast<long long>(b) * p.max_blocks : nullptr;
      const int seq0 = s_walk.seq0, L = s_walk.L;
      const int t_begin = s_walk.t * kTok;
      const int t_end = min(L, t_begin + ntiles * kTok);
      // c1: decompose the query rows of this segment's heads (one warp per head, round robin) into the stacked operand
      // (the head slots and padding columns that were zeroed at the start are never written)
      if (kNH > 4 && kMaxHG == 8 && p.D <= 128) {
        // more than four rows of at most 128 values: a warp takes its two rows side by side, 16 lanes each (one after
        // the other the stacked operand was ready 5.4 us after the CTA's start instead of 3.0 us with one row per warp)
        if (wi < nh) attn_decompose_q_pair(p, b, hk, grp, wi, wi + kNSW < nh ? wi + kNSW : -1, lane, sm_q, s_aq, s_bq);
      } else {
        for (int h = wi; h < nh; h += kNSW) attn_decompose_q_row(p, b, hk, grp, h, lane, sm_q, &s_aq[h], &s_bq[h]);
      }
      fence_proxy_async_smem();
      __syncwarp();
      if (lane == 0) mbar_arrive(&q_ready);           // the stacked Q operand is in shared memory
      named_bar_sync(8, 128);                         // s_aq / s_bq visible to all softmax warps
      if (threadIdx.x == 64 && g0 == 0) attn_mark(p, 3);

      // running state per head; scores are kept in the log2 domain (log2(e) is folded into the key scale)
      // the state that is uniform across the four warps (running maxima, query scales) lives in registers
      float l_part[kNH];
      float m_run[kRegState], aq[kRegState], bq[kRegState], resc_keep[kRegState], resc_next[kRegState];
      float o_run[kMaxDVT][kNH];
#pragma unroll
      for (int h = 0; h < kNH; ++h) {
        l_part[h] = 0.0f;
        m_run[h] = -INFINITY;
        aq[h] = (!kSmemState && hs0 + h < nh) ? s_aq[hs0 + h] : 0.0f;
        bq[h] = (!kSmemState && hs0 + h < nh) ? s_bq[hs0 + h] : 0.0f;
#pragma unroll
        for (int j = 0; j < kMaxDVT; ++j) o_run[j][h] = 0.0f;
      }
      // State a tile's softmax hands to its merge: rescale factors and the P scales.  The softmax of tile t+1 runs
      // BEFORE the merge of tile t (it overlaps the PV product of tile t), so two sets are alive at a time.
      float ap_cur = 0.0f, bp_cur = 0.0f, ap_nxt = 0.0f, bp_nxt = 0.0f;

      // Per-token scales of tile t for this thread's token lane (0 past the end of the segment).  They are fetched one
      // tile ahead: a cold 512-byte run of the scale arrays would otherwise sit on every tile's critical path.
      auto load_scales = [&](int t, float& ks_out, float& vs_out) {
        const int tok_rel = t_begin + t * kTok + tl;
        const bool valid = t < ntiles && tok_rel < t_end;
        long long sidx;
        if constexpr (kPaged) {
          const long long prow = valid ? static_cast<long long>(__ldg(bt + (tok_rel >> p.page_shift))) * p.page + (tok_rel & (p.page - 1)) : 0;
          sidx = prow * p.Hkv + hk;
        } else {
          sidx = static_cast<long long>(seq0 + tok_rel) * p.Hkv + hk;
        }
        ks_out = valid ? __ldg(p.k_scale + sidx) : 0.0f;
        vs_out = valid ? __ldg(p.v_scale + sidx) : 0.0f;
      };
      float ks_pre, vs_pre;
      if (g0 == 0) { ks_pre = ks_first; vs_pre = vs_first; }
      else load_scales(0, ks_pre, vs_pre);
      // c3-c5 for tile t of the segment (tile g0 + t of the CTA): scores -> running max -> P -> two INT8 components
      // into P buffer ((g0 + t) & 1)
      auto softmax_tile = [&](int t, float (&resc_out)[kRegState], float& alpha_p, float& beta_p) -> bool {
        const int gt = g0 + t;
        const int tok_rel = t_begin + t * kTok + tl;
        const bool valid = tok_rel < t_end;
        const float ks = ks_pre * scale2;
        const float vs = vs_pre;
        load_scales(t + 1, ks_pre, vs_pre);
        if (!wait_bounded(&s_full[gt & 1], (gt >> 1) & 1, abort, p.status)) return false;
        if (threadIdx.x == 64 && gt < 6) attn_mark(p, 4 + 4 * gt);
        tc_fence_after();
        float s[kNH];
        const uint32_t srow = tmem_base + (static_cast<uint32_t>(quad * 32) << 16) + (gt & 1) * p.Rp;
        {
          uint32_t v1[kMaxHG], v2[kMaxHG];          // first / second component columns
          tmem_ldw<kMaxHG>(srow + hs0, v1);
          tmem_ldw<kMaxHG>(srow + kSlots + hs0, v2);
          tmem_ld_wait();
          if (p.s_dbg && valid) {
            long long tok_row = seq0 + tok_rel;
            if constexpr (kPaged) tok_row = static_cast<long long>(__ldg(bt + (tok_rel >> p.page_shift))) * p.page + (tok_rel & (p.page - 1));
            attn_dump_scores<kMaxHG>(p, tok_row, hk, grp, hs0, nh, v1, v2);
          }
#pragma unroll
          for (int h = 0; h < kNH; ++h)
          {
            const float a_q = kSmemState ? s_aq[hs0 + h] : aq[h], b_q = kSmemState ? s_bq[hs0 + h] : bq[h];
            bool vh = valid;
            if (p.Sq > 1) vh = valid && tok_rel < L - p.Sq + 1 + (grp * p.HG + hs0 + h) / p.Gr;    // causal among the new tokens
            s[h] = vh ? __fmaf_rn(a_q, static_cast<float>(static_cast<int32_t>(v1[h])), b_q * static_cast<float>(static_cast<int32_t>(v2[h]))) * ks : -INFINITY;
          }
        }
        // c4: tile maxima per head (and of the value scales) over the 128 token lanes
        float (*rb)[kNH + 1] = red[gt & 1];
#pragma unroll
        for (int h = 0; h < kNH; ++h) {
          const float wm = warp_max(s[h]);
          if (lane == 0) rb[wq][h] = wm;
        }
        {
          const float wv = warp_max(vs);
          if (lane == 0) rb[wq][kNH] = wv;
        }
        named_bar_sync(bar_id, 128);  // one barrier per tile: the other parity buffer is rewritten only after the next one
        // running maximum of every head before and after the tile; rescale factor of what was accumulated so far
        // (all heads first: as many independent exponentials in flight as there are heads)
        float mn_t[kRegState], resc_t[kRegState];
#pragma unroll
        for (int h = 0; h < kNH; ++h) {
          const float mt = fmaxf(fmaxf(rb[0][h], rb[1][h]), fmaxf(rb[2][h], rb[3][h]));
          mn_t[h] = fmaxf(m_run[h], mt);
          resc_t[h] = (m_run[h] == -INFINITY) ? 0.0f : ex2_approx(m_run[h] - mn_t[h]);
          m_run[h] = mn_t[h];
          if constexpr (kSmemState) { if (lane == 0) s_resc[gt & 1][wq][h] = resc_t[h]; }      // (__syncwarp below, before P is announced)
          else resc_out[h] = resc_t[h];
        }
        const float vs_max = fmaxf(fmaxf(rb[0][kNH], rb[1][kNH]), fmaxf(rb[2][kNH], rb[3][kNH]));
        // c5: P = exp(S - m), fold the value scale, two-pass INT8 with the fixed scale alpha_P = max(v_scale)/127
        alpha_p = vs_max * (1.0f / 127.0f);
        beta_p = alpha_p * (1.0f / 254.0f);
        const float inv_a = alpha_p > 0.0f ? __frcp_rn(alpha_p) : 0.0f, inv_b = beta_p > 0.0f ? __frcp_rn(beta_p) : 0.0f;
        uint8_t* pbuf = sm_p + (gt & 1) * p.Rp * kChunk;      // PV of tile gt-2 (same buffer) finished before merge(gt-2)
#pragma unroll
        for (int h = 0; h < kNH; ++h) {
          // branch-free: an absent head or a token past the end contributes P = 0 (s is -inf there)
          const float mn = mn_t[h], resc = resc_t[h];
          // (a row that has seen no visible token yet keeps m = -inf: the clamp turns -inf - -inf into -inf, P = 0)
          const float pr = (hs0 + h < nh) ? ex2_approx(s[h] - fmaxf(mn, -1e30f)) : 0.0f;
          l_part[h] = __fmaf_rn(l_part[h], resc, pr);
          const float pt = pr * vs;
          // Two-pass INT8 by the 1.5 * 2^23 trick: adding it rounds to the nearest integer (ties to even) and leaves that
          // integer in the low mantissa bits, so neither pass needs a float <-> int conversion.  No clamps: P <= 1 and
          // v_scale <= its tile maximum give pt / alpha_P <= 127, and |r| <= alpha_P / 2 gives |r / beta_P| <= 127.
          const float kMagic = 12582912.0f;
          const float u1 = __fmaf_rn(pt, inv_a, kMagic);
          const float r = __fmaf_rn(-alpha_p, u1 - kMagic, pt);
          const float u2 = __fmaf_rn(r, inv_b, kMagic);
          pbuf[swz_off(hs0 + h, tl)] = static_cast<uint8_t>(__float_as_uint(u1));
          pbuf[swz_off(kSlots + hs0 + h, tl)] = static_cast<uint8_t>(__float_as_uint(u2));
        }
        fence_proxy_async_smem();
        tc_fence_before();
        __syncwarp();
        if (lane == 0) mbar_arrive(&p_full[gt & 1]);
        if (threadIdx.x == 64 && gt < 6) attn_mark(p, 5 + 4 * gt);
        return true;
      };

      ok = softmax_tile(0, resc_keep, ap_cur, bp_cur);
      for (int t = 0; t < ntiles && ok; ++t) {
        const int gt = g0 + t;
        if (t + 1 < ntiles) {
          ok = softmax_tile(t + 1, resc_next, ap_nxt, bp_nxt);     // overlaps the PV product of tile t
          if (!ok) break;
        }
        // c6/c7: wait for O^T of tile t, merge it into the running output with that tile's rescale factors
        ok = wait_bounded(&o_full, gt & 1, abort, p.status);
        if (!ok) break;
        if (threadIdx.x == 64 && gt < 6) attn_mark(p, 6 + 4 * gt);
        tc_fence_after();
        float resc_cur[kNH];                 // e^(m before tile t - m after tile t), from the softmax of tile t
#pragma unroll
        for (int h = 0; h < kNH; ++h) resc_cur[h] = kSmemState ? s_resc[gt & 1][wq][h] : resc_keep[h];
#pragma unroll
        for (int j = 0; j < kMaxDVT; ++j) {
          if (j < p.DVT) {
            const uint32_t orow = tmem_o + (static_cast<uint32_t>(quad * 32) << 16) + j * p.Rp;
            uint32_t v1[kMaxHG], v2[kMaxHG];
            tmem_ldw<kMaxHG>(orow + hs0, v1);
            tmem_ldw<kMaxHG>(orow + kSlots + hs0, v2);
            tmem_ld_wait();
#pragma unroll
            for (int h = 0; h < kNH; ++h)
              // alpha_P O1 + beta_P O2 with beta_P = alpha_P / 254: one integer multiply-add and one conversion
              // (|254 O1 + O2| <= 255 * 128 * 127 * 127 < 2^31)
              o_run[j][h] = __fmaf_rn(o_run[j][h], resc_cur[h], bp_cur * static_cast<float>(254 * static_cast<int32_t>(v1[h]) + static_cast<int32_t>(v2[h])));
          }
        }
        tc_fence_before();
        __syncwarp();
        if (lane == 0) mbar_arrive(&o_empty);
        if (threadIdx.x == 64 && gt < 6) attn_mark(p, 7 + 4 * gt);
#pragma unroll
        for (int h = 0; h < kRegState; ++h) resc_keep[h] = resc_next[h];
        ap_cur = ap_nxt;
        bp_cur = bp_nxt;
      }
      (void)ap_cur;
      if (threadIdx.x == 64) attn_mark(p, 28);
      // partial results of this segment: running max, sum of P and unnormalised output per head
      if (ok) {
        float (*rb)[kNH + 1] = red[(g0 + ntiles) & 1];
        named_bar_sync(bar_id, 128);
#pragma unroll
        for (int h = 0; h < kNH; ++h) {
          float l = l_part[h];
#pragma unroll
          for (int o = 16; o > 0; o >>= 1) l += __shfl_xor_sync(0xffffffffu, l, o);
          if (lane == 0) rb[wq][h] = l;
        }
        named_bar_sync(bar_id, 128);
        const int slot = s_slot, bb = s_walk.b;
        const int h0 = hk * p.G + grp * p.HG;                      // first query head
        if (slot < p.n_splits) {
#pragma unroll
          for (int h = 0; h < kNH; ++h) {
            if (hs0 + h < nh) {
              float* dst = p.partial + ((static_cast<long long>(bb) * p.Hq + h0 + hs0 + h) * p.n_splits + slot) * (p.Dv + kPartHdr);
              // the running maximum goes out in natural-log units (it was kept in the log2 domain)
              if (tl == 0) { dst[0] = m_run[h] * 0.6931471805599453f; dst[1] = rb[0][h] + rb[1][h] + rb[2][h] + rb[3][h]; }
#pragma unroll
              for (int j = 0; j < kMaxDVT; ++j)
                if (j < p.DVT && j * kChunk + tl < p.Dv) dst[kPartHdr + j * kChunk + tl] = o_run[j][h];
            }
          }
        } else if (tl == 0) {
          atomicMax(p.status, kStatusBadShape);     // a sequence longer than the max_seqlen the workspace was sized for
        }
        // the CTA that reaches the end of a sequence records how many partial results its unit of the sequence has
        if (kBalanced && tl == 0 && s_walk.t + ntiles == s_walk.nb)
          p.n_slots[static_cast<long long>(bb) * U + blockIdx.x % U] = min(slot + 1, p.n_splits);
      }
      if constexpr (kBalanced) {
        g0 += ntiles;
        named_bar_sync(bar_id, 128);                 // everybody has read the walk
        if (tl == 0) {
          AttnWalk w = s_walk;
          attn_walk_advance<true>(p, w, ntiles);
          s_walk = w;
          s_slot = 0;                                // every later segment starts its sequence
        }
        named_bar_sync(bar_id, 128);
        more = s_walk.left > 0;
      } else {
        more = false;                                // a fixed split is one segment
      }
    }
  }

  tc_fence_before();
  __syncthreads();
  if (threadIdx.x == 0) attn_mark(p, 29);
  if (warp == 1) {
    tc_fence_after();
    tmem_dealloc(tmem_base, p.tmem_cols);
  }
}


// ------------------------------------------------------------------------------------------------------------------
// Wide head groups (more than 16 query rows per KV head, e.g. an MLA latent cache shared by 64 heads): 32 head slots per
// CTA, sixteen softmax warps (four groups of four; a group owns 8 head slots, a thread one token lane of them).
//
// The PV products of consecutive tiles accumulate in the SAME INT32 tensor-memory accumulators (Alg. 3 lines 10-12
// applied once per run of tiles): that needs the reference maximum of every head and the probability scale alpha_P to
// stay put between tiles, so both are HELD - the reference moves only when a score exceeds it, to that tile's maximum
// plus kHoldMarginLog2 octaves, and alpha_P = a_ref / 127 with a_ref raised to kHoldScaleGrowth times the tile's largest
// value scale when one exceeds it.  P <= 1 and P * v_scale <= a_ref hold at all times, so nothing clips.  A tile in
// which nothing is exceeded (almost all of them) costs the softmax warps no reduction and no barrier among
// themselves: scores -> exp2 -> two-pass INT8 -> shared memory.  Otherwise every warp learns it from a stamp next to
// the P buffer, the accumulators are drained into the FP32 running output with the old scales, the references move,
// and P of that tile is written again before the MMA warp may use it.
//
// (Asking for the tiles further ahead with cp.async.bulk.prefetch.tensor was measured and dropped: the two KV stages
// that fit shared memory for a 576-byte row bound the pipeline, not the latency of L2 misses.)
constexpr float kHoldMarginLog2 = 3.0f;
constexpr float kHoldScaleGrowth = 1.25f;
constexpr int kWideSlots = 32;                      // head slots per CTA, Rp = 64 stacked rows
template <int W> __device__ __forceinline__ void tmem_stw(uint32_t taddr, const uint32_t (&v)[W]) {
  static_assert(W == 8 || W == 16, "8 or 16 columns per store");
  if constexpr (W == 8) tmem_st8(taddr, v);
  else tmem_st16(taddr, v);
}


// kWideHS: head slots per softmax thread (8 or 16); the 32 slots of the CTA are shared out over 32 / kWideHS groups of
// four softmax warps.  kFixDC / kFixDVT: the chunk counts of D and Dv when known at compile time (0: taken from the
// plan) - the MMA thread shares its scheduler with four busy softmax warps, so every instruction it spends per MMA on
// loop control and address arithmetic delays the tensor pipe; with fixed counts its loops unroll to an add per operand.
template <int kWideHS, bool kPaged, int kFixDC, int kFixDVT>
__global__ void __launch_bounds__(((kFixDC == 5 && kFixDVT == 4 && !kPaged) ? 64 : 96) + 128 * (kWideSlots / kWideHS), 1)
attn_decode_wide_kernel(const __grid_constant__ CUtensorMap tmap_k, const __grid_constant__ CUtensorMap tmap_v, const AttnParams p) {
  extern __shared__ uint8_t smem_dyn[];
  __shared__ __align__(8) uint64_t kv_full[4], kv_empty[4], v_full[4], v_empty[4], s_full[2], p_full[2], q_ready, pv_done[2], p_redo;
  __shared__ uint32_t tmem_base_slot;
  __shared__ int abort_flag;
  __shared__ int flush_stamp[2];                    // tile number + 1 of the last tile whose references had to move, per P buffer
  __shared__ float s_aq[kWideSlots];
  __shared__ float red[kWideSlots / kWideHS][4][kWideHS + 1];    // per-warp tile maxima (slow path only)
  constexpr int kWideWG = kWideSlots / kWideHS;
  constexpr int kNSW = 4 * kWideWG;
  // Latent cache of 576 bytes per token with V aliased to its first 512 (the launcher picks this instantiation only
  // then): the two KV stages are given back chunk by chunk (five 128-byte-wide chunks of 16 KB): every chunk is
  // requested again as soon as its last reader is done - the rotary chunk after QK^T, value chunk j after the j-th
  // 128-wide tile of PV - instead of the whole 80 KB stage waiting for the last PV MMA.  Every chunk lands on a barrier of
  // its own and QK^T starts on a tile's first chunks while the others are in flight.  (While one thread issued both
  // products that measured slower - five short bursts cost it far more than one long one; with PV issued elsewhere
  // the thread has nothing else to do and the scores are ready 0.2-0.5 us earlier.)
  constexpr bool kChunked = kFixDC == 5 && kFixDVT == 4 && !kPaged;
  __shared__ __align__(8) uint64_t ck_empty[2][5], ck_full[2][5];      // per stage and chunk: free again / landed
  constexpr int kDVT = 4;

  const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
  // splits along x, units along y (the two head groups of a sequence split, which read the same tiles, a few CTAs apart:
  // launched side by side they miss L2 together, measured 4 us slower)
  const int split = blockIdx.x;
  int unit = blockIdx.y;
  const int grp = unit % p.groups; unit /= p.groups;
  const int hk = unit % p.Hkv;
  const int b = unit / p.Hkv;
  const int32_t* bt = kPaged ? p.block_table + static_cast<long long>(b) * p.max_blocks : nullptr;
  const int seq0 = kPaged ? 0 : p.cu[b];
  const int L = kPaged ? p.seqlens[b] : p.cu[b + 1] - seq0;
  const int t_begin = split * p.chunk;
  const int t_end = min(L, t_begin + p.chunk);
  const int h0 = hk * p.G + grp * p.HG;
  const int nh = min(p.HG, p.G - grp * p.HG);
  const int ntiles = (t_end > t_begin) ? (t_end - t_begin + kTok - 1) / kTok : 0;
  if (threadIdx.x == 0 && p.trace) {
    attn_mark(p, 0);
    unsigned long long g;
    asm volatile("mov.u64 %0, %globaltimer;" : "=l"(g));
    const int cta = blockIdx.y * gridDim.x + blockIdx.x;
    if (cta < 1024) { p.trace[cta * 32 + 1] = static_cast<long long>(g); p.trace[cta * 32 + 2] = ntiles; }
  }

  if (ntiles == 0) {      // nothing in this split: neutral partials, before any barrier or TMEM use
    for (int i = threadIdx.x; i < nh * (p.Dv + kPartHdr); i += blockDim.x) {
      const int h = i / (p.Dv + kPartHdr), e = i % (p.Dv + kPartHdr);
      float* dst = p.partial + ((static_cast<long long>(b) * p.Hq + h0 + h) * p.n_splits + split) * (p.Dv + kPartHdr);
      dst[e] = (e == 0) ? -INFINITY : 0.0f;
    }
    return;
  }

  uint8_t* smem = reinterpret_cast<uint8_t*>((reinterpret_cast<uintptr_t>(smem_dyn) + 1023) & ~static_cast<uintptr_t>(1023));
  const int kv_stage_bytes = p.kv_chunks * kChunkBytes;
  uint8_t* sm_q = smem + p.stages * kv_stage_bytes;          // DC chunks of [Rp x 128]
  uint8_t* sm_p = sm_q + p.DC * p.Rp * kChunk;               // two buffers of [Rp x 128]

  if (threadIdx.x == 0) {
    for (int s = 0; s < p.stages; ++s) {
      mbar_init(&kv_full[s], 1); mbar_init(&kv_empty[s], 1);
      mbar_init(&v_full[s], 1); mbar_init(&v_empty[s], 1);
    }
    mbar_init(&s_full[0], 1); mbar_init(&s_full[1], 1);
    mbar_init(&p_full[0], kNSW); mbar_init(&p_full[1], kNSW);
    mbar_init(&q_ready, 1);
    mbar_init(&pv_done[0], 1); mbar_init(&pv_done[1], 1); mbar_init(&p_redo, kNSW);
    if constexpr (kChunked)
      for (int s2 = 0; s2 < 2; ++s2)
        for (int c = 0; c < 5; ++c) { mbar_init(&ck_empty[s2][c], 1); mbar_init(&ck_full[s2][c], 1); }
    abort_flag = 0;
    flush_stamp[0] = 0; flush_stamp[1] = 0;
    mbar_init_fence();
    tma_prefetch_desc(&tmap_k);
    tma_prefetch_desc(&tmap_v);
  }
  if (warp == 1) tmem_alloc(&tmem_base_slot, p.tmem_cols);
  tc_fence_before();
  __syncthreads();
  tc_fence_after();
  const uint32_t tmem_base = tmem_base_slot;
  const uint32_t tmem_o = tmem_base + 2 * p.Rp;             // O^T tiles after the two S^T buffers
  volatile int* abort = &abort_flag;
  volatile int* stamp = flush_stamp;

  if (warp == 0) {
    // ------------------------------ TMA producer: K (and V) tiles ------------------------------
    if (lane == 0) {
      const int k_bytes = p.DC * kChunkBytes, v_bytes = p.DVT * kChunkBytes;
      int kq = 0, vq = p.v_alias ? ntiles : 0;
      if constexpr (kChunked) {
        bool okp = true;
        for (; kq < ntiles && okp; ++kq) {
          const int st = kq & 1;
          const uint32_t ph = (kq >> 1) & 1;
          uint8_t* dst = smem + st * kv_stage_bytes;
          const int tok0 = seq0 + t_begin + kq * kTok;
          if (kq >= 2 && kq < 5) attn_mark(p, 9 + 6 * (kq - 2));
          // Chunk by chunk as the tile two back lets go of the stage: the rotary chunk (read by QK^T only) when its
          // scores are complete (s_full of that tile: same index, same phase; a commit costs its thread about 80 ns,
          // so the rotary chunk has no barrier of its own), value chunk j when the dv tile of PV that reads it is
          // complete.  (Parity ph ^ 1 passes at once on a barrier that has not completed a phase yet.)
#pragma unroll
          for (int i = 0; i < 5; ++i) {
            const int c = (i == 0) ? 4 : i - 1;
            if (i == 0) okp = wait_bounded(&s_full[st], ph ^ 1, abort, p.status);
            else okp = wait_bounded(&ck_empty[st][c], ph ^ 1, abort, p.status);
            if (!okp) break;
            mbar_arrive_expect_tx(&ck_full[st][c], kChunkBytes);      // every chunk lands on a barrier of its own
            tma_load_3d(dst + c * kChunkBytes, &tmap_k, c * kChunk, hk, tok0, &ck_full[st][c]);
          }
        }
      }
      long long t_idle = clock64();
      while (kq < ntiles || vq < ntiles) {
        bool progressed = false;
        if (kq < ntiles && mbar_test_wait(&kv_empty[kq % p.stages], ((kq / p.stages) & 1) ^ 1)) {
          const int st = kq % p.stages;
          uint8_t* dst = smem + st * kv_stage_bytes;
          const int u0 = t_begin + kq * kTok;
          if (kq >= 2 && kq < 5) attn_mark(p, 9 + 6 * (kq - 2));
          if constexpr (!kPaged) {
            mbar_arrive_expect_tx(&kv_full[st], k_bytes);
            for (int c = 0; c < p.DC; ++c) tma_load_3d(dst + c * kChunkBytes, &tmap_k, c * kChunk, hk, seq0 + u0, &kv_full[st]);
          } else {
            const int npg = min(kTok >> p.page_shift, (t_end - u0 + p.page - 1) >> p.page_shift);
            mbar_arrive_expect_tx(&kv_full[st], p.DC * kChunk * p.page * npg);
            for (int pg = 0; pg < npg; ++pg) {
              const int tok = __ldg(bt + (u0 >> p.page_shift) + pg) * p.page;
              for (int c = 0; c < p.DC; ++c)
                tma_load_3d(dst + c * kChunkBytes + pg * p.page * kChunk, &tmap_k, c * kChunk, hk, tok, &kv_full[st]);
            }
          }
          ++kq;
          progressed = true;
        }
        if (vq < ntiles && mbar_test_wait(&v_empty[vq % p.stages], ((vq / p.stages) & 1) ^ 1)) {
          const int st = vq % p.stages;
          uint8_t* dst = smem + st * kv_stage_bytes + k_bytes;
          const int u0 = t_begin + vq * kTok;
          if constexpr (!kPaged) {
            mbar_arrive_expect_tx(&v_full[st], v_bytes);
            for (int j = 0; j < p.DVT; ++j) tma_load_3d(dst + j * kChunkBytes, &tmap_v, j * kChunk, hk, seq0 + u0, &v_full[st]);
          } else {
            const int npg = min(kTok >> p.page_shift, (t_end - u0 + p.page - 1) >> p.page_shift);
            mbar_arrive_expect_tx(&v_full[st], p.DVT * kChunk * p.page * npg);
            for (int pg = 0; pg < npg; ++pg) {
              const int tok = __ldg(bt + (u0 >> p.page_shift) + pg) * p.page;
              for (int j = 0; j < p.DVT; ++j)
                tma_load_3d(dst + j * kChunkBytes + pg * p.page * kChunk, &tmap_v, j * kChunk, hk, tok, &v_full[st]);
            }
          }
          ++vq;
          progressed = true;
        }
        if (progressed) {
          t_idle = clock64();
        } else {
          if (*abort) break;
          if (clock64() - t_idle > kWaitBudgetCycles) {
            *abort = 1;
            atomicMax(p.status, kStatusTimeout);
            break;
          }
        }
      }
    }
  } else if (warp == 1) {
    // ------------------------------ MMA issuer ------------------------------
    if (lane == 0) {
      const uint32_t idesc_qk = idesc_dense(2, 1, 1, 0, 0, kTok, p.Rp);     // S8 x S8 -> S32, both K-major
      const uint32_t idesc_pv = idesc_dense(2, 1, 1, 1, 1, kTok, p.Rp);     // A (V^T) and B (P) MN-major
      bool ok = true;
      // the stacked Q operand of this (sequence, KV head, head group) comes ready-made from attn_qstack_kernel, the
      // kernel launched just before this one (the producer's KV loads, which do not depend on it, are already under way)
      pdl_wait_primary();
      {
        const int unit_q = blockIdx.y, chunk_bytes = p.Rp * kChunk;
        mbar_arrive_expect_tx(&q_ready, p.DC * chunk_bytes);
        for (int c = 0; c < p.DC; ++c)
          bulk_load(sm_q + c * chunk_bytes, p.q_img + (static_cast<size_t>(unit_q) * p.DC + c) * chunk_bytes, chunk_bytes, &q_ready);
      }
      ok = wait_bounded(&q_ready, 0, abort, p.status);
      const uint64_t dk = smem_desc(0, 16, 1024, kSwizzle128B);         // K-major tiles: K, stacked Q
      const uint64_t dvt = smem_desc(0, 16384, 1024, kSwizzle128B);     // V^T read MN-major from the token-major tile
      const uint64_t q_enc = dk + (smem_u32(sm_q) >> 4);
      // P lies token-major, [128 tokens][64 bytes = 2 x 32 head slots], 64-byte swizzle: an MN-major B operand whose
      // groups of 8 tokens are 512 bytes apart (a softmax thread then stores its token's codes as whole words)
      const uint64_t p_enc = smem_desc(0, 512, 512, kSwizzle64B) + (smem_u32(sm_p) >> 4);
      const uint32_t smem_enc = smem_u32(smem) >> 4;
      const uint32_t q_step = static_cast<uint32_t>(p.Rp * kChunk) >> 4;
      const int nDC = kFixDC ? kFixDC : p.DC;
      // 32-byte K steps of the last chunk of D that hold data (the stacked Q operand is zero past D)
      const int last_steps = (p.D - (nDC - 1) * kChunk + 31) >> 5;
      auto issue_qk = [&](int t) {
        const int st = t % p.stages;
        tc_fence_after();
        const uint64_t ka = dk + smem_enc + static_cast<uint32_t>(st * (kv_stage_bytes >> 4));
        const uint32_t d = tmem_base + (t & 1) * p.Rp;
        if constexpr (kFixDC > 0) {
          // (address fields never carry out of the descriptors' lower words: shared memory is 227 KB, the field counts 16 bytes)
          const uint32_t ka_lo = static_cast<uint32_t>(ka), k_hi = static_cast<uint32_t>(ka >> 32);
          const uint32_t qa_lo = static_cast<uint32_t>(q_enc), q_hi = static_cast<uint32_t>(q_enc >> 32);
#pragma unroll
          for (int c = 0; c < kFixDC; ++c)
#pragma unroll
            for (int k = 0; k < 4; ++k)
              if (c + 1 < kFixDC || k < last_steps) {
                if (c > 0 || k > 0)
                  mma_i8_lohi<true>(d, ka_lo + (c * (kChunkBytes >> 4) + 2 * k), k_hi, qa_lo + (c * ((kWideSlots * 2 * kChunk) >> 4) + 2 * k), q_hi, idesc_qk);
                else
                  mma_i8_lohi<false>(d, ka_lo, k_hi, qa_lo, q_hi, idesc_qk);
              }
        } else {
          uint64_t kc = ka, qa = q_enc;
          for (int c = 0; c < nDC; ++c) {
#pragma unroll
            for (int k = 0; k < 4; ++k)
              if (c + 1 < nDC || k < last_steps) mma_i8(d, kc + 2 * k, qa + 2 * k, idesc_qk, (c > 0 || k > 0) ? 1u : 0u);
            kc += kChunkBytes >> 4;
            qa += q_step;
          }
        }
        tc_commit(&s_full[t & 1]);
        if constexpr (kChunked) { /* the producer takes s_full as "the rotary chunk has been read" */ }
        else if (!p.v_alias) tc_commit(&kv_empty[st]);       // separate V: the K buffer is free once QK^T has read it
      };
      // PV is issued by softmax threads (below), one dv tile each; this thread issues QK^T only.
      int q = 0;
      if constexpr (kChunked) {
        // PV is issued by four softmax threads (below); this thread issues QK^T only.  QK^T(q) needs KV tile q in shared
        // memory and the score buffer q&1 read, i.e. P of tile q-2 written by every softmax warp (the slow path works
        // from registers).  The P buffer q&1 is free by then as well: KV tile q arrives in the stage that PV(q-2) gave
        // back chunk by chunk, so its arrival implies that PV(q-2) is complete.
        // The K steps of a chunk are issued as soon as that chunk has landed, in the order the chunks are requested
        // (rotary chunk first: it was free long before the value chunks): by the time the last chunk arrives only its
        // own four MMAs are left to run.
        const uint32_t k_hi = static_cast<uint32_t>(dk >> 32), q_hi = static_cast<uint32_t>(q_enc >> 32);
        const uint32_t k_lo0 = static_cast<uint32_t>(dk) + smem_enc, q_lo0 = static_cast<uint32_t>(q_enc);
        for (; q < ntiles && ok; ++q) {
          const int st = q & 1;
          const uint32_t ph = (q >> 1) & 1;
          if (q >= 2) ok = wait_bounded(&p_full[q & 1], ((q - 2) >> 1) & 1, abort, p.status);
          if (!ok) break;
          const uint32_t d = tmem_base + (q & 1) * p.Rp;
          const uint32_t k_lo = k_lo0 + static_cast<uint32_t>(st * (kv_stage_bytes >> 4));
#pragma unroll
          for (int i = 0; i < 5; ++i) {
            const int c = (i == 0) ? 4 : i - 1;
            ok = wait_bounded(&ck_full[st][c], ph, abort, p.status);
            if (!ok) break;
            if (i == 0 && q >= 2 && q < 5) attn_mark(p, 7 + 6 * (q - 2));
            tc_fence_after();
#pragma unroll
            for (int k = 0; k < 4; ++k)
              if (c < 4 || k < last_steps) {
                const uint32_t ka = k_lo + (c * (kChunkBytes >> 4) + 2 * k), qa = q_lo0 + (c * ((kWideSlots * 2 * kChunk) >> 4) + 2 * k);
                if (i == 0 && k == 0) mma_i8_lohi<false>(d, ka, k_hi, qa, q_hi, idesc_qk);
                else mma_i8_lohi<true>(d, ka, k_hi, qa, q_hi, idesc_qk);
              }
          }
          if (!ok) break;
          tc_commit(&s_full[q & 1]);
          if (q >= 2 && q < 5) attn_mark(p, q == 4 ? 30 : 23 + q);
        }
      } else {
        // QK^T(q) needs KV tile q in shared memory and the score buffer q&1 read (P of tile q-2 written by every softmax
        // warp; the slow path works from registers).  PV is issued by a warp of its own (below); that PV(q-2) has read
        // the P buffer before P of tile q is written there is the softmax warps' wait on pv_done.
        for (; q < ntiles && ok; ++q) {
          if (q >= 2) ok = wait_bounded(&p_full[q & 1], ((q - 2) >> 1) & 1, abort, p.status);
          if (ok) ok = wait_bounded(&kv_full[q % p.stages], (q / p.stages) & 1, abort, p.status);
          if (!ok) break;
          if (q >= 2 && q < 5) attn_mark(p, 7 + 6 * (q - 2));
          issue_qk(q);
          if (q >= 2 && q < 5) attn_mark(p, q == 4 ? 30 : 23 + q);
        }
      }
    }
  } else if (warp == 2 + kNSW) {
    // ------------------------------ PV issuer (rows whose tiles are not handled chunk by chunk) ------------------------------
    // A warp of its own: one thread issuing QK^T and PV alike was never idle (1.7 us per tile at D = Dv = 128 for 8 MMAs,
    // 4 commits and its polling, everything else waiting for it), and a softmax thread issuing PV puts it on the
    // softmax warps' critical path.
    if constexpr (!kChunked) {
      if (lane == 0) {
        const uint64_t vdesc = smem_desc(0, 16384, 1024, kSwizzle128B) + (smem_u32(smem) >> 4);       // V^T, MN-major from the token-major tile
        const uint64_t pdesc = smem_desc(0, 512, 512, kSwizzle64B) + (smem_u32(sm_p) >> 4);           // P, token-major
        const uint32_t va0 = static_cast<uint32_t>(vdesc), v_hi = static_cast<uint32_t>(vdesc >> 32);
        const uint32_t pa0 = static_cast<uint32_t>(pdesc), p_hi = static_cast<uint32_t>(pdesc >> 32);
        const uint32_t p_step = static_cast<uint32_t>(p.Rp * kChunk) >> 4;
        const uint32_t idesc = idesc_dense(2, 1, 1, 1, 1, kTok, p.Rp);     // S8 x S8 -> S32, A (V^T) and B (P) MN-major
        const int n_dvt = kFixDVT ? kFixDVT : p.DVT;
        bool ok = true;
        int n_slow = 0;
        for (int t = 0; t < ntiles && ok; ++t) {
          const int st = t % p.stages;
          // P of tile t final: written by every softmax warp and, when the references had to move, written again
          ok = wait_bounded(&p_full[t & 1], (t >> 1) & 1, abort, p.status);
          bool fresh = false;
          if (ok && stamp[t & 1] == t + 1) {
            ok = wait_bounded(&p_redo, n_slow & 1, abort, p.status);
            ++n_slow;
            fresh = true;                          // the accumulators were drained: start them again
          }
          if (ok) ok = wait_bounded(p.v_alias ? &kv_full[st] : &v_full[st], (t / p.stages) & 1, abort, p.status);     // the value tile
          if (!ok) break;
          tc_fence_after();
          if (t >= 2 && t < 5) attn_mark(p, 8 + 6 * (t - 2));
          const uint32_t va = va0 + static_cast<uint32_t>(st * (kv_stage_bytes >> 4)) + (p.v_alias ? 0u : static_cast<uint32_t>(p.DC * (kChunkBytes >> 4)));
          const uint32_t pa = pa0 + (t & 1) * p_step;
          for (int j = 0; j < n_dvt; ++j) {
            const uint32_t acc = tmem_o + j * (2 * kWideSlots);
            if (fresh) mma_i8_lohi<false>(acc, va + j * (kChunkBytes >> 4), v_hi, pa, p_hi, idesc);
            else mma_i8_lohi<true>(acc, va + j * (kChunkBytes >> 4), v_hi, pa, p_hi, idesc);
#pragma unroll
            for (int k = 1; k < 4; ++k)      // 32 tokens per MMA: four 8-token groups of 1024 bytes
              mma_i8_lohi<true>(acc, va + j * (kChunkBytes >> 4) + k * (4096 >> 4), v_hi, pa + k * (2048 >> 4), p_hi, idesc);
          }
          tc_commit(&pv_done[t & 1]);
          tc_commit(p.v_alias ? &kv_empty[st] : &v_empty[st]);
          if (t >= 2 && t < 5) attn_mark(p, 20 + t);
        }
      }
    }
  } else {
    // ------------------------------ softmax warps ------------------------------
    const int quad = warp & 3;
    const int tl = quad * 32 + lane;                // token lane (softmax) / dv lane (drain)
    const int wi = warp - 2;                        // 0 .. 15
    const int hh = wi >> 2;                         // which group of head slots this warp looks after
    const int wq = wi & 3;
    const int hs0 = hh * kWideHS;                   // its first head slot
    {
      // alpha_Q of this CTA's heads, computed by attn_qstack_kernel (launched just before this kernel);
      // beta_Q = alpha_Q / 254 is applied as a constant factor
      pdl_wait_primary();
      const int i = threadIdx.x - 64;
      const float* sc = p.q_scales + static_cast<size_t>(blockIdx.y) * 2 * p.HG;
      if (i < kWideSlots) s_aq[i] = __ldg(sc + i);
    }
    named_bar_sync(8, 128 * kWideWG);
    if (threadIdx.x == 64) attn_mark(p, 3);
    const int bar_id = 1 + hh;

    // Per head slot: query scale, NEGATED reference maximum in the log2 domain (+1e30 while no score has been seen,
    // -1e30 for a slot without a head, so that "score + nm > 0" means "exceeds the reference"), partial sum of P over
    // this thread's tokens.  The FP32 running output of this thread's dv lane (4 x 8 values) lives in the tensor-memory
    // columns behind the accumulators: it is touched only by the rare drains, and 32 registers fewer per thread let
    // the compiler keep the eight heads' dependent chains of the per-tile code in flight side by side.
    float aq[kWideHS], nm[kWideHS], l_part[kWideHS];
    const uint32_t orun_row = tmem_o + kDVT * p.Rp + (static_cast<uint32_t>(quad * 32) << 16) + hs0;
#pragma unroll
    for (int h = 0; h < kWideHS; ++h) {
      const bool present = hs0 + h < nh;
      aq[h] = present ? s_aq[hs0 + h] : 0.0f;
      nm[h] = present ? 1e30f : -1e30f;
      l_part[h] = 0.0f;
    }
    {
      uint32_t z[kWideHS];
#pragma unroll
      for (int h = 0; h < kWideHS; ++h) z[h] = 0u;
#pragma unroll
      for (int j = 0; j < kDVT; ++j) tmem_stw<kWideHS>(orun_row + j * kWideSlots, z);
      tmem_st_wait();
    }
    float a_ref = 0.0f, alpha_p = 0.0f, inv_a = 0.0f, inv_b = 0.0f;
    const float kLog2e = 1.4426950408889634f;
    const float scale2 = p.scale * kLog2e;
    const float kInv254 = 1.0f / 254.0f;
    const float kMagic = 12582912.0f;

    auto load_scales = [&](int t, float& ks_out, float& vs_out) {
      const int tok_rel = t_begin + t * kTok + tl;
      const bool valid = t < ntiles && tok_rel < t_end;
      long long sidx;
      if constexpr (kPaged) {
        const long long prow = valid ? static_cast<long long>(__ldg(bt + (tok_rel >> p.page_shift))) * p.page + (tok_rel & (p.page - 1)) : 0;
        sidx = prow * p.Hkv + hk;
      } else {
        sidx = static_cast<long long>(seq0 + tok_rel) * p.Hkv + hk;
      }
      ks_out = valid ? __ldg(p.k_scale + sidx) : 0.0f;
      vs_out = valid ? __ldg(p.v_scale + sidx) : 0.0f;
    };
    // c3: scores of this thread's token against its 8 head slots in the log2 domain (-inf where the token is past the
    // end of the split or not visible to the row)
    auto load_scores = [&](int t, float ks, float (&s)[kWideHS]) {
      const int tok_rel = t_begin + t * kTok + tl;
      const bool valid = tok_rel < t_end;
      const uint32_t srow = tmem_base + (static_cast<uint32_t>(quad * 32) << 16) + (t & 1) * p.Rp;
      uint32_t v1[kWideHS], v2[kWideHS];
      tmem_ldw<kWideHS>(srow + hs0, v1);
      tmem_ldw<kWideHS>(srow + kWideSlots + hs0, v2);
      tmem_ld_wait();
      if (p.s_dbg && valid) {
        long long tok_row = seq0 + tok_rel;
        if constexpr (kPaged) tok_row = static_cast<long long>(__ldg(bt + (tok_rel >> p.page_shift))) * p.page + (tok_rel & (p.page - 1));
        attn_dump_scores<kWideHS>(p, tok_row, hk, grp, hs0, nh, v1, v2);
      }
#pragma unroll
      for (int h = 0; h < kWideHS; ++h) {
        bool vh = valid;
        if (p.Sq > 1) vh = valid && tok_rel < L - p.Sq + 1 + (grp * p.HG + hs0 + h) / p.Gr;    // causal among the new tokens
        const float tsum = __fmaf_rn(static_cast<float>(static_cast<int32_t>(v2[h])), kInv254, static_cast<float>(static_cast<int32_t>(v1[h])));
        s[h] = vh ? (aq[h] * ks) * tsum : -INFINITY;
      }
    };
    // c4-c5: P = 2^(s - reference), value scale folded in, two-pass INT8 with the scale in force, into P buffer t&1.
    // Returns the largest s - reference of this thread (> 0: the reference must move).
    auto write_p = [&](int t, const float (&s)[kWideHS], float vs, float (&pl)[kWideHS]) -> float {
      // this token's row of the P buffer: 64 bytes, the 16-byte pieces XORed with (token / 2) % 4 (64-byte swizzle)
      uint8_t* prow = sm_p + (t & 1) * p.Rp * kChunk + tl * 64;
      const int sw = (tl >> 1) & 3;
      uint32_t c1[kWideHS], c2[kWideHS];
      float xm = -INFINITY;
#pragma unroll
      for (int h = 0; h < kWideHS; ++h) {
        const float x = s[h] + nm[h];
        xm = fmaxf(xm, x);
        const float pr = ex2_approx(x);
        pl[h] = pr;
        const float pt = pr * vs;
        // 1.5 * 2^23 trick: the rounded integer lands in the low mantissa bits (P <= 1, v_scale <= a_ref: no clamps)
        const float u1 = __fmaf_rn(pt, inv_a, kMagic);
        const float r = __fmaf_rn(-alpha_p, u1 - kMagic, pt);
        const float u2 = __fmaf_rn(r, inv_b, kMagic);
        c1[h] = __float_as_uint(u1);
        c2[h] = __float_as_uint(u2);
      }
      // the codes are the low bytes; kWideHS of them make one 8- or 16-byte store per component
      uint32_t w1[kWideHS / 4], w2[kWideHS / 4];
#pragma unroll
      for (int g = 0; g < kWideHS / 4; ++g) {
        w1[g] = __byte_perm(__byte_perm(c1[4 * g], c1[4 * g + 1], 0x0040), __byte_perm(c1[4 * g + 2], c1[4 * g + 3], 0x0040), 0x5410);
        w2[g] = __byte_perm(__byte_perm(c2[4 * g], c2[4 * g + 1], 0x0040), __byte_perm(c2[4 * g + 2], c2[4 * g + 3], 0x0040), 0x5410);
      }
      uint8_t* d1 = prow + ((((hs0 >> 4) ^ sw) & 3) << 4) + (hs0 & 15);
      uint8_t* d2 = prow + (((((kWideSlots + hs0) >> 4) ^ sw) & 3) << 4) + (hs0 & 15);
      if constexpr (kWideHS == 8) {
        *reinterpret_cast<uint2*>(d1) = make_uint2(w1[0], w1[1]);
        *reinterpret_cast<uint2*>(d2) = make_uint2(w2[0], w2[1]);
      } else {
        *reinterpret_cast<uint4*>(d1) = make_uint4(w1[0], w1[1], w1[2], w1[3]);
        *reinterpret_cast<uint4*>(d2) = make_uint4(w2[0], w2[1], w2[2], w2[3]);
      }
      return xm;
    };
    // Alg. 3 line 12 for everything accumulated since the last drain: O <- (O + alpha_P (O1 + O2 / 254)) * resc
    auto drain = [&](const float (&resc)[kWideHS], float alpha_old) {
#pragma unroll
      for (int j = 0; j < kDVT; ++j) {
        if (j < p.DVT) {
          const uint32_t orow = tmem_o + (static_cast<uint32_t>(quad * 32) << 16) + j * p.Rp;
          uint32_t v1[kWideHS], v2[kWideHS], o[kWideHS];
          tmem_ldw<kWideHS>(orow + hs0, v1);
          tmem_ldw<kWideHS>(orow + kWideSlots + hs0, v2);
          tmem_ldw<kWideHS>(orun_row + j * kWideSlots, o);
          tmem_ld_wait();
#pragma unroll
          for (int h = 0; h < kWideHS; ++h) {
            const float acc = __fmaf_rn(static_cast<float>(static_cast<int32_t>(v2[h])), kInv254, static_cast<float>(static_cast<int32_t>(v1[h])));
            // the drained sums belong to the OLD reference: add them, then rescale
            o[h] = __float_as_uint(__fmaf_rn(alpha_old, acc, __uint_as_float(o[h])) * resc[h]);
          }
          tmem_stw<kWideHS>(orun_row + j * kWideSlots, o);
        }
      }
      tmem_st_wait();
    };

    // operand descriptors of PV as lower / upper words (see mma_i8_lohi): V^T read MN-major from the token-major KV tile,
    // P an MN-major operand too (token-major, 64-byte swizzle, groups of 8 tokens 512 bytes apart)
    const uint64_t pv_vdesc = smem_desc(0, 16384, 1024, kSwizzle128B) + (smem_u32(smem) >> 4);
    const uint64_t pv_pdesc = smem_desc(0, 512, 512, kSwizzle64B) + (smem_u32(sm_p) >> 4);
    const uint32_t pv_va_lo = static_cast<uint32_t>(pv_vdesc), pv_v_hi = static_cast<uint32_t>(pv_vdesc >> 32);
    const uint32_t pv_pa_lo = static_cast<uint32_t>(pv_pdesc), pv_p_hi = static_cast<uint32_t>(pv_pdesc >> 32);
    const uint32_t pv_p_step = static_cast<uint32_t>(p.Rp * kChunk) >> 4;
    const uint32_t pv_idesc = idesc_dense(2, 1, 1, 1, 1, kTok, p.Rp);     // S8 x S8 -> S32, A (V^T) and B (P) MN-major

    bool ok = true;
    int n_slow = 0;
    // this warp's group of head slots holds at least one head (the kernel for 576-byte rows, where every instruction
    // in the tile loop counts and all 32 slots are normally in use, is compiled without the distinction)
    const bool active = kChunked ? true : hs0 < nh;
    float ks_pre, vs_pre;
    load_scales(0, ks_pre, vs_pre);
    for (int t = 0; t < ntiles && ok; ++t) {
      const float ks = ks_pre * scale2, vs = vs_pre;
      load_scales(t + 1, ks_pre, vs_pre);
      ok = wait_bounded(&s_full[t & 1], (t >> 1) & 1, abort, p.status);
      if (!ok) break;
      if (threadIdx.x == 64 && t >= 2 && t < 5) attn_mark(p, 4 + 6 * (t - 2));
      tc_fence_after();
      float s[kWideHS], pl[kWideHS];
      if (active) {
        load_scores(t, ks, s);
        if constexpr (!kChunked) {
          // the P buffer t&1 was the operand of PV(t-2), issued by another thread than QK^T(t): its completion is not implied
          if (t >= 2) ok = wait_bounded(&pv_done[t & 1], ((t - 2) >> 1) & 1, abort, p.status);
          if (!ok) break;
        }
        const float xm = write_p(t, s, vs, pl);
        const bool exceeded = __any_sync(0xffffffffu, xm > 0.0f || vs > a_ref);
        if (exceeded && lane == 0) stamp[t & 1] = t + 1;
      } else {
        // a group of head slots without a head (9 to 24 rows per KV head): nothing to compute, but the barriers count
        // every softmax warp; its P columns keep whatever codes they hold and its accumulator columns are never read
#pragma unroll
        for (int h = 0; h < kWideHS; ++h) pl[h] = 0.0f;
      }
      fence_proxy_async_smem();
      tc_fence_before();
      __syncwarp();
      if (lane == 0) mbar_arrive(&p_full[t & 1]);
      if (threadIdx.x == 64 && t >= 2 && t < 5) attn_mark(p, 5 + 6 * (t - 2));
      // every softmax warp has written its part (and said whether it saw a reference exceeded): did any have to move?
      ok = wait_bounded(&p_full[t & 1], (t >> 1) & 1, abort, p.status);
      if (!ok) break;
      if (threadIdx.x == 64 && t >= 2 && t < 5) attn_mark(p, 6 + 6 * (t - 2));
      bool slow = false;
      if (!active) {
        if (stamp[t & 1] == t + 1) {      // the other groups drain and write P again: be counted among the warps that are done
          __syncwarp();
          if (lane == 0) mbar_arrive(&p_redo);
          ++n_slow;
          slow = true;
        }
      } else if (stamp[t & 1] == t + 1) {
        // ---- the references move: tile maxima per head over the group's 128 tokens, largest value scale ----
#pragma unroll
        for (int h = 0; h < kWideHS; ++h) {
          const float wm = warp_max(s[h]);
          if (lane == 0) red[hh][wq][h] = wm;
        }
        {
          const float wv = warp_max(vs);
          if (lane == 0) red[hh][wq][kWideHS] = wv;
        }
        named_bar_sync(bar_id, 128);
        float resc[kWideHS];
#pragma unroll
        for (int h = 0; h < kWideHS; ++h) {
          const float tmax = fmaxf(fmaxf(red[hh][0][h], red[hh][1][h]), fmaxf(red[hh][2][h], red[hh][3][h]));
          resc[h] = 1.0f;
          if (hs0 + h < nh && tmax + nm[h] > 0.0f) {
            const float m_new = tmax + kHoldMarginLog2;
            resc[h] = (nm[h] == 1e30f) ? 0.0f : ex2_approx(-nm[h] - m_new);
            nm[h] = -m_new;
          }
        }
        const float vmax = fmaxf(fmaxf(red[hh][0][kWideHS], red[hh][1][kWideHS]), fmaxf(red[hh][2][kWideHS], red[hh][3][kWideHS]));
        const float alpha_old = alpha_p;
        if (vmax > a_ref) {
          a_ref = vmax * kHoldScaleGrowth;
          alpha_p = a_ref * (1.0f / 127.0f);
          inv_a = __frcp_rn(alpha_p);
          inv_b = 254.0f * inv_a;
        }
        if (t > 0) {
          // everything accumulated so far was scaled by the old references: PV(t-1) and all before it are complete
          if constexpr (kChunked) {
#pragma unroll
            for (int j = 0; j < 4; ++j) ok = ok && wait_bounded(&ck_empty[(t - 1) & 1][j], ((t - 1) >> 1) & 1, abort, p.status);
          } else {
            ok = wait_bounded(&pv_done[(t - 1) & 1], ((t - 1) >> 1) & 1, abort, p.status);
          }
          if (!ok) break;
          tc_fence_after();
          drain(resc, alpha_old);
#pragma unroll
          for (int h = 0; h < kWideHS; ++h) l_part[h] *= resc[h];
        }
        write_p(t, s, vs, pl);
        fence_proxy_async_smem();
        tc_fence_before();
        __syncwarp();
        if (lane == 0) mbar_arrive(&p_redo);
        ++n_slow;
        named_bar_sync(bar_id, 128);          // `red` may be rewritten
        slow = true;
      }
      if constexpr (kChunked) {
        // PV(t), one dv tile per thread: lane 0 of the first four softmax warps, which sit on the four different warp
        // schedulers.  The softmax warps are idle here (the next score tile is not there yet), the product starts the
        // moment P is final instead of when the QK^T-issuing thread gets round to it, and its 16 MMAs are issued four
        // abreast.  An accumulator is only ever written by its own thread, so its MMAs stay in program order.
        if (hh == 0 && lane == 0) {
          const int st = t & 1;
          if (slow) ok = wait_bounded(&p_redo, (n_slow - 1) & 1, abort, p.status);      // every warp has drained and rewritten P
          if (ok) ok = wait_bounded(&ck_full[st][wq], (t >> 1) & 1, abort, p.status);      // its value chunk (long landed: QK^T(t) has read the tile)
          if (ok) {
            tc_fence_after();
            if (wq == 0 && t >= 2 && t < 5) attn_mark(p, 8 + 6 * (t - 2));
            const uint32_t va_lo = pv_va_lo + static_cast<uint32_t>(st * (kv_stage_bytes >> 4)) + wq * (kChunkBytes >> 4);
            const uint32_t pa_lo = pv_pa_lo + (t & 1) * pv_p_step;
            const uint32_t acc = tmem_o + wq * (2 * kWideSlots);
            if (slow) mma_i8_lohi<false>(acc, va_lo, pv_v_hi, pa_lo, pv_p_hi, pv_idesc);
            else mma_i8_lohi<true>(acc, va_lo, pv_v_hi, pa_lo, pv_p_hi, pv_idesc);
#pragma unroll
            for (int k = 1; k < 4; ++k)      // 32 tokens per MMA: four 8-token groups of 1024 bytes
              mma_i8_lohi<true>(acc, va_lo + k * (4096 >> 4), pv_v_hi, pa_lo + k * (2048 >> 4), pv_p_hi, pv_idesc);
            tc_commit(&ck_empty[st][wq]);      // value chunk wq may be requested again; also "this dv tile of PV(t) is complete"
            if (wq == 0 && t >= 2 && t < 5) attn_mark(p, 20 + t);
          }
        }
        ok = __shfl_sync(0xffffffffu, ok ? 1 : 0, 0) != 0;
      }
#pragma unroll
      for (int h = 0; h < kWideHS; ++h) l_part[h] += pl[h];
    }
    if (ok) {
      // what the accumulators still hold
      if constexpr (kChunked) {
#pragma unroll
        for (int j = 0; j < 4; ++j) ok = ok && wait_bounded(&ck_empty[(ntiles - 1) & 1][j], ((ntiles - 1) >> 1) & 1, abort, p.status);
      } else {
        ok = wait_bounded(&pv_done[(ntiles - 1) & 1], ((ntiles - 1) >> 1) & 1, abort, p.status);
      }
      if (ok && active) {
        tc_fence_after();
        float one[kWideHS];
#pragma unroll
        for (int h = 0; h < kWideHS; ++h) one[h] = 1.0f;
        drain(one, alpha_p);
      }
    }
    if (threadIdx.x == 64) { attn_mark(p, 28); if (p.trace && blockIdx.y * gridDim.x + blockIdx.x < 1024) p.trace[(blockIdx.y * gridDim.x + blockIdx.x) * 32 + 27] = n_slow; }
    // partial results of this split: reference maximum, sum of P and unnormalised output per head
    if (ok) {
#pragma unroll
      for (int h = 0; h < kWideHS; ++h) {
        float l = l_part[h];
#pragma unroll
        for (int o = 16; o > 0; o >>= 1) l += __shfl_xor_sync(0xffffffffu, l, o);
        if (lane == 0) red[hh][wq][h] = l;
      }
      named_bar_sync(bar_id, 128);
#pragma unroll
      for (int h = 0; h < kWideHS; ++h) {
        if (hs0 + h < nh) {
          float* dst = p.partial + ((static_cast<long long>(b) * p.Hq + h0 + hs0 + h) * p.n_splits + split) * (p.Dv + kPartHdr);
          if (tl == 0) {
            // the reference goes out in natural-log units (it was kept in the log2 domain); -inf: no visible token
            dst[0] = (nm[h] == 1e30f) ? -INFINITY : -nm[h] * 0.6931471805599453f;
            dst[1] = red[hh][0][h] + red[hh][1][h] + red[hh][2][h] + red[hh][3][h];
          }
        }
      }
#pragma unroll
      for (int j = 0; j < kDVT; ++j) {
        if (j < p.DVT) {            // (warp-uniform: the tensor-memory load is a whole-warp instruction)
          uint32_t o[kWideHS];
          tmem_ldw<kWideHS>(orun_row + j * kWideSlots, o);
          tmem_ld_wait();
#pragma unroll
          for (int h = 0; h < kWideHS; ++h)
            if (hs0 + h < nh && j * kChunk + tl < p.Dv)
              p.partial[((static_cast<long long>(b) * p.Hq + h0 + hs0 + h) * p.n_splits + split) * (p.Dv + kPartHdr) + kPartHdr + j * kChunk + tl] =
                  __uint_as_float(o[h]);
        }
      }
    }
  }

  tc_fence_before();
  __syncthreads();
  if (threadIdx.x == 0) attn_mark(p, 29);
  if (warp == 1) {
    tc_fence_after();
    tmem_dealloc(tmem_base, p.tmem_cols);
  }
}

static long long* g_attn_trace = nullptr;
static int8_t* g_attn_q_dbg = nullptr;
static float* g_attn_qs_dbg = nullptr;
static int32_t* g_attn_s_dbg = nullptr;

// c8: merge the splits of one (sequence, query head) and normalise:  O = sum_s e^{m_s - m} O_s / sum_s e^{m_s - m} l_s
// (a separate small kernel: letting the last-arriving split do it inside the attention kernel measured slower).
// One CTA per row; the weights e^{m_s - m} are computed once per split and the O_s rows are read as 16-byte vectors,
// eight splits' loads in flight per thread.  O is summed over the splits in ascending order.
__global__ void __launch_bounds__(128)
attn_combine_kernel(const float* __restrict__ partial, int n_splits_alloc, const int32_t* __restrict__ n_slots, int G, int HG,
                    int groups, int Dv, __nv_bfloat16* __restrict__ out, float* __restrict__ lse, int Sq, int Gr, int Hkv) {
  __shared__ float s_w[128];
  __shared__ float s_red[2][4];
  pdl_wait_primary();              // the partial results come from the attention kernel launched just before
  const int PS = Dv + kPartHdr;
  const float* base = partial + static_cast<long long>(blockIdx.x) * n_splits_alloc * PS;
  // balanced schedule: only the first n_slots[unit] partial results of the row exist (unit = (sequence, KV head, head
  // group) of the row; rows are [B][KV head][G rows], HG rows per group)
  int n_splits = n_splits_alloc;
  if (n_slots) {
    const long long kvh = blockIdx.x / G;
    const int r = static_cast<int>(blockIdx.x - kvh * G);
    n_splits = min(n_splits_alloc, __ldg(n_slots + kvh * groups + r / HG));
  }
  // partial rows are [B][KV head][query token][head of the group]; the output is [B][query token][head]
  long long row = blockIdx.x;
  if (Sq > 1) {
    const int per_kv = Sq * Gr, per_seq = Hkv * per_kv;
    const long long bq = row / per_seq;
    const int v = static_cast<int>(row - bq * per_seq), hk = v / per_kv, r = v - hk * per_kv, sq = r / Gr;
    row = (bq * Sq + sq) * (Hkv * Gr) + hk * Gr + (r - sq * Gr);
  }
  const int tid = threadIdx.x, warp = tid >> 5, lane = tid & 31;
  float m = -INFINITY;
  for (int s = tid; s < n_splits; s += 128) m = fmaxf(m, __ldg(base + static_cast<long long>(s) * PS));
#pragma unroll
  for (int o = 16; o > 0; o >>= 1) m = fmaxf(m, __shfl_xor_sync(0xffffffffu, m, o));
  if (lane == 0) s_red[0][warp] = m;
  __syncthreads();
  m = fmaxf(fmaxf(s_red[0][0], s_red[0][1]), fmaxf(s_red[0][2], s_red[0][3]));
  const bool act = tid < (Dv >> 2);
  const float4* o4 = reinterpret_cast<const float4*>(base + kPartHdr) + tid;
  const int ps4 = PS >> 2;
  float4 acc = make_float4(0.0f, 0.0f, 0.0f, 0.0f);
  float l = 0.0f;                  // this thread's share of the normaliser: the splits s with s % 128 == tid
  for (int s0 = 0; s0 < n_splits; s0 += 128) {
    float w = 0.0f;
    if (s0 + tid < n_splits) {
      const float2 ml = __ldg(reinterpret_cast<const float2*>(base + static_cast<long long>(s0 + tid) * PS));
      if (ml.x != -INFINITY) { w = expf(ml.x - m); l += w * ml.y; }
    }
    __syncthreads();               // the previous chunk's weights have been used
    s_w[tid] = w;
    __syncthreads();
    const int n = min(128, n_splits - s0);
    if (act) {
      const float4* q = o4 + static_cast<long long>(s0) * ps4;
#pragma unroll 8
      for (int i = 0; i < n; ++i) {
        const float4 v = __ldg(q + static_cast<long long>(i) * ps4);
        const float wi = s_w[i];
        acc.x += wi * v.x; acc.y += wi * v.y; acc.z += wi * v.z; acc.w += wi * v.w;
      }
    }
  }
#pragma unroll
  for (int o = 16; o > 0; o >>= 1) l += __shfl_xor_sync(0xffffffffu, l, o);
  if (lane == 0) s_red[1][warp] = l;
  __syncthreads();
  l = (s_red[1][0] + s_red[1][1]) + (s_red[1][2] + s_red[1][3]);
  if (act) {
    const float o0 = l > 0.0f ? acc.x / l : 0.0f, o1 = l > 0.0f ? acc.y / l : 0.0f;
    const float o2 = l > 0.0f ? acc.z / l : 0.0f, o3 = l > 0.0f ? acc.w / l : 0.0f;
    const __nv_bfloat162 lo = __floats2bfloat162_rn(o0, o1), hi = __floats2bfloat162_rn(o2, o3);
    uint2 pk;
    pk.x = *reinterpret_cast<const uint32_t*>(&lo);
    pk.y = *reinterpret_cast<const uint32_t*>(&hi);
    *reinterpret_cast<uint2*>(out + row * Dv + 4 * tid) = pk;
  }
  if (lse && tid == 0) lse[row] = (l > 0.0f) ? m + logf(l) : -INFINITY;
}

struct AttnPlan {
  int HG, Rp, groups, DC, DVT, n_splits, stages, tmem_cols, v_alias, chunk, kv_chunks;
  int balanced, q_min;      // balanced schedule: n_splits is the largest number of partial results a unit can have
  size_t smem_bytes, ws_bytes, ws_partial_bytes, ws_qimg_bytes, ws_qscale_bytes;
};

static bool plan_attn(int B, int Hq, int Hkv, int D, int Dv, int max_seqlen, bool v_alias, AttnPlan* pl) {
  if (B < 1 || Hq < 1 || Hkv < 1 || Hq % Hkv != 0 || D < 16 || D % 16 != 0 || Dv < 16 || Dv % 16 != 0) return false;
  const int G = Hq / Hkv;
  // up to 8 rows per KV head: the narrow kernel (three CTAs per SM); more: the wide kernel's 32 head slots (a 16-slot
  // narrow kernel needs 166 registers, runs one or two CTAs per SM and measured 5-12 % slower than the wide one half full)
  pl->HG = (G <= 8) ? 8 : 32;
  pl->Rp = 2 * pl->HG;
  pl->groups = (G + pl->HG - 1) / pl->HG;
  pl->DC = (D + kChunk - 1) / kChunk;
  pl->DVT = (Dv + kChunk - 1) / kChunk;
  if (pl->DC > 5 || pl->DVT > 4) return false;
  if (pl->DVT == 3) pl->DVT = 4;
  if (v_alias && Dv > D) return false;
  pl->v_alias = v_alias ? 1 : 0;
  // V aliased to the K rows: PV reads DVT chunks of the stage, which can be one more than the DC chunks the loads fill
  // (Dv of 257..384 bytes is computed as four 128-wide tiles) - the stage is sized for the larger of the two
  pl->kv_chunks = v_alias ? (pl->DC > pl->DVT ? pl->DC : pl->DVT) : pl->DC + pl->DVT;
  const int kv_stage = pl->kv_chunks * kChunkBytes;
  const size_t fixed = static_cast<size_t>(pl->DC) * pl->Rp * kChunk + 2 * pl->Rp * kChunk + 1024;   // Q stack, two P buffers
  pl->stages = (2 * static_cast<size_t>(kv_stage) + fixed <= 227 * 1024 - 2048) ? 2 : 1;
  // Splits of equal size (a fixed number of tiles) keep the CTAs' work uniform whatever the mix of sequence lengths;
  // the size is shrunk until there are enough splits to fill the machine a few times over.
  const int tiles = (max_seqlen + kTok - 1) / kTok;
  const long long units = static_cast<long long>(B) * Hkv * pl->groups;
  int chunk_tiles = option(OPT_ATTN_CHUNK_TILES);       // testing aid
  if (chunk_tiles < 1) chunk_tiles = pl->Rp <= 16 ? 16 : 32;
  while (chunk_tiles > 2 && units * ((tiles + chunk_tiles - 1) / chunk_tiles) < static_cast<long long>(sm_count()) * 4) chunk_tiles >>= 1;
  while ((tiles + chunk_tiles - 1) / chunk_tiles > 65535) chunk_tiles <<= 1;      // splits may run along the grid's y axis
  int ns = (tiles + chunk_tiles - 1) / chunk_tiles;
  if (ns < 1) ns = 1;
  if (const int forced = option(OPT_ATTN_SPLITS); forced >= 1) {      // testing aid: a given number of splits
    ns = forced;
    chunk_tiles = (tiles + ns - 1) / ns;
    if (chunk_tiles < 1) chunk_tiles = 1;
  }
  pl->n_splits = ns;
  pl->chunk = chunk_tiles * kTok;
  // Balanced schedule: every CTA of a grid that just fills the machine gets the same number of tiles, at least q_min
  // (a unit of n tiles then meets at most ceil(n / q_min) + 1 CTAs).  It pays where full-size fixed splits (16 tiles)
  // would leave the resident CTAs between one and three items each to share out - there the SMs that get one more
  // finish a whole split later - and the sequences are long enough (32 tiles) for a run to stay inside one or two of
  // them; elsewhere it costs a few percent (every CTA starts at once and cuts its own run first; every sequence a run
  // enters is a new set-up).  Built for the kernels that keep three CTAs per SM (up to 8 rows per KV head, D and
  // Dv <= 128).
  const bool can_balance = pl->HG == 8 && pl->DC == 1 && pl->DVT == 1 && option(OPT_ATTN_SPLITS) < 1 &&
                           option(OPT_ATTN_CHUNK_TILES) < 1;
  const long long items16 = units * ((tiles + 15) / 16), resident = 3LL * sm_count();
  const int want = option(OPT_ATTN_BALANCED);
  pl->balanced = (can_balance && (want >= 0 ? want > 0 : (tiles >= 32 && items16 >= resident && items16 <= 3 * resident))) ? 1 : 0;
  pl->q_min = chunk_tiles >= 4 ? chunk_tiles / 2 : 2;
  if (pl->balanced) {
    pl->n_splits = (tiles + pl->q_min - 1) / pl->q_min + 1;
    ns = pl->n_splits;
  }
  pl->smem_bytes = static_cast<size_t>(pl->stages) * kv_stage + fixed;
  int cols = 32;
  // wide head groups keep the FP32 running output (4 x 32 columns) behind the two score buffers and the accumulators
  const int cols_needed = pl->HG > 16 ? 2 * pl->Rp + 4 * pl->Rp + 4 * 32 : 2 * pl->Rp + pl->DVT * pl->Rp;
  while (cols < cols_needed) cols <<= 1;
  pl->tmem_cols = cols;
  pl->ws_partial_bytes = round_up(static_cast<size_t>(B) * Hq * ns * (Dv + kPartHdr) * sizeof(float), 1024);
  pl->ws_qimg_bytes = round_up(static_cast<size_t>(units) * pl->DC * pl->Rp * kChunk, 1024);     // stacked Q operands
  pl->ws_qscale_bytes = round_up(static_cast<size_t>(units) * 2 * pl->HG * sizeof(float), 1024);
  pl->ws_bytes = pl->ws_partial_bytes + round_up(static_cast<size_t>(units) * sizeof(unsigned), 1024) + pl->ws_qimg_bytes + pl->ws_qscale_bytes;
  return pl->smem_bytes <= 227 * 1024 - 2048;
}

// The split merge for another attention kernel of this library (rows in output order, every row n_splits partial results).
msd_status_t launch_attn_combine(const float* partial, int n_splits, int Dv, void* out_bf16, float* lse, int rows, cudaStream_t s) {
  if (launch_pdl(attn_combine_kernel, dim3(rows), dim3(128), 0, s, option(OPT_NO_PDL) <= 0, partial, n_splits,
                 static_cast<const int32_t*>(nullptr), 1, 1, 1, Dv, static_cast<__nv_bfloat16*>(out_bf16), lse, 1, 1, 1) != cudaSuccess)
    return MSD_ERR_CUDA;
  return launch_status();
}

using AttnKernel = void (*)(CUtensorMap, CUtensorMap, AttnParams);

// The kernel instantiation for a plan (G: query rows per KV head) and its block size.
static AttnKernel pick_attn_kernel(const AttnPlan& pl, int G, bool paged, int* block_threads) {
  AttnKernel kernel = nullptr;
#define MSD_ATTN_PICK_B(HG_, NH_, P_, B_) \
  kernel = (pl.DVT == 1) ? attn_decode_kernel<HG_, NH_, 1, P_, B_> : (pl.DVT == 2) ? attn_decode_kernel<HG_, NH_, 2, P_, B_> \
                                                                                   : attn_decode_kernel<HG_, NH_, 4, P_, B_>
#define MSD_ATTN_PICK(HG_, NH_) \
  do { if (paged) { MSD_ATTN_PICK_B(HG_, NH_, true, false); } else { MSD_ATTN_PICK_B(HG_, NH_, false, false); } } while (0)
  *block_threads = kAttnThreads;
  if (pl.balanced) {        // (plan_attn: HG == 8, one chunk of D and of Dv)
    if (G <= 4) kernel = paged ? attn_decode_kernel<8, 4, 1, true, true> : attn_decode_kernel<8, 4, 1, false, true>;
    else kernel = paged ? attn_decode_kernel<8, 8, 1, true, true> : attn_decode_kernel<8, 8, 1, false, true>;
  } else if (pl.HG == 8) {
    if (G <= 4) { MSD_ATTN_PICK(8, 4); } else { MSD_ATTN_PICK(8, 8); }
  } else {
    // wide head groups: 32 head slots per CTA, sixteen softmax warps, held references (attn_decode_wide_kernel)
    const bool mla = pl.DC == 5 && pl.DVT == 4 && pl.v_alias && pl.stages == 2;     // a 513..640-byte latent row whose first 512 bytes are V
    if (paged) kernel = mla ? attn_decode_wide_kernel<8, true, 5, 4> : attn_decode_wide_kernel<8, true, 0, 0>;
    else kernel = mla ? attn_decode_wide_kernel<8, false, 5, 4> : attn_decode_wide_kernel<8, false, 0, 0>;
    *block_threads = ((mla && !paged) ? 64 : 96) + 128 * 4;      // producer, QK^T issuer, 16 softmax warps and, except for the chunk-wise kernel, a PV issuer
  }
#undef MSD_ATTN_PICK
#undef MSD_ATTN_PICK_B
  return kernel;
}

// Raises the dynamic shared-memory limit once per kernel instantiation.
static bool prepare_attn_kernel(AttnKernel kernel) {
  static std::mutex mu;
  static void* done[32] = {};
  std::lock_guard<std::mutex> lock(mu);
  int free_slot = -1;
  for (int i = 0; i < 32; ++i) {
    if (done[i] == reinterpret_cast<void*>(kernel)) return true;
    if (!done[i] && free_slot < 0) free_slot = i;
  }
  if (cudaFuncSetAttribute(kernel, cudaFuncAttributeMaxDynamicSharedMemorySize, 227 * 1024 - 2048) != cudaSuccess) return false;
  if (cudaFuncSetAttribute(kernel, cudaFuncAttributePreferredSharedMemoryCarveout, cudaSharedmemCarveoutMaxShared) != cudaSuccess) return false;
  if (free_slot >= 0) done[free_slot] = reinterpret_cast<void*>(kernel);
  return true;
}

// Grid of the balanced schedule: as many CTAs as are resident at once, rounded down to whole sets of U (one CTA per
// unit), at least one set (0: the query failed).
static int attn_balanced_ctas(AttnKernel kernel, int block_threads, size_t smem_bytes, int tmem_cols, int U) {
  struct Entry { void* k; size_t smem; int ctas; };
  static std::mutex mu;
  static Entry cache[32] = {};
  std::lock_guard<std::mutex> lock(mu);
  for (const Entry& e : cache)
    if (e.k == reinterpret_cast<void*>(kernel) && e.smem == smem_bytes) return std::max(e.ctas / U, 1) * U;
  // Resident CTAs per SM from the kernel's own resource use (the runtime's occupancy query assumes the default
  // shared-memory carve-out, not the one a kernel with this much dynamic shared memory gets).
  cudaFuncAttributes fa;
  int dev = 0, smem_sm = 0, smem_resv = 0, regs_sm = 0, threads_sm = 0;
  if (cudaFuncGetAttributes(&fa, kernel) != cudaSuccess || cudaGetDevice(&dev) != cudaSuccess ||
      cudaDeviceGetAttribute(&smem_sm, cudaDevAttrMaxSharedMemoryPerMultiprocessor, dev) != cudaSuccess ||
      cudaDeviceGetAttribute(&smem_resv, cudaDevAttrReservedSharedMemoryPerBlock, dev) != cudaSuccess ||
      cudaDeviceGetAttribute(&regs_sm, cudaDevAttrMaxRegistersPerMultiprocessor, dev) != cudaSuccess ||
      cudaDeviceGetAttribute(&threads_sm, cudaDevAttrMaxThreadsPerMultiProcessor, dev) != cudaSuccess)
    return 0;
  const int warps = (block_threads + 31) / 32;
  const int regs_warp = (fa.numRegs * 32 + 255) / 256 * 256;                 // registers are handed out per warp, 256 at a time
  int per_sm = static_cast<int>(smem_sm / (smem_bytes + fa.sharedSizeBytes + smem_resv));
  // (the register file is four banks, one per scheduler; a CTA's warps are dealt out over them)
  while (per_sm > 1 && (per_sm * warps + 3) / 4 * regs_warp > regs_sm / 4) --per_sm;
  per_sm = std::min(per_sm, threads_sm / block_threads);
  per_sm = std::min(per_sm, 512 / tmem_cols);                                // tensor memory: 512 columns per SM
  if (per_sm < 1) per_sm = 1;
  const int ctas = per_sm * sm_count();
  for (Entry& e : cache)
    if (!e.k) { e.k = reinterpret_cast<void*>(kernel); e.smem = smem_bytes; e.ctas = ctas; break; }
  return std::max(ctas / U, 1) * U;
}

}  // namespace msd

extern "C" {

void msd_debug_set_attn_trace(void* device_buffer) { msd::g_attn_trace = static_cast<long long*>(device_buffer); }

void msd_debug_set_attn_dump(int8_t* q_dbg, float* q_scale_dbg, int32_t* s_dbg) {
  msd::g_attn_q_dbg = q_dbg;
  msd::g_attn_qs_dbg = q_scale_dbg;
  msd::g_attn_s_dbg = s_dbg;
}

msd_status_t msd_attn_decode_softmax_rule(int32_t B, int32_t Hq, int32_t Hkv, int32_t D, int32_t Dv, int32_t max_seqlen,
                                          float* m_margin, float* sv_growth) {
  msd::AttnPlan pl;
  if (!m_margin || !sv_growth) return MSD_ERR_NULL_POINTER;
  if (!msd::plan_attn(B, Hq, Hkv, D, Dv, max_seqlen, false, &pl)) return MSD_ERR_BAD_SHAPE;
  const bool held = pl.HG > 16;
  *m_margin = held ? msd::kHoldMarginLog2 * 0.6931471805599453f : 0.0f;
  *sv_growth = held ? msd::kHoldScaleGrowth : 0.0f;
  return MSD_OK;
}

size_t msd_attn_decode_int8kv_workspace_bytes(int32_t B, int32_t Hq, int32_t Hkv, int32_t D, int32_t Dv, int32_t max_seqlen) {
  msd::AttnPlan pl;
  if (!msd::plan_attn(B, Hq, Hkv, D, Dv, max_seqlen, false, &pl)) return 0;
  return pl.ws_bytes;
}

msd_status_t msd_attn_decode_schedule(int32_t B, int32_t Hq, int32_t Hkv, int32_t D, int32_t Dv, int32_t max_seqlen,
                                      int32_t* tile, int32_t* n_splits, int32_t* split_tokens) {
  msd::AttnPlan pl;
  if (!tile || !n_splits) return MSD_ERR_NULL_POINTER;
  if (!msd::plan_attn(B, Hq, Hkv, D, Dv, max_seqlen, false, &pl)) return MSD_ERR_BAD_SHAPE;
  *tile = msd::kTok;
  *n_splits = pl.n_splits;
  if (split_tokens) *split_tokens = pl.balanced ? 0 : pl.chunk;
  return MSD_OK;
}

// resident_ctas > 0: the number of CTAs the balanced schedule's grid would have is given (host arithmetic only, no
// CUDA call: what the CPU tests use); <= 0: asked of the device as the launch does.
static msd_status_t attn_split_starts(int32_t B, int32_t q_len, int32_t Hq, int32_t Hkv, int32_t D, int32_t Dv, int32_t max_seqlen,
                                      int32_t paged, int32_t v_aliased, int32_t resident_ctas, const int32_t* seqlens, int32_t* starts) {
  using namespace msd;
  if (!seqlens || !starts) return MSD_ERR_NULL_POINTER;
  if (q_len < 1 || Hq < 1 || Hkv < 1 || Hq % Hkv != 0 || B < 1) return MSD_ERR_BAD_SHAPE;
  AttnPlan pl;
  if (!plan_attn(B, Hq * q_len, Hkv, D, Dv, max_seqlen > 0 ? max_seqlen : 1, v_aliased != 0, &pl)) return MSD_ERR_BAD_SHAPE;
  const int G = Hq * q_len / Hkv, U = Hkv * pl.groups, ns = pl.n_splits;
  long long R = 0, W = 0;
  if (pl.balanced) {
    int ctas = resident_ctas > 0 ? std::max(resident_ctas / U, 1) * U : 0;
    if (ctas == 0) {
      int block_threads = 0;
      AttnKernel kernel = pick_attn_kernel(pl, G, paged != 0, &block_threads);
      if (!prepare_attn_kernel(kernel)) return MSD_ERR_CUDA;
      ctas = attn_balanced_ctas(kernel, block_threads, pl.smem_bytes, pl.tmem_cols, U);
    }
    if (ctas < 1) return MSD_ERR_CUDA;
    for (int b = 0; b < B; ++b) W += seqlens[b] > 0 ? (seqlens[b] + kTok - 1) / kTok : 0;
    R = std::min<long long>(W / pl.q_min, ctas / U);
    R = R < 1 ? 1 : R;
  }
  long long P = 0;                                   // tiles of the sequences in front
  for (int b = 0; b < B; ++b) {
    const int L = seqlens[b] > 0 ? seqlens[b] : 0;
    const long long nb = (L + kTok - 1) / kTok;
    int32_t* first_row = starts + static_cast<long long>(b) * Hkv * G * (ns + 1);
    int n = 0;
    first_row[n++] = 0;
    if (pl.balanced) {
      // the runs [i W / R, (i+1) W / R) that begin inside this sequence's tiles [P, P + nb)
      if (nb > 0)
        for (long long i = ((P + 1) * R - 1) / W + 1; i < R && i * W / R < P + nb && n < ns; ++i)
          first_row[n++] = static_cast<int32_t>((i * W / R - P) * kTok);
    } else {
      for (int sidx = 1; sidx < ns; ++sidx) first_row[n++] = static_cast<int32_t>(std::min<long long>(L, static_cast<long long>(sidx) * pl.chunk));
    }
    while (n <= ns) first_row[n++] = L;
    for (int r = 1; r < Hkv * G; ++r) std::copy(first_row, first_row + ns + 1, first_row + static_cast<long long>(r) * (ns + 1));
    P += nb;
  }
  return MSD_OK;
}

msd_status_t msd_attn_decode_split_starts(int32_t B, int32_t q_len, int32_t Hq, int32_t Hkv, int32_t D, int32_t Dv,
                                          int32_t max_seqlen, int32_t paged, int32_t v_aliased, const int32_t* seqlens,
                                          int32_t* starts) {
  return attn_split_starts(B, q_len, Hq, Hkv, D, Dv, max_seqlen, paged, v_aliased, 0, seqlens, starts);
}

msd_status_t msd_debug_attn_split_starts(int32_t B, int32_t q_len, int32_t Hq, int32_t Hkv, int32_t D, int32_t Dv,
                                         int32_t max_seqlen, int32_t v_aliased, int32_t resident_ctas, const int32_t* seqlens,
                                         int32_t* starts) {
  if (resident_ctas < 1) return MSD_ERR_BAD_SHAPE;
  return attn_split_starts(B, q_len, Hq, Hkv, D, Dv, max_seqlen, 0, v_aliased, resident_ctas, seqlens, starts);
}

}  // extern "C"

namespace msd {

// Shared by the contiguous and the paged entry points.  Paged: block_table / seqlens non-null, `page` tokens per block
// (a power of two from 8 to 128, so that pages tile the 128-token MMA tile), total_tokens = num_blocks * page.
static msd_status_t attn_launch(const void* q_bf16, const int8_t* k_cache, const int8_t* v_cache,
                                const float* k_scale, const float* v_scale, const int32_t* cu_seqlens,
                                const int32_t* block_table, const int32_t* seqlens, int32_t page, int32_t max_blocks,
                                int64_t total_tokens, int32_t max_seqlen, int32_t B, int32_t q_len, int32_t Hq_real, int32_t Hkv,
                                int32_t D, int32_t Dv, float softmax_scale, void* out_bf16, float* lse, void* workspace,
                                size_t workspace_bytes, void* stream) {
  if (q_len < 1 || q_len > 64 || Hq_real < 1 || Hkv < 1 || Hq_real % Hkv != 0) return MSD_ERR_BAD_SHAPE;
  const int32_t Hq = Hq_real * q_len;          // (query token, head) rows per sequence
  if (B < 0 || max_seqlen < 0 || total_tokens < 0 || total_tokens > 0x7FFFFFFF) return MSD_ERR_BAD_SHAPE;
  if (B == 0) return MSD_OK;
  AttnPlan pl;
  if (!plan_attn(B, Hq, Hkv, D, Dv, max_seqlen > 0 ? max_seqlen : 1, v_cache == nullptr, &pl)) return MSD_ERR_BAD_SHAPE;
  const bool paged = block_table != nullptr;
  if (!q_bf16 || !k_cache || !k_scale || (!paged && !cu_seqlens) || (paged && !seqlens) || !out_bf16 || !workspace)
    return MSD_ERR_NULL_POINTER;
  if (!aligned(q_bf16, 16) || !aligned(k_cache, 16) || (v_cache && !aligned(v_cache, 16)) || !aligned(out_bf16, 16) ||
      !aligned(workspace, 1024))
    return MSD_ERR_BAD_ALIGNMENT;
  if (workspace_bytes < pl.ws_bytes) return MSD_ERR_WORKSPACE_TOO_SMALL;
  unsigned* status = device_status_ptr();
  if (!status) return MSD_ERR_CUDA;
  cudaStream_t s = static_cast<cudaStream_t>(stream);

  // The tensor maps end at total_tokens: a tile that runs past the cache is zero-filled instead of read.
  const uint64_t T_extent = static_cast<uint64_t>(total_tokens > 0 ? total_tokens : 1);
  const uint32_t box_rows = paged ? static_cast<uint32_t>(page) : static_cast<uint32_t>(kTok);     // one box per page
  CUtensorMap tmap_k, tmap_v;
  if (!encode_tmap_3d(&tmap_k, CU_TENSOR_MAP_DATA_TYPE_UINT8, k_cache, D, Hkv, T_extent, D, static_cast<uint64_t>(Hkv) * D,
                      kChunk, 1, box_rows, CU_TENSOR_MAP_SWIZZLE_128B))
    return MSD_ERR_CUDA;
  const void* vbase = v_cache ? static_cast<const void*>(v_cache) : static_cast<const void*>(k_cache);
  const int vD = v_cache ? Dv : D;
  if (!encode_tmap_3d(&tmap_v, CU_TENSOR_MAP_DATA_TYPE_UINT8, vbase, vD, Hkv, T_extent, vD, static_cast<uint64_t>(Hkv) * vD,
                      kChunk, 1, box_rows, CU_TENSOR_MAP_SWIZZLE_128B))
    return MSD_ERR_CUDA;

  AttnParams p;
  p.q = static_cast<const uint16_t*>(q_bf16);
  p.k_scale = k_scale;
  p.v_scale = v_scale ? v_scale : k_scale;
  p.cu = cu_seqlens;
  p.block_table = block_table;
  p.seqlens = seqlens;
  p.page = paged ? page : kTok;
  p.page_shift = 0;
  while ((1 << p.page_shift) < p.page) ++p.page_shift;
  p.max_blocks = max_blocks;
  p.partial = static_cast<float*>(workspace);
  uint8_t* q_img = static_cast<uint8_t*>(workspace) + (pl.ws_bytes - pl.ws_qimg_bytes - pl.ws_qscale_bytes);
  float* q_scales = reinterpret_cast<float*>(q_img + pl.ws_qimg_bytes);
  p.q_img = q_img; p.q_scales = q_scales;
  p.B = B; p.Hq = Hq; p.Hkv = Hkv; p.D = D; p.Dv = Dv; p.G = Hq / Hkv;
  p.Sq = q_len; p.Gr = Hq_real / Hkv;
  p.HG = pl.HG; p.Rp = pl.Rp; p.groups = pl.groups; p.DC = pl.DC; p.DVT = pl.DVT;
  p.chunk = pl.chunk;
  p.n_splits = pl.n_splits; p.stages = pl.stages; p.v_alias = pl.v_alias; p.kv_chunks = pl.kv_chunks; p.tmem_cols = pl.tmem_cols;
  p.q_dbg = g_attn_q_dbg; p.qs_dbg = g_attn_qs_dbg; p.s_dbg = g_attn_s_dbg; p.dbg_T = total_tokens;
  p.scale = softmax_scale;
  p.status = status;
  p.trace = g_attn_trace;

  int block_threads = kAttnThreads;
  AttnKernel kernel = pick_attn_kernel(pl, Hq / Hkv, paged, &block_threads);
  if (!prepare_attn_kernel(kernel)) return MSD_ERR_CUDA;
  p.balanced = pl.balanced; p.q_min = pl.q_min;
  p.n_slots = reinterpret_cast<int32_t*>(static_cast<uint8_t*>(workspace) + pl.ws_partial_bytes);
  int balanced_ctas = 0;
  if (pl.balanced && (balanced_ctas = attn_balanced_ctas(kernel, block_threads, pl.smem_bytes, pl.tmem_cols, Hkv * pl.groups)) < 1) return MSD_ERR_CUDA;
  // narrow groups: units along x; wide groups: splits along x (see the kernels)
  dim3 grid(B * Hkv * pl.groups, pl.n_splits);
  if (block_threads > kAttnThreads) grid = dim3(pl.n_splits, B * Hkv * pl.groups);
  if (pl.balanced) grid = dim3(balanced_ctas);
  if (block_threads > kAttnThreads) {
    // wide head groups: the stacked Q operands come from a kernel of their own, the attention kernel is its
    // programmatic dependent (its CTAs start their KV loads while it runs)
    attn_qstack_kernel<<<B * Hkv * pl.groups, 32 * pl.HG, 0, s>>>(p, q_img, q_scales);
    if (cudaGetLastError() != cudaSuccess) return MSD_ERR_CUDA;
    if (launch_pdl(kernel, grid, dim3(block_threads), pl.smem_bytes, s, option(OPT_NO_PDL) <= 0, tmap_k, tmap_v, p) != cudaSuccess)
      return MSD_ERR_CUDA;
  } else {
    kernel<<<grid, block_threads, pl.smem_bytes, s>>>(tmap_k, tmap_v, p);
    if (cudaGetLastError() != cudaSuccess) return MSD_ERR_CUDA;
  }
  if (launch_pdl(attn_combine_kernel, dim3(B * Hq), dim3(128), 0, s, option(OPT_NO_PDL) <= 0, static_cast<const float*>(p.partial),
                 pl.n_splits, static_cast<const int32_t*>(pl.balanced ? p.n_slots : nullptr), Hq / Hkv, pl.HG, pl.groups, Dv,
                 static_cast<__nv_bfloat16*>(out_bf16), lse, q_len, Hq / (Hkv * q_len), Hkv) != cudaSuccess)
    return MSD_ERR_CUDA;
  return launch_status();
}

}  // namespace msd

extern "C" {

msd_status_t msd_attn_decode_int8kv(const void* q_bf16, const int8_t* k_cache, const int8_t* v_cache,
                                    const float* k_scale, const float* v_scale, const int32_t* cu_seqlens,
                                    int64_t total_tokens, int32_t max_seqlen, int32_t B, int32_t Hq, int32_t Hkv, int32_t D, int32_t Dv,
                                    float softmax_scale, void* out_bf16, float* lse, void* workspace,
                                    size_t workspace_bytes, void* stream) {
  return msd::attn_launch(q_bf16, k_cache, v_cache, k_scale, v_scale, cu_seqlens, nullptr, nullptr, 0, 0, total_tokens, max_seqlen,
                          B, 1, Hq, Hkv, D, Dv, softmax_scale, out_bf16, lse, workspace, workspace_bytes, stream);
}

msd_status_t msd_attn_decode_int8kv_spec(const void* q_bf16, const int8_t* k_cache, const int8_t* v_cache,
                                         const float* k_scale, const float* v_scale, const int32_t* cu_seqlens,
                                         int64_t total_tokens, int32_t max_seqlen, int32_t B, int32_t q_len, int32_t Hq, int32_t Hkv,
                                         int32_t D, int32_t Dv, float softmax_scale, void* out_bf16, float* lse, void* workspace,
                                         size_t workspace_bytes, void* stream) {
  return msd::attn_launch(q_bf16, k_cache, v_cache, k_scale, v_scale, cu_seqlens, nullptr, nullptr, 0, 0, total_tokens, max_seqlen,
                          B, q_len, Hq, Hkv, D, Dv, softmax_scale, out_bf16, lse, workspace, workspace_bytes, stream);
}

msd_status_t msd_attn_decode_int8kv_paged(const void* q_bf16, const int8_t* k_cache, const int8_t* v_cache,
                                          const float* k_scale, const float* v_scale, const int32_t* block_table,
                                          const int32_t* seqlens, int64_t num_blocks, int32_t page_size,
                                          int32_t max_blocks_per_seq, int32_t max_seqlen, int32_t B, int32_t Hq, int32_t Hkv,
                                          int32_t D, int32_t Dv, float softmax_scale, void* out_bf16, float* lse,
                                          void* workspace, size_t workspace_bytes, void* stream) {
  if (page_size < 8 || page_size > msd::kTok || (page_size & (page_size - 1)) != 0) return MSD_ERR_UNSUPPORTED;
  if (num_blocks < 0 || max_blocks_per_seq < 0 || num_blocks * page_size > 0x7FFFFFFF) return MSD_ERR_BAD_SHAPE;
  if (static_cast<int64_t>(max_blocks_per_seq) * page_size < max_seqlen) return MSD_ERR_BAD_SHAPE;
  if (B > 0 && (!block_table || !seqlens)) return MSD_ERR_NULL_POINTER;
  return msd::attn_launch(q_bf16, k_cache, v_cache, k_scale, v_scale, nullptr, block_table, seqlens, page_size, max_blocks_per_seq,
                          num_blocks * page_size, max_seqlen, B, 1, Hq, Hkv, D, Dv, softmax_scale, out_bf16, lse, workspace,
                          workspace_bytes, stream);
}

}  // extern "C"

// Decode attention over a BF16 KV cache: the arm the INT8-KV MSD kernel is compared with (Sec. 6.4, "Dequant": the
// cache expanded to BF16 by msd_kv_dequant_bf16, attention computed in BF16 with FP32 accumulation).  No MSD in here:
// Q, K, V and the softmax probabilities are BF16 tensor-core operands (tcgen05 kind::f16), everything else FP32.
//
// Same orientation as attn_decode.cu: tokens on the MMA M axis / TMEM lanes,
//   S^T[128 tokens x 16]  = K_tile[128 x D] (K-major, TMA, 128-byte swizzle)  x  Q[16 x D]^T     (16 head slots per KV head)
//   O^T[128 dv x 16]      = V_tile^T[dv x 128 tokens] (the TMA tile read as an MN-major operand)  x  P[16 x 128]^T
// split over the context (flash-decoding) with fixed splits and merged by the same kernel as the INT8 path.
// Warps: 0 = TMA producer, 1 = MMA issuer + TMEM owner, 2..5 = softmax / merge.  Every wait is bounded.
#include <cuda_bf16.h>

#include <cmath>
#include <mutex>

#include "host_common.h"
#include "sm100.cuh"

namespace msd {

namespace {

constexpr int kBTok = 128;               // tokens per tile
constexpr int kBThreads = 192;
constexpr int kBSlots = 16;              // head slots (MMA N): up to 16 query rows per KV head
constexpr int kBRowBytes = 128;          // bytes of a row per TMA box / operand chunk: 64 BF16 values
constexpr int kBChunkBytes = kBTok * kBRowBytes;
constexpr int kBPartHdr = 4;             // as in the INT8 kernel: reference maximum, sum of P, two unused words

struct AttnBf16Params {
  const uint16_t* q;      // [B,Hq,D] BF16
  const int32_t* cu;      // [B+1]
  float* partial;         // [B,Hq,n_splits,4+Dv]
  int B, Hq, Hkv, D, Dv, G;
  int DC, DVC;            // 128-byte chunks of a K row / of a V row
  int n_splits, stages, chunk;
  int tmem_cols;
  float scale;
  unsigned* status;
};

__device__ __forceinline__ float ex2_ftz(float x) {
  float y;
  asm("ex2.approx.ftz.f32 %0, %1;" : "=f"(y) : "f"(x));
  return y;
}

// kNH: heads the softmax code is unrolled for (the group's heads, at most 16)
template <int kNH>
__global__ void __launch_bounds__(kBThreads, 1)
attn_decode_bf16_kernel(const __grid_constant__ CUtensorMap tmap_k, const __grid_constant__ CUtensorMap tmap_v, const AttnBf16Params p) {
  extern __shared__ uint8_t smem_dyn[];
  __shared__ __align__(8) uint64_t k_full[4], k_empty[4], v_full[4], v_empty[4], s_full[2], p_full[2], q_ready, o_full, o_empty;
  __shared__ uint32_t tmem_base_slot;
  __shared__ int abort_flag;
  __shared__ float red[2][4][kNH];
  constexpr int kNSW = 4;

  const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
  const int split = blockIdx.y;
  const int hk = blockIdx.x % p.Hkv, b = blockIdx.x / p.Hkv;
  const int seq0 = p.cu[b];
  const int L = p.cu[b + 1] - seq0;
  const int t_begin = split * p.chunk;
  const int t_end = min(L, t_begin + p.chunk);
  const int h0 = hk * p.G, nh = p.G;
  const int ntiles = (t_end > t_begin) ? (t_end - t_begin + kBTok - 1) / kBTok : 0;
  if (ntiles == 0) {      // nothing in this split: neutral partials, before any barrier or TMEM use
    for (int i = threadIdx.x; i < nh * (p.Dv + kBPartHdr); i += blockDim.x) {
      const int h = i / (p.Dv + kBPartHdr), e = i % (p.Dv + kBPartHdr);
      float* dst = p.partial + ((static_cast<long long>(b) * p.Hq + h0 + h) * p.n_splits + split) * (p.Dv + kBPartHdr);
      dst[e] = (e == 0) ? -INFINITY : 0.0f;
    }
    return;
  }

  uint8_t* smem = reinterpret_cast<uint8_t*>((reinterpret_cast<uintptr_t>(smem_dyn) + 1023) & ~static_cast<uintptr_t>(1023));
  const int stage_bytes = (p.DC + p.DVC) * kBChunkBytes;
  const int q_chunk_bytes = kBSlots * kBRowBytes;          // [16 rows x 128 bytes]
  uint8_t* sm_q = smem + p.stages * stage_bytes;             // DC chunks of the Q operand
  uint8_t* sm_p = sm_q + p.DC * q_chunk_bytes;               // two buffers of two chunks (64 tokens each) of the P operand

  if (threadIdx.x == 0) {
    for (int s = 0; s < p.stages; ++s) {
      mbar_init(&k_full[s], 1); mbar_init(&k_empty[s], 1);
      mbar_init(&v_full[s], 1); mbar_init(&v_empty[s], 1);
    }
    mbar_init(&s_full[0], 1); mbar_init(&s_full[1], 1);
    mbar_init(&p_full[0], kNSW); mbar_init(&p_full[1], kNSW); mbar_init(&q_ready, kNSW);
    mbar_init(&o_full, 1); mbar_init(&o_empty, kNSW);
    abort_flag = 0;
    mbar_init_fence();
    tma_prefetch_desc(&tmap_k);
    tma_prefetch_desc(&tmap_v);
  }
  if (warp == 1) tmem_alloc(&tmem_base_slot, p.tmem_cols);
  // the P buffers start as zeros: the rows of head slots without a head are never written, and what the MMA reads
  // there must at least be finite
  for (int i = threadIdx.x; i < 2 * 2 * q_chunk_bytes / 16; i += blockDim.x) reinterpret_cast<uint4*>(sm_p)[i] = make_uint4(0, 0, 0, 0);
  tc_fence_before();
  __syncthreads();
  tc_fence_after();
  const uint32_t tmem_base = tmem_base_slot;
  const uint32_t tmem_o = tmem_base + 2 * kBSlots;           // O^T tiles after the two S^T buffers
  volatile int* abort = &abort_flag;
  const int n_dvt = p.Dv / 128;                              // 128-wide tiles of Dv (two V chunks each)

  if (warp == 0) {
    // ------------------------------ TMA producer: K and V tiles in rings of their own ------------------------------
    if (lane == 0) {
      int kq = 0, vq = 0;
      long long t_idle = clock64();
      while (kq < ntiles || vq < ntiles) {
        bool progressed = false;
        if (kq < ntiles && mbar_test_wait(&k_empty[kq % p.stages], ((kq / p.stages) & 1) ^ 1)) {
          const int st = kq % p.stages;
          uint8_t* dst = smem + st * stage_bytes;
          mbar_arrive_expect_tx(&k_full[st], p.DC * kBChunkBytes);
          for (int c = 0; c < p.DC; ++c) tma_load_3d(dst + c * kBChunkBytes, &tmap_k, c * 64, hk, seq0 + t_begin + kq * kBTok, &k_full[st]);
          ++kq;
          progressed = true;
        }
        if (vq < ntiles && mbar_test_wait(&v_empty[vq % p.stages], ((vq / p.stages) & 1) ^ 1)) {
          const int st = vq % p.stages;
          uint8_t* dst = smem + st * stage_bytes + p.DC * kBChunkBytes;
          mbar_arrive_expect_tx(&v_full[st], p.DVC * kBChunkBytes);
          for (int c = 0; c < p.DVC; ++c) tma_load_3d(dst + c * kBChunkBytes, &tmap_v, c * 64, hk, seq0 + t_begin + vq * kBTok, &v_full[st]);
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
      const uint32_t idesc_qk = idesc_dense(/*D=F32*/ 1, /*A=BF16*/ 1, /*B=BF16*/ 1, 0, 0, kBTok, kBSlots);     // both K-major
      const uint32_t idesc_pv = idesc_dense(1, 1, 1, /*A (V^T) MN-major*/ 1, 0, kBTok, kBSlots);
      const uint64_t dk = smem_desc(0, 16, 1024, kSwizzle128B);                  // K-major tiles: K, Q, P
      const uint64_t dvt = smem_desc(0, kBChunkBytes, 1024, kSwizzle128B);       // V^T, MN-major: the next 64 dv are one chunk on
      const uint64_t q_enc = dk + (smem_u32(sm_q) >> 4);
      const uint64_t p_enc = dk + (smem_u32(sm_p) >> 4);
      const uint32_t smem_enc = smem_u32(smem) >> 4;
      bool ok = wait_bounded(&q_ready, 0, abort, p.status);
      auto issue_qk = [&](int t) {
        const int st = t % p.stages;
        tc_fence_after();
        uint64_t ka = dk + smem_enc + static_cast<uint32_t>(st * (stage_bytes >> 4));
        uint64_t qa = q_enc;
        const uint32_t d = tmem_base + (t & 1) * kBSlots;
        for (int c = 0; c < p.DC; ++c) {
#pragma unroll
          for (int k = 0; k < 4; ++k) mma_f16(d, ka + 2 * k, qa + 2 * k, idesc_qk, (c > 0 || k > 0) ? 1u : 0u);      // 16 values of d per MMA
          ka += kBChunkBytes >> 4;
          qa += q_chunk_bytes >> 4;
        }
        tc_commit(&s_full[t & 1]);
        tc_commit(&k_empty[st]);
      };
      auto issue_pv = [&](int t) {
        tc_fence_after();
        const int st = t % p.stages;
        uint64_t va = dvt + smem_enc + static_cast<uint32_t>(st * (stage_bytes >> 4)) + static_cast<uint32_t>(p.DC * (kBChunkBytes >> 4));
        const uint64_t pa = p_enc + static_cast<uint32_t>((t & 1) * (2 * q_chunk_bytes >> 4));
        uint32_t d = tmem_o;
        for (int j = 0; j < n_dvt; ++j) {
#pragma unroll
          for (int k = 0; k < 8; ++k)        // 16 tokens per MMA: two 8-token groups of 1024 bytes; P: 32 bytes on, the second chunk after four
            mma_f16(d, va + k * (2048 >> 4), pa + (k >> 2) * (q_chunk_bytes >> 4) + 2 * (k & 3), idesc_pv, k > 0 ? 1u : 0u);
          va += 2 * (kBChunkBytes >> 4);
          d += kBSlots;
        }
        tc_commit(&o_full);
        tc_commit(&v_empty[st]);
      };
      int q = 0, v = 0;
      long long t_idle = clock64();
      while (ok && v < ntiles) {
        bool progressed = false;
        if (q < ntiles && q < v + 2 && mbar_test_wait(&k_full[q % p.stages], (q / p.stages) & 1)) {    // (q < v + 2: P of tile q-2 is written)
          issue_qk(q);
          ++q;
          progressed = true;
        }
        if (v < q && mbar_test_wait(&p_full[v & 1], (v >> 1) & 1) && (v == 0 || mbar_test_wait(&o_empty, (v - 1) & 1)) &&
            mbar_test_wait(&v_full[v % p.stages], (v / p.stages) & 1)) {
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
    const int wq = warp - 2;
    // the Q operand: rows of 64 BF16 values per chunk, 128-byte swizzle, head slots without a head zero
    {
      const int per_row = p.D >> 3;                 // 16-byte pieces per row
      for (int i = threadIdx.x - 64; i < kBSlots * per_row; i += 128) {
        const int h = i / per_row, j = i - h * per_row;
        uint4 v = make_uint4(0, 0, 0, 0);
        if (h < nh) v = __ldg(reinterpret_cast<const uint4*>(p.q + (static_cast<long long>(b) * p.Hq + h0 + h) * p.D) + j);
        const int d0 = j << 3;
        *reinterpret_cast<uint4*>(sm_q + (d0 >> 6) * q_chunk_bytes + swz_off(h, (d0 & 63) * 2)) = v;
      }
    }
    fence_proxy_async_smem();
    __syncwarp();
    if (lane == 0) mbar_arrive(&q_ready);

    float l_part[kNH], m_run[kNH], o_run[kNH], resc_keep[kNH], resc_next[kNH];
#pragma unroll
    for (int h = 0; h < kNH; ++h) { l_part[h] = 0.0f; m_run[h] = -INFINITY; o_run[h] = 0.0f; }
    const float scale2 = p.scale * 1.4426950408889634f;      // scores in the log2 domain
    bool ok = true;

    auto softmax_tile = [&](int t, float (&resc_out)[kNH]) -> bool {
      const int tok_rel = t_begin + t * kBTok + tl;
      const bool valid = tok_rel < t_end;
      if (!wait_bounded(&s_full[t & 1], (t >> 1) & 1, abort, p.status)) return false;
      tc_fence_after();
      float s[kNH];
      {
        uint32_t v[kBSlots];
        tmem_ld16(tmem_base + (static_cast<uint32_t>(quad * 32) << 16) + (t & 1) * kBSlots, v);
        tmem_ld_wait();
#pragma unroll
        for (int h = 0; h < kNH; ++h) s[h] = valid ? __uint_as_float(v[h]) * scale2 : -INFINITY;
      }
      float (*rb)[kNH] = red[t & 1];
#pragma unroll
      for (int h = 0; h < kNH; ++h) {
        const float wm = warp_max(s[h]);
        if (lane == 0) rb[wq][h] = wm;
      }
      named_bar_sync(1, 128);
      uint8_t* pbuf = sm_p + (t & 1) * (2 * q_chunk_bytes) + (tl >> 6) * q_chunk_bytes;
#pragma unroll
      for (int h = 0; h < kNH; ++h) {
        const float mt = fmaxf(fmaxf(rb[0][h], rb[1][h]), fmaxf(rb[2][h], rb[3][h]));
        const float mn = fmaxf(m_run[h], mt);
        const float resc = (m_run[h] == -INFINITY) ? 0.0f : ex2_ftz(m_run[h] - mn);
        m_run[h] = mn;
        resc_out[h] = resc;
        const float pr = (h < nh) ? ex2_ftz(s[h] - fmaxf(mn, -1e30f)) : 0.0f;
        l_part[h] = __fmaf_rn(l_part[h], resc, pr);
        const __nv_bfloat16 pb = __float2bfloat16_rn(pr);              // P goes into the product as BF16
        *reinterpret_cast<__nv_bfloat16*>(pbuf + swz_off(h, (tl & 63) * 2)) = pb;
      }
      fence_proxy_async_smem();
      tc_fence_before();
      __syncwarp();
      if (lane == 0) mbar_arrive(&p_full[t & 1]);
      return true;
    };

    ok = softmax_tile(0, resc_keep);
    for (int t = 0; t < ntiles && ok; ++t) {
      if (t + 1 < ntiles) {
        ok = softmax_tile(t + 1, resc_next);     // overlaps the PV product of tile t
        if (!ok) break;
      }
      ok = wait_bounded(&o_full, t & 1, abort, p.status);
      if (!ok) break;
      tc_fence_after();
      {
        uint32_t v[kBSlots];
        tmem_ld16(tmem_o + (static_cast<uint32_t>(quad * 32) << 16), v);
        tmem_ld_wait();
#pragma unroll
        for (int h = 0; h < kNH; ++h) o_run[h] = __fmaf_rn(o_run[h], resc_keep[h], __uint_as_float(v[h]));
      }
      tc_fence_before();
      __syncwarp();
      if (lane == 0) mbar_arrive(&o_empty);
#pragma unroll
      for (int h = 0; h < kNH; ++h) resc_keep[h] = resc_next[h];
    }
    if (ok) {
      float (*rb)[kNH] = red[ntiles & 1];
      named_bar_sync(1, 128);
#pragma unroll
      for (int h = 0; h < kNH; ++h) {
        float l = l_part[h];
#pragma unroll
        for (int o = 16; o > 0; o >>= 1) l += __shfl_xor_sync(0xffffffffu, l, o);
        if (lane == 0) rb[wq][h] = l;
      }
      named_bar_sync(1, 128);
#pragma unroll
      for (int h = 0; h < kNH; ++h) {
        if (h < nh) {
          float* dst = p.partial + ((static_cast<long long>(b) * p.Hq + h0 + h) * p.n_splits + split) * (p.Dv + kBPartHdr);
          if (tl == 0) { dst[0] = m_run[h] * 0.6931471805599453f; dst[1] = rb[0][h] + rb[1][h] + rb[2][h] + rb[3][h]; }
          dst[kBPartHdr + tl] = o_run[h];
        }
      }
    }
  }

  tc_fence_before();
  __syncthreads();
  if (warp == 1) {
    tc_fence_after();
    tmem_dealloc(tmem_base, p.tmem_cols);
  }
}

struct Bf16Plan {
  int DC, DVC, n_splits, stages, chunk, tmem_cols;
  size_t smem_bytes, ws_bytes;
};

// D in {64, 128}, Dv = 128, up to 16 query rows per KV head (one CTA computes all of them)
bool plan_bf16(int B, int Hq, int Hkv, int D, int Dv, int max_seqlen, Bf16Plan* pl) {
  if (B < 1 || Hq < 1 || Hkv < 1 || Hq % Hkv != 0 || Hq / Hkv > kBSlots) return false;
  if ((D != 64 && D != 128) || Dv != 128) return false;
  pl->DC = D * 2 / kBRowBytes;
  pl->DVC = Dv * 2 / kBRowBytes;
  const size_t stage = static_cast<size_t>(pl->DC + pl->DVC) * kBChunkBytes;
  const size_t fixed = static_cast<size_t>(pl->DC) * kBSlots * kBRowBytes + 2 * 2 * kBSlots * kBRowBytes + 1024;
  pl->stages = 2;
  while (pl->stages < 4 && (pl->stages + 1) * stage + fixed <= 227 * 1024 - 2048) ++pl->stages;
  pl->smem_bytes = pl->stages * stage + fixed;
  const int tiles = (max_seqlen + kBTok - 1) / kBTok;
  const long long units = static_cast<long long>(B) * Hkv;
  int chunk_tiles = 16;
  while (chunk_tiles > 2 && units * ((tiles + chunk_tiles - 1) / chunk_tiles) < static_cast<long long>(sm_count()) * 2) chunk_tiles >>= 1;
  while ((tiles + chunk_tiles - 1) / chunk_tiles > 65535) chunk_tiles <<= 1;
  pl->n_splits = (tiles + chunk_tiles - 1) / chunk_tiles;
  if (pl->n_splits < 1) pl->n_splits = 1;
  pl->chunk = chunk_tiles * kBTok;
  pl->tmem_cols = 64;                                        // 2 x 16 score columns + 16 output columns
  pl->ws_bytes = round_up(static_cast<size_t>(B) * Hq * pl->n_splits * (Dv + kBPartHdr) * sizeof(float), 1024);
  return true;
}

}  // namespace

}  // namespace msd

extern "C" {

size_t msd_attn_decode_bf16kv_workspace_bytes(int32_t B, int32_t Hq, int32_t Hkv, int32_t D, int32_t Dv, int32_t max_seqlen) {
  msd::Bf16Plan pl;
  if (!msd::plan_bf16(B, Hq, Hkv, D, Dv, max_seqlen > 0 ? max_seqlen : 1, &pl)) return 0;
  return pl.ws_bytes;
}

msd_status_t msd_attn_decode_bf16kv(const void* q_bf16, const void* k_bf16, const void* v_bf16, const int32_t* cu_seqlens,
                                    int64_t total_tokens, int32_t max_seqlen, int32_t B, int32_t Hq, int32_t Hkv, int32_t D,
                                    int32_t Dv, float softmax_scale, void* out_bf16, float* lse, void* workspace,
                                    size_t workspace_bytes, void* stream) {
  using namespace msd;
  if (B < 0 || max_seqlen < 0 || total_tokens < 0 || total_tokens > 0x7FFFFFFF) return MSD_ERR_BAD_SHAPE;
  if (B == 0) return MSD_OK;
  Bf16Plan pl;
  if (Hq < 1 || Hkv < 1 || Hq % Hkv != 0) return MSD_ERR_BAD_SHAPE;
  if (!plan_bf16(B, Hq, Hkv, D, Dv, max_seqlen > 0 ? max_seqlen : 1, &pl)) return MSD_ERR_UNSUPPORTED;
  if (!q_bf16 || !k_bf16 || !v_bf16 || !cu_seqlens || !out_bf16 || !workspace) return MSD_ERR_NULL_POINTER;
  if (!aligned(q_bf16, 16) || !aligned(k_bf16, 16) || !aligned(v_bf16, 16) || !aligned(out_bf16, 16) || !aligned(workspace, 1024))
    return MSD_ERR_BAD_ALIGNMENT;
  if (workspace_bytes < pl.ws_bytes) return MSD_ERR_WORKSPACE_TOO_SMALL;
  unsigned* status = device_status_ptr();
  if (!status) return MSD_ERR_CUDA;
  cudaStream_t s = static_cast<cudaStream_t>(stream);

  // The tensor maps end at total_tokens: a tile that runs past the cache is zero-filled instead of read.
  const uint64_t T_extent = static_cast<uint64_t>(total_tokens > 0 ? total_tokens : 1);
  CUtensorMap tmap_k, tmap_v;
  if (!encode_tmap_3d(&tmap_k, CU_TENSOR_MAP_DATA_TYPE_BFLOAT16, k_bf16, D, Hkv, T_extent, static_cast<uint64_t>(D) * 2,
                      static_cast<uint64_t>(Hkv) * D * 2, 64, 1, kBTok, CU_TENSOR_MAP_SWIZZLE_128B))
    return MSD_ERR_CUDA;
  if (!encode_tmap_3d(&tmap_v, CU_TENSOR_MAP_DATA_TYPE_BFLOAT16, v_bf16, Dv, Hkv, T_extent, static_cast<uint64_t>(Dv) * 2,
                      static_cast<uint64_t>(Hkv) * Dv * 2, 64, 1, kBTok, CU_TENSOR_MAP_SWIZZLE_128B))
    return MSD_ERR_CUDA;

  AttnBf16Params p;
  p.q = static_cast<const uint16_t*>(q_bf16);
  p.cu = cu_seqlens;
  p.partial = static_cast<float*>(workspace);
  p.B = B; p.Hq = Hq; p.Hkv = Hkv; p.D = D; p.Dv = Dv; p.G = Hq / Hkv;
  p.DC = pl.DC; p.DVC = pl.DVC;
  p.n_splits = pl.n_splits; p.stages = pl.stages; p.chunk = pl.chunk; p.tmem_cols = pl.tmem_cols;
  p.scale = softmax_scale;
  p.status = status;

  void (*kernel)(CUtensorMap, CUtensorMap, AttnBf16Params) =
      p.G <= 4 ? attn_decode_bf16_kernel<4> : (p.G <= 8 ? attn_decode_bf16_kernel<8> : attn_decode_bf16_kernel<16>);
  {
    static std::mutex mu;
    static void* prepared[4] = {};
    std::lock_guard<std::mutex> lock(mu);
    bool seen = false;
    for (void* k : prepared) seen = seen || k == reinterpret_cast<void*>(kernel);
    if (!seen) {
      if (cudaFuncSetAttribute(kernel, cudaFuncAttributeMaxDynamicSharedMemorySize, 227 * 1024 - 2048) != cudaSuccess) return MSD_ERR_CUDA;
      for (void*& k : prepared)
        if (!k) { k = reinterpret_cast<void*>(kernel); break; }
    }
  }
  kernel<<<dim3(B * Hkv, pl.n_splits), kBThreads, pl.smem_bytes, s>>>(tmap_k, tmap_v, p);
  if (cudaGetLastError() != cudaSuccess) return MSD_ERR_CUDA;
  return launch_attn_combine(p.partial, pl.n_splits, Dv, out_bf16, lse, B * Hq, s);
}

}  // extern "C"

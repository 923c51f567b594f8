// Stage 2 on tensor cores: the key-side feature map and the two key-side contractions
// (arxiv 2306.15799, Eq. (2): phi(K')^T V' and, for the normaliser of Appendix D, phi(K')^T 1),
// kept per feature in the log domain:
//
//   PERFORMER   L_ij = w_i . k'_j - |k'_j|^2 / 2          (rows i = features, columns j = projected keys)
//               b_i  = log sum_j exp(L_ij),  a_i = sum_j softmax_j(L_i.) v'_j
//   RNN         f_ij = elu(k'_ji) + 1,  z_i = sum_j f_ij,  a_i = sum_j f_ij v'_j / z_i
//
// One CTA owns 128 features of one head and walks the keys in chunks of 128.  K' and V' arrive as
// fp32 (stage 1's workspace): a bulk copy brings the rows of a chunk, which are contiguous, into a
// staging buffer while the previous chunk's MMAs run, and short rolled loops (each part of this
// kernel runs only a few times per CTA, so its time is largely instruction fetch and compact code
// matters) split them into bf16 / fp16 terms so that the tensor-core
// products are fp32-accurate: K' = hi + mid + lo (three bf16 terms, exact to 24 bits) against the
// exact bf16 W, and -|k'|^2/2 as three bf16 terms in one extra 16-wide contraction step; V' = hi + lo
// in fp16.  L for all k keys sits in TMEM (k <= 512 columns); the thread that owns a row takes its
// maximum, writes exp(L - max) back as fp16 pairs and keeps the sum of the rounded values, so the
// dominant term cancels exactly in a_i.  The second product reads those weights straight from TMEM.
//
// With few heads the keys are split over `nsplit` CTAs per (head, feature tile): each keeps its own
// maximum, sum and unnormalised accumulator, writes them to a scratch area, and the CTA that arrives
// last at the tile's counter merges them (log-sum-exp over the partial maxima) and writes a_i, b_i.
// Nobody waits for anybody: the last arrival finds every partial result already in memory.
#pragma once

#include <cuda_bf16.h>
#include <cuda_fp16.h>

#include "tc_common.cuh"

namespace flurka {

struct K2Params {
  int d, k, p, BH;          // p = feature dimension (m, or d for RNN)
  int ftiles;               // ceil(p / 128)
  const float* kpvp;        // [2][BH][k][d] fp32
  float* weight;            // [BH][p]      b_i (PERFORMER) or z_i (RNN)
  __half* aT16;             // [BH][d][p]   a^T
  float* a32;               // [BH][p][d]   a in fp32 as well (the backward pass wants it), or NULL
  int* status;
  int nsplit;               // CTAs per (head, feature tile) along the keys (1..4; PERFORMER only)
  float* part;              // nsplit > 1: [BH * ftiles][nsplit][d + 2][128]  max, sum, accumulator columns
  int* counters;            // nsplit > 1: [BH * ftiles], zero on entry, zero again on exit
};

constexpr int kK2Threads = 256;
constexpr int kK2Chunk = 128;  // keys per chunk (the last chunk may hold 64)
// shared memory: W tile (<= 32 KB) | ones 4 KB | -|k'|^2/2 tile 4 KB | three 32 KB operand tiles |
// 64 KB fp32 staging (128 rows x d <= 128) | barriers
constexpr int kK2SmemBytes = 32768 + 4096 + 4096 + 3 * 32768 + 65536 + 256 + 1024;
constexpr int kK2OCol = 256;   // TMEM column of the a accumulator

// two floats -> {lo: bf16(a), hi: bf16(b)} with one rounding instruction
__device__ __forceinline__ uint32_t pack_bf16x2(float a, float b) {
  uint32_t r;
  asm("cvt.rn.bf16x2.f32 %0, %2, %1;" : "=r"(r) : "f"(a), "f"(b));
  return r;
}

__device__ __forceinline__ float k2_ex2(float x) {
  float y;
  asm("ex2.approx.ftz.f32 %0, %1;" : "=f"(y) : "f"(x));
  return y;
}

template <bool kPerformer>
__global__ void __launch_bounds__(kK2Threads, 1)
k2_key_side(const __grid_constant__ CUtensorMap tmW, const K2Params prm) {
  using namespace tc;
  extern __shared__ uint8_t smem_raw[];
  const uint32_t base = (smem_u32(smem_raw) + 1023u) & ~1023u;
  uint8_t* base_ptr = smem_raw + (base - smem_u32(smem_raw));
  const uint32_t sm_w = base;
  const uint32_t sm_ones = base + 32768;
  const uint32_t sm_nrm = sm_ones + 4096;
  const uint32_t sm_op = sm_nrm + 4096;          // 3 x 32 KB, 1024-aligned
  const uint32_t sm_stage = sm_op + 3 * 32768;   // fp32 rows of the current chunk
  const uint32_t bar_w = sm_stage + 65536;
  const uint32_t bar_mma = bar_w + 8;
  const uint32_t bar_stage = bar_w + 16;
  const uint32_t bar_kp = bar_w + 24;             // RNN: a piece of K' has arrived
  const uint32_t tmem_slot = bar_w + 32;
  __shared__ int abort_flag;
  __shared__ uint32_t tmem_base_shared;

  const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31, tid = threadIdx.x;
  const int d = prm.d, k = prm.k, p = prm.p;
  const int nsplit = prm.nsplit;
  const int sp = blockIdx.x % nsplit;                         // which part of the keys
  const int unit = blockIdx.x / nsplit;                       // (head, feature tile)
  const int head = unit / prm.ftiles;
  const int i0 = (unit % prm.ftiles) * 128;                   // first feature of this CTA
  const float* __restrict__ Kp = prm.kpvp + (size_t)head * k * d;
  const float* __restrict__ Vp = prm.kpvp + ((size_t)prm.BH + head) * (size_t)k * d;
  const int kq = d >> 6;                                      // 64-wide blocks of the head dimension
  const int nchunks_all = (k + kK2Chunk - 1) / kK2Chunk;
  const int jc_begin = (sp * nchunks_all) / nsplit;           // this CTA's chunks [jc_begin, jc_begin + nchunks)
  const int nchunks = ((sp + 1) * nchunks_all) / nsplit - jc_begin;
  const int klocal = min(k, (jc_begin + nchunks) * kK2Chunk) - jc_begin * kK2Chunk;   // keys of this CTA

  if (tid == 0) {
    abort_flag = 0;
    mbar_init(bar_w, 1);
    mbar_init(bar_mma, 1);
    mbar_init(bar_stage, 1);
    mbar_init(bar_kp, 1);
    fence_mbar_init();
  }
  if (warp == 4) {
    tmem_alloc(tmem_slot, 512);
    tmem_relinquish();
  }
  if (kPerformer && warp == 5) {
    // A operand of the bias step: [128 x 16] bf16, columns 0..2 = 1, no swizzle
    // (element (r, c) at (r/8)*256 + (c/8)*128 + (r%8)*16 + (c%8)*2 bytes)
    __nv_bfloat16* ones = reinterpret_cast<__nv_bfloat16*>(base_ptr + (sm_ones - base));
    for (int e = lane; e < 128 * 16; e += 32) {
      const int r = e >> 4, c = e & 15;
      ones[(r >> 3) * 128 + (c >> 3) * 64 + (r & 7) * 8 + (c & 7)] = __float2bfloat16_rn(c < 3 ? 1.f : 0.f);
    }
    fence_proxy_async_smem();
  }
  tcgen05_fence_before();
  __syncthreads();
  tcgen05_fence_after();
  if (tid == 0) {
    uint32_t v;
    asm volatile("ld.shared.u32 %0, [%1];" : "=r"(v) : "r"(tmem_slot));
    tmem_base_shared = v;
    if (kPerformer) {
      prefetch_tmap(&tmW);
      mbar_arrive_expect_tx(bar_w, (uint32_t)(128 * d * 2));
      for (int kb = 0; kb < kq; ++kb) tma_load_2d(sm_w + kb * 16384, &tmW, bar_w, kb * 64, i0);
    }
  }
  __syncthreads();
  const uint32_t tmem = tmem_base_shared;
  bool ok = true;
  uint32_t mma_phase = 0;
  // everything above (and the W tile on its way) is independent of stage 1
  grid_dependency_wait();

  // conversion geometry: a warp instruction reads whole rows (d/4 lanes x float4 per row), so the fp32
  // rows arrive in full 128-byte lines; each lane converts four consecutive columns of its rows
  const int lpr = d >> 2;                        // lanes per row: 16 or 32
  const int rpi = 32 / lpr;                      // rows per warp instruction: 2 or 1
  const int ccol = (lane % lpr) * 4;             // this lane's first column
  const int crow0 = warp * rpi + lane / lpr;     // this lane's row in iteration 0; iteration t adds 8*rpi
  const int citers = kK2Chunk / (8 * rpi);       // 8 or 16 iterations cover the 128 rows of a chunk
  const uint32_t coff = (uint32_t)(ccol >> 6) * 16384 + (uint32_t)((ccol & 7) >> 2) * 8;
  const int cchunk = (ccol & 63) >> 3;           // 16-byte chunk of the 128-byte row before the swizzle
  // thread 0 starts the copy of a chunk's fp32 rows (contiguous in the workspace) into the staging buffer
  uint32_t stage_phase = 0;
  auto stage_chunk = [&](const float* mat, int jg) {
    const int rows = min(kK2Chunk, k - jg * kK2Chunk);
    const uint32_t bytes = (uint32_t)rows * d * 4;
    mbar_arrive_expect_tx(bar_stage, bytes);
    bulk_load(sm_stage, mat + (size_t)jg * kK2Chunk * d, bytes, bar_stage);
  };
  auto wait_stage = [&]() {
    bool mine = true;
    if (warp == 4) mine = mbar_wait(bar_stage, stage_phase, prm.status, &abort_flag);
    ok = __syncthreads_and(mine) != 0;
    stage_phase ^= 1;
  };
  auto stage_ld = [&](int r) {
    float4 v;
    asm volatile("ld.shared.v4.f32 {%0, %1, %2, %3}, [%4];"
                 : "=f"(v.x), "=f"(v.y), "=f"(v.z), "=f"(v.w) : "r"(sm_stage + (uint32_t)(r * d + ccol) * 4u));
    return v;
  };
  // only the issuing warp polls the MMA barrier; everybody else sleeps in the block barrier
  auto wait_mma = [&]() {
    bool mine = true;
    if (warp == 4) mine = mbar_wait(bar_mma, mma_phase, prm.status, &abort_flag);
    ok = __syncthreads_and(mine) != 0;
    mma_phase ^= 1;
    tcgen05_fence_after();
  };

  if (kPerformer) {
    {
      bool mine = true;
      if (warp == 4) mine = mbar_wait(bar_w, 0, prm.status, &abort_flag);
      ok = __syncthreads_and(mine) != 0;
    }
    if (tid == 0) stage_chunk(Kp, jc_begin);
    for (int jc = 0; jc < nchunks && ok; ++jc) {
      const int rows = min(kK2Chunk, k - (jc_begin + jc) * kK2Chunk);   // 64 or 128 keys in this chunk
      wait_stage();
      if (!ok) break;
      // ---- K' rows of the chunk: fp32 -> three bf16 tiles (K-major, 128-byte swizzle) and -|k'|^2/2
#pragma unroll 2
      for (int t = 0; t < citers; ++t) {
        const int r = crow0 + t * 8 * rpi;
        if (r < rows) {                                        // uniform over the warp (rows is even)
          const float4 x = stage_ld(r);
          // packed conversions: one instruction rounds two values; a bf16 is the top half of an fp32
          float a = x.x, b = x.y, c = x.z, e = x.w;
          float sq = fmaf(a, a, fmaf(b, b, fmaf(c, c, e * e)));
          const uint32_t h0 = pack_bf16x2(a, b), h1 = pack_bf16x2(c, e);
          a -= __uint_as_float(h0 << 16); b -= __uint_as_float(h0 & 0xffff0000u);
          c -= __uint_as_float(h1 << 16); e -= __uint_as_float(h1 & 0xffff0000u);
          const uint32_t m0 = pack_bf16x2(a, b), m1 = pack_bf16x2(c, e);
          a -= __uint_as_float(m0 << 16); b -= __uint_as_float(m0 & 0xffff0000u);
          c -= __uint_as_float(m1 << 16); e -= __uint_as_float(m1 & 0xffff0000u);
          const uint32_t l0 = pack_bf16x2(a, b), l1 = pack_bf16x2(c, e);
          const uint32_t off = sm_op + coff + r * 128 + ((cchunk ^ (r & 7)) << 4);
          asm volatile("st.shared.v2.b32 [%0], {%1, %2};" ::"r"(off), "r"(h0), "r"(h1) : "memory");
          asm volatile("st.shared.v2.b32 [%0], {%1, %2};" ::"r"(off + 32768), "r"(m0), "r"(m1) : "memory");
          asm volatile("st.shared.v2.b32 [%0], {%1, %2};" ::"r"(off + 65536), "r"(l0), "r"(l1) : "memory");
          // |k'_r|^2 over the lanes that share the row
          if (lpr == 32) sq += __shfl_xor_sync(0xffffffffu, sq, 16);
#pragma unroll
          for (int o = 8; o > 0; o >>= 1) sq += __shfl_xor_sync(0xffffffffu, sq, o);
          if ((lane % lpr) == 0) {
            // B operand of the bias step: row r, columns 0..2 = three bf16 terms of -|k'_r|^2/2
            float bb = -0.5f * sq;
            const __nv_bfloat16 g0 = __float2bfloat16_rn(bb);  bb -= __bfloat162float(g0);
            const __nv_bfloat16 g1 = __float2bfloat16_rn(bb);  bb -= __bfloat162float(g1);
            const __nv_bfloat16 g2 = __float2bfloat16_rn(bb);
            const uint32_t na = sm_nrm + (r >> 3) * 256 + (r & 7) * 16;
            const uint32_t z = 0;
            asm volatile("st.shared.v4.b32 [%0], {%1, %2, %3, %4};" ::"r"(na),
                         "r"((uint32_t)__bfloat16_as_ushort(g0) | ((uint32_t)__bfloat16_as_ushort(g1) << 16)),
                         "r"((uint32_t)__bfloat16_as_ushort(g2)), "r"(z), "r"(z) : "memory");
            asm volatile("st.shared.v4.b32 [%0], {%1, %2, %3, %4};" ::"r"(na + 128), "r"(z), "r"(z), "r"(z), "r"(z) : "memory");
          }
        }
      }
      fence_proxy_async_smem();
      __syncthreads();
      // the staging buffer has been read out: start the next copy (the next K' chunk, or the first
      // V' chunk of the second product) under this chunk's MMAs
      if (tid == 0) stage_chunk(jc + 1 < nchunks ? Kp : Vp, jc + 1 < nchunks ? jc_begin + jc + 1 : jc_begin);
      if (tid == 128) {
        tcgen05_fence_after();
        const uint32_t idesc1 = make_idesc(kFmtBF16, 0, 0, 128, (uint32_t)rows);
        const uint32_t dcol = tmem + jc * kK2Chunk;
        for (int s3 = 0; s3 < 3; ++s3) {
          for (int kb = 0; kb < kq; ++kb) {
            const uint64_t ad = make_sdesc(sm_w + kb * 16384, 16, 1024, kSwizzle128);
            const uint64_t bd = make_sdesc(sm_op + s3 * 32768 + kb * 16384, 16, 1024, kSwizzle128);
            mma_ss_x4(dcol, ad, bd, 2, 2, idesc1, (s3 > 0 || kb > 0) ? 1u : 0u);
          }
        }
        const uint64_t ad = make_sdesc(sm_ones, 128, 256, kSwizzleNone);
        const uint64_t bd = make_sdesc(sm_nrm, 128, 256, kSwizzleNone);
        mma_ss(dcol, ad, bd, idesc1, 1u);
        mma_commit(bar_mma);
      }
      // the operand tiles are rewritten for the next chunk: wait until the MMAs have read them
      wait_mma();
    }
  }

  // ---- feature weights: one thread per feature row (warps 0..3)
  float zsum = 0.f, row_max = 0.f;
  const int feat = i0 + (warp & 3) * 32 + lane;             // valid for warps 0..3
  if (kPerformer) {
    if (warp < 4 && ok) {
      const uint32_t tb = tmem + ((uint32_t)(warp * 32) << 16);
      const float kLog2e = 1.4426950408889634f;
      float mx = -INFINITY;
      for (int c = 0; c < klocal; c += 32) {
        uint32_t r[32];
        tmem_ld32(tb + c, r);
        tmem_wait_ld(r);
#pragma unroll
        for (int e = 0; e < 32; e += 2) mx = fmax3(mx, __uint_as_float(r[e]), __uint_as_float(r[e + 1]));
      }
      row_max = mx;
      const float shift = mx * kLog2e;
      for (int c = 0; c < klocal; c += 32) {
        uint32_t r[32], h[16];
        tmem_ld32(tb + c, r);
        tmem_wait_ld(r);
#pragma unroll
        for (int e = 0; e < 16; ++e) {
          const float e0 = k2_ex2(fmaf(__uint_as_float(r[2 * e]), kLog2e, -shift));
          const float e1 = k2_ex2(fmaf(__uint_as_float(r[2 * e + 1]), kLog2e, -shift));
          const __half2 hh = __floats2half2_rn(e0, e1);
          const float2 back = __half22float2(hh);
          zsum += back.x + back.y;
          h[e] = *reinterpret_cast<const uint32_t*>(&hh);
        }
        tmem_st16(tb + (c >> 1), h);
      }
      if (nsplit == 1 && feat < p) prm.weight[(size_t)head * p + feat] = mx + __logf(zsum);
      tmem_wait_st();
      tcgen05_fence_before();
    }
  } else {
    if (tid == 0) stage_chunk(Vp, jc_begin);
    // RNN: f_ij = elu(k'_ji) + 1.  K' arrives by bulk copy, in pieces of up to 96 KB, in the operand
    // area (unused until the conversion of V'); the thread that owns feature i walks down column i
    // (consecutive lanes read consecutive words).  Two threads share a feature: warps w and w + 4 see
    // the same TMEM lanes and take alternate groups of 32 keys.
    const float* stage = reinterpret_cast<const float*>(base_ptr + (sm_op - base));
    const uint32_t tb = tmem + ((uint32_t)((warp & 3) * 32) << 16);
    const int piece_rows = ((3 * 32768) / (d * 4)) & ~63;       // 384 rows at d = 64, 192 at d = 128
    const int col = feat < p ? feat : 0;
    uint32_t kp_phase = 0;
    for (int r0 = 0; r0 < k && ok; r0 += piece_rows) {
      const int rows = min(piece_rows, k - r0);
      __syncthreads();                                            // the previous piece has been read
      if (tid == 0) {
        mbar_arrive_expect_tx(bar_kp, (uint32_t)rows * d * 4);
        bulk_load(sm_op, Kp + (size_t)r0 * d, (uint32_t)rows * d * 4, bar_kp);
      }
      {
        bool mine = true;
        if (warp == 4) mine = mbar_wait(bar_kp, kp_phase, prm.status, &abort_flag);
        ok = __syncthreads_and(mine) != 0;
        kp_phase ^= 1;
      }
      if (!ok) break;
      for (int g = warp >> 2; g < (rows >> 5); g += 2) {
        uint32_t h[16];
        const float* src = stage + (size_t)(g * 32) * d + col;
#pragma unroll
        for (int e = 0; e < 16; ++e) {
          const float x0 = src[(2 * e) * d];
          const float x1 = src[(2 * e + 1) * d];
          const float f0 = fmaxf(x0, 0.f) + __expf(fminf(x0, 0.f));      // elu(x) + 1
          const float f1 = fmaxf(x1, 0.f) + __expf(fminf(x1, 0.f));
          const __half2 hh = __floats2half2_rn(f0, f1);
          const float2 back = __half22float2(hh);
          zsum += back.x + back.y;
          h[e] = *reinterpret_cast<const uint32_t*>(&hh);
        }
        tmem_st16(tb + ((r0 + g * 32) >> 1), h);
      }
    }
    // the two threads of a feature add up their sums
    __shared__ float zpart[128];
    if (warp >= 4) zpart[(warp & 3) * 32 + lane] = zsum;
    tmem_wait_st();
    tcgen05_fence_before();
    __syncthreads();
    if (warp < 4) zsum += zpart[warp * 32 + lane];
    if (warp < 4) {
      if (feat < p) prm.weight[(size_t)head * p + feat] = zsum;
      tmem_wait_st();
      tcgen05_fence_before();
    }
  }
  __syncthreads();

  // ---- a = weights x V', streamed in chunks of up to 128 keys; V' = hi + lo in fp16, MN-major slabs
  {
    const uint32_t idesc2 = make_idesc(kFmtF16, 0, /*B MN-major*/ 1, 128, (uint32_t)d);
    for (int jc = 0; jc < nchunks && ok; ++jc) {
      const int rows = min(kK2Chunk, k - (jc_begin + jc) * kK2Chunk);
      wait_stage();
      if (!ok) break;
#pragma unroll 2
      for (int t = 0; t < citers; ++t) {
        const int r = crow0 + t * 8 * rpi;
        if (r < rows) {
          const float4 x = stage_ld(r);
          const __half2 hi0 = __floats2half2_rn(x.x, x.y), hi1 = __floats2half2_rn(x.z, x.w);
          const float2 b0 = __half22float2(hi0), b1 = __half22float2(hi1);
          const __half2 lo0 = __floats2half2_rn(x.x - b0.x, x.y - b0.y);
          const __half2 lo1 = __floats2half2_rn(x.z - b1.x, x.w - b1.y);
          const uint32_t off = sm_op + coff + r * 128 + ((cchunk ^ (r & 7)) << 4);
          asm volatile("st.shared.v2.b32 [%0], {%1, %2};" ::"r"(off), "r"(*reinterpret_cast<const uint32_t*>(&hi0)),
                       "r"(*reinterpret_cast<const uint32_t*>(&hi1)) : "memory");
          asm volatile("st.shared.v2.b32 [%0], {%1, %2};" ::"r"(off + 32768), "r"(*reinterpret_cast<const uint32_t*>(&lo0)),
                       "r"(*reinterpret_cast<const uint32_t*>(&lo1)) : "memory");
        }
      }
      fence_proxy_async_smem();
      __syncthreads();
      if (tid == 0 && jc + 1 < nchunks) stage_chunk(Vp, jc_begin + jc + 1);
      if (tid == 128) {
        tcgen05_fence_after();
        // B: 64-column slabs 16384 B apart, 8-key groups 1024 B apart, 16 keys = 2048 B per step;
        // A: the fp16 weights of these keys, 8 TMEM columns per step
        for (int s2 = 0; s2 < 2; ++s2) {
          for (int q4 = 0; q4 < (rows >> 6); ++q4) {
            const uint64_t bd = make_sdesc(sm_op + s2 * 32768 + q4 * 8192, 16384, 1024, kSwizzle128);
            mma_ts_x4(tmem + kK2OCol, tmem + jc * (kK2Chunk >> 1) + q4 * 32, bd, 128, idesc2,
                      (jc > 0 || s2 > 0 || q4 > 0) ? 1u : 0u);
          }
        }
        mma_commit(bar_mma);
      }
      wait_mma();
    }
  }

  if (tid == 0) grid_launch_dependents();   // only the write-out (and the merge) is left
  // ---- a_i = accumulator / z_i, stored transposed ([d][p], fp16) for stage 3
  if (nsplit == 1) {
    // through shared memory (the staging buffer is free by now): every row owner drops its feature's d
    // values into a [d][128] fp16 tile, then all threads copy the tile out 16 bytes at a time, so a^T
    // leaves in whole 128- or 256-byte runs
    if (warp < 4 && ok) {
      const uint32_t tb = tmem + ((uint32_t)(warp * 32) << 16) + kK2OCol;
      const float inv = 1.f / zsum;
      const uint32_t col_addr = sm_stage + (uint32_t)(warp * 32 + lane) * 2u;
      for (int c = 0; c < d; c += 32) {
        uint32_t r[32];
        tmem_ld32(tb + c, r);
        tmem_wait_ld(r);
#pragma unroll
        for (int e = 0; e < 32; ++e) {
          const unsigned short h = __half_as_ushort(__float2half_rn(__uint_as_float(r[e]) * inv));
          asm volatile("st.shared.u16 [%0], %1;" ::"r"(col_addr + (uint32_t)(c + e) * 256u), "h"(h) : "memory");
        }
        if (prm.a32 && feat < p) {
          float4* arow = reinterpret_cast<float4*>(prm.a32 + ((size_t)head * p + feat) * d + c);
#pragma unroll
          for (int e = 0; e < 32; e += 4)
            arow[e >> 2] = make_float4(__uint_as_float(r[e]) * inv, __uint_as_float(r[e + 1]) * inv,
                                       __uint_as_float(r[e + 2]) * inv, __uint_as_float(r[e + 3]) * inv);
        }
      }
    }
    __syncthreads();
    if (ok) {
      const int live = min(128, p - i0);                    // a multiple of 64
      const int cpr = live >> 3;                            // 16-byte pieces per row
      __half* dst = prm.aT16 + (size_t)head * d * p + i0;
      for (int idx = tid; idx < d * cpr; idx += kK2Threads) {
        const int c = idx / cpr, ch = idx % cpr;
        uint32_t v0, v1, v2, v3;
        asm volatile("ld.shared.v4.b32 {%0, %1, %2, %3}, [%4];"
                     : "=r"(v0), "=r"(v1), "=r"(v2), "=r"(v3) : "r"(sm_stage + (uint32_t)c * 256u + (uint32_t)ch * 16u));
        *reinterpret_cast<uint4*>(dst + (size_t)c * p + ch * 8) = make_uint4(v0, v1, v2, v3);
      }
    }
  } else {
    // partial results of this part of the keys: row 0 = maxima, row 1 = sums, rows 2.. = accumulator
    // columns, each row 128 features wide (consecutive lanes write consecutive words)
    const size_t part_stride = (size_t)(d + 2) * 128;
    float* mine = prm.part + ((size_t)unit * nsplit + sp) * part_stride;
    if (warp < 4 && ok) {
      const int fl = warp * 32 + lane;
      const uint32_t tb = tmem + ((uint32_t)(warp * 32) << 16) + kK2OCol;
      mine[fl] = row_max;
      mine[128 + fl] = zsum;
      for (int c = 0; c < d; c += 32) {
        uint32_t r[32];
        tmem_ld32(tb + c, r);
        tmem_wait_ld(r);
#pragma unroll
        for (int e = 0; e < 32; ++e) mine[(size_t)(2 + c + e) * 128 + fl] = __uint_as_float(r[e]);
      }
    }
    __threadfence();
    __syncthreads();
    __shared__ int last_arrival;
    if (tid == 0) last_arrival = (atomicAdd(prm.counters + unit, 1) == nsplit - 1) ? 1 : 0;
    __syncthreads();
    if (last_arrival && ok) {
      __threadfence();
      // merge: feature fl, half of the d columns per thread; the partial results bypass L1
      const float* all = prm.part + (size_t)unit * nsplit * part_stride;
      const int fl = tid & 127, half = tid >> 7;
      const int f = i0 + fl;
      float m_all = -INFINITY;
#pragma unroll
      for (int q = 0; q < 4; ++q)
        if (q < nsplit) m_all = fmaxf(m_all, __ldcg(all + q * part_stride + fl));
      float scale[4] = {0.f, 0.f, 0.f, 0.f};
      float z_all = 0.f;
#pragma unroll
      for (int q = 0; q < 4; ++q) {
        if (q < nsplit) {
          scale[q] = __expf(__ldcg(all + q * part_stride + fl) - m_all);
          z_all = fmaf(scale[q], __ldcg(all + q * part_stride + 128 + fl), z_all);
        }
      }
      if (half == 0 && f < p) prm.weight[(size_t)head * p + f] = m_all + __logf(z_all);
      const float inv = 1.f / z_all;
      __half* dst = prm.aT16 + (size_t)head * d * p + f;
      // sixteen columns at a time so that up to 64 loads are in flight per thread
      for (int c0 = half * (d >> 1); c0 < (half + 1) * (d >> 1); c0 += 16) {
        float v[4][16];
#pragma unroll
        for (int q = 0; q < 4; ++q) {
          if (q < nsplit) {
#pragma unroll
            for (int e = 0; e < 16; ++e) v[q][e] = __ldcg(all + q * part_stride + (size_t)(2 + c0 + e) * 128 + fl);
          }
        }
#pragma unroll
        for (int e = 0; e < 16; ++e) {
          float acc = 0.f;
#pragma unroll
          for (int q = 0; q < 4; ++q)
            if (q < nsplit) acc = fmaf(scale[q], v[q][e], acc);
          if (f < p) dst[(size_t)(c0 + e) * p] = __float2half_rn(acc * inv);
          if (prm.a32 && f < p) prm.a32[((size_t)head * p + f) * d + c0 + e] = acc * inv;
        }
      }
      if (tid == 0) prm.counters[unit] = 0;
    }
  }
  tcgen05_fence_before();
  __syncthreads();
  if (warp == 4) tmem_dealloc(tmem, 512);
}

}  // namespace flurka

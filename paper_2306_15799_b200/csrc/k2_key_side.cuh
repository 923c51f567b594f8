// Stage 2 on tensor cores: the key-side feature map and the two key-side contractions
// (arxiv 2306.15799, Eq. (2): phi(K')^T V' and, for the normaliser of Appendix D, phi(K')^T 1),
// kept per feature in the log domain:
//
//   PERFORMER   L_ij = w_i . k'_j - |k'_j|^2 / 2          (rows i = features, columns j = projected keys)
//               b_i  = log sum_j exp(L_ij),  a_i = sum_j softmax_j(L_i.) v'_j
//   RNN         f_ij = elu(k'_ji) + 1,  z_i = sum_j f_ij,  a_i = sum_j f_ij v'_j / z_i
//
// One CTA owns 128 features of one head.  K' and V' arrive as fp32 (stage 1's workspace) and are
// split on the fly into bf16 / fp16 terms so that the tensor-core products are fp32-accurate:
// K' = hi + mid + lo (three bf16 terms, exact to 24 bits) against the exact bf16 W, and
// -|k'|^2/2 as three bf16 terms in one extra 16-wide contraction step; V' = hi + lo in fp16.
// L for all k keys sits in TMEM (k <= 512 columns); the thread that owns a row takes its maximum,
// writes exp(L - max) back as fp16 pairs and keeps the sum of the rounded values, so the dominant
// term cancels exactly in a_i.  The second product reads those weights straight from TMEM.
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
  int* status;
};

constexpr int kK2Threads = 256;
// shared memory: W tile (<= 32 KB) | ones 4 KB | -|k'|^2/2 tile 2 KB | three 16 KB operand tiles | barrier
constexpr int kK2SmemBytes = 32768 + 4096 + 2048 + 3 * 16384 + 256 + 1024;
constexpr int kK2OCol = 256;   // TMEM column of the a accumulator

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
  const uint32_t sm_op = sm_nrm + 2048;          // 3 x 16 KB, 1024-aligned
  const uint32_t bar_w = sm_op + 3 * 16384;
  const uint32_t bar_mma = bar_w + 8;
  const uint32_t tmem_slot = bar_w + 16;
  __shared__ int abort_flag;
  __shared__ uint32_t tmem_base_shared;

  const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31, tid = threadIdx.x;
  const int d = prm.d, k = prm.k, p = prm.p;
  const int head = blockIdx.x / prm.ftiles;
  const int i0 = (blockIdx.x % prm.ftiles) * 128;            // first feature of this CTA
  const float* __restrict__ Kp = prm.kpvp + (size_t)head * k * d;
  const float* __restrict__ Vp = prm.kpvp + ((size_t)prm.BH + head) * (size_t)k * d;
  const int kq = d >> 6;                                      // 64-wide blocks of the head dimension
  const int nchunks = k >> 6;                                 // 64 keys per chunk

  if (tid == 0) {
    abort_flag = 0;
    mbar_init(bar_w, 1);
    mbar_init(bar_mma, 1);
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

  // conversion geometry: 4 threads per key row, each a contiguous quarter of the d columns
  const int crow = tid >> 2;                   // 0..63
  const int cseg = (tid & 3) * (d >> 2);       // first column of this thread's segment
  const int cper = d >> 2;                     // 16 or 32 columns

  if (kPerformer) {
    ok = __syncthreads_and(mbar_wait(bar_w, 0, prm.status, &abort_flag)) != 0;
    const uint32_t idesc1 = make_idesc(kFmtBF16, 0, 0, 128, 64);
    for (int jc = 0; jc < nchunks && ok; ++jc) {
      // ---- K' rows jc*64 .. +64: fp32 -> three bf16 tiles (K-major, 128-byte swizzle) and -|k'|^2/2
      const float* src = Kp + (size_t)(jc * 64 + crow) * d + cseg;
      float sq = 0.f;
      for (int c8 = 0; c8 < cper; c8 += 8) {
        const float4 v0 = *reinterpret_cast<const float4*>(src + c8);
        const float4 v1 = *reinterpret_cast<const float4*>(src + c8 + 4);
        const float x[8] = {v0.x, v0.y, v0.z, v0.w, v1.x, v1.y, v1.z, v1.w};
        uint32_t w0[4], w1[4], w2[4];
#pragma unroll
        for (int e = 0; e < 4; ++e) {
          float a = x[2 * e], b = x[2 * e + 1];
          sq = fmaf(a, a, sq);
          sq = fmaf(b, b, sq);
          const __nv_bfloat16 a0 = __float2bfloat16_rn(a), b0 = __float2bfloat16_rn(b);
          a -= __bfloat162float(a0); b -= __bfloat162float(b0);
          const __nv_bfloat16 a1 = __float2bfloat16_rn(a), b1 = __float2bfloat16_rn(b);
          a -= __bfloat162float(a1); b -= __bfloat162float(b1);
          const __nv_bfloat16 a2 = __float2bfloat16_rn(a), b2 = __float2bfloat16_rn(b);
          w0[e] = (uint32_t)__bfloat16_as_ushort(a0) | ((uint32_t)__bfloat16_as_ushort(b0) << 16);
          w1[e] = (uint32_t)__bfloat16_as_ushort(a1) | ((uint32_t)__bfloat16_as_ushort(b1) << 16);
          w2[e] = (uint32_t)__bfloat16_as_ushort(a2) | ((uint32_t)__bfloat16_as_ushort(b2) << 16);
        }
        const int col = cseg + c8;
        const uint32_t off = (uint32_t)(col >> 6) * 8192 + crow * 128 + ((((col & 63) >> 3) ^ (crow & 7)) << 4);
        asm volatile("st.shared.v4.b32 [%0], {%1, %2, %3, %4};" ::"r"(sm_op + off), "r"(w0[0]), "r"(w0[1]), "r"(w0[2]), "r"(w0[3]) : "memory");
        asm volatile("st.shared.v4.b32 [%0], {%1, %2, %3, %4};" ::"r"(sm_op + 16384 + off), "r"(w1[0]), "r"(w1[1]), "r"(w1[2]), "r"(w1[3]) : "memory");
        asm volatile("st.shared.v4.b32 [%0], {%1, %2, %3, %4};" ::"r"(sm_op + 32768 + off), "r"(w2[0]), "r"(w2[1]), "r"(w2[2]), "r"(w2[3]) : "memory");
      }
      sq += __shfl_xor_sync(0xffffffffu, sq, 1);
      sq += __shfl_xor_sync(0xffffffffu, sq, 2);
      if ((tid & 3) == 0) {
        // B operand of the bias step: row j, columns 0..2 = three bf16 terms of -|k'_j|^2/2
        float b = -0.5f * sq;
        const __nv_bfloat16 h0 = __float2bfloat16_rn(b);  b -= __bfloat162float(h0);
        const __nv_bfloat16 h1 = __float2bfloat16_rn(b);  b -= __bfloat162float(h1);
        const __nv_bfloat16 h2 = __float2bfloat16_rn(b);
        const uint32_t a = sm_nrm + (crow >> 3) * 256 + (crow & 7) * 16;
        const uint32_t z = 0;
        asm volatile("st.shared.v4.b32 [%0], {%1, %2, %3, %4};" ::"r"(a),
                     "r"((uint32_t)__bfloat16_as_ushort(h0) | ((uint32_t)__bfloat16_as_ushort(h1) << 16)),
                     "r"((uint32_t)__bfloat16_as_ushort(h2)), "r"(z), "r"(z) : "memory");
        asm volatile("st.shared.v4.b32 [%0], {%1, %2, %3, %4};" ::"r"(a + 128), "r"(z), "r"(z), "r"(z), "r"(z) : "memory");
      }
      fence_proxy_async_smem();
      __syncthreads();
      if (tid == 128) {
        tcgen05_fence_after();
        const int ksteps = d >> 4;
        bool first = true;
        for (int s = 0; s < 3; ++s) {
          for (int ks = 0; ks < ksteps; ++ks) {
            const uint64_t ad = make_sdesc(sm_w + (ks >> 2) * 16384 + (ks & 3) * 32, 16, 1024, kSwizzle128);
            const uint64_t bd = make_sdesc(sm_op + s * 16384 + (ks >> 2) * 8192 + (ks & 3) * 32, 16, 1024, kSwizzle128);
            mma_ss(tmem + jc * 64, ad, bd, idesc1, first ? 0u : 1u);
            first = false;
          }
        }
        const uint64_t ad = make_sdesc(sm_ones, 128, 256, kSwizzleNone);
        const uint64_t bd = make_sdesc(sm_nrm, 128, 256, kSwizzleNone);
        mma_ss(tmem + jc * 64, ad, bd, idesc1, 1u);
        mma_commit(bar_mma);
      }
      // the operand tiles are rewritten for the next chunk: wait until the MMAs have read them
      ok = __syncthreads_and(mbar_wait(bar_mma, mma_phase, prm.status, &abort_flag)) != 0;
      mma_phase ^= 1;
      tcgen05_fence_after();
    }
  }

  // ---- feature weights: one thread per feature row (warps 0..3)
  float zsum = 0.f;
  const int feat = i0 + warp * 32 + lane;                   // valid for warps 0..3
  if (warp < 4 && ok) {
    const uint32_t tb = tmem + ((uint32_t)(warp * 32) << 16);
    if (kPerformer) {
      const float kLog2e = 1.4426950408889634f;
      float mx = -INFINITY;
      for (int c = 0; c < k; c += 32) {
        uint32_t r[32];
        tmem_ld32(tb + c, r);
        tmem_wait_ld();
#pragma unroll
        for (int e = 0; e < 32; ++e) mx = fmaxf(mx, __uint_as_float(r[e]));
      }
      const float shift = mx * kLog2e;
      for (int c = 0; c < k; c += 32) {
        uint32_t r[32], h[16];
        tmem_ld32(tb + c, r);
        tmem_wait_ld();
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
      if (feat < p) prm.weight[(size_t)head * p + feat] = mx + __logf(zsum);
    } else {
      // RNN: f_ij = elu(k'_ji) + 1 for this thread's feature i, all keys j (coalesced over i)
      for (int c = 0; c < k; c += 32) {
        uint32_t h[16];
#pragma unroll
        for (int e = 0; e < 16; ++e) {
          float x0 = 0.f, x1 = 0.f;
          if (feat < p) {
            x0 = Kp[(size_t)(c + 2 * e) * d + feat];
            x1 = Kp[(size_t)(c + 2 * e + 1) * d + feat];
          }
          const float f0 = x0 > 0.f ? x0 + 1.f : __expf(x0);
          const float f1 = x1 > 0.f ? x1 + 1.f : __expf(x1);
          const __half2 hh = __floats2half2_rn(f0, f1);
          const float2 back = __half22float2(hh);
          zsum += back.x + back.y;
          h[e] = *reinterpret_cast<const uint32_t*>(&hh);
        }
        tmem_st16(tb + (c >> 1), h);
      }
      if (feat < p) prm.weight[(size_t)head * p + feat] = zsum;
    }
    tmem_wait_st();
    tcgen05_fence_before();
  }
  __syncthreads();

  // ---- a = weights x V', streamed in chunks of 64 keys; V' = hi + lo in fp16, MN-major slabs
  {
    const uint32_t idesc2 = make_idesc(kFmtF16, 0, /*B MN-major*/ 1, 128, (uint32_t)d);
    for (int jc = 0; jc < nchunks && ok; ++jc) {
      const float* src = Vp + (size_t)(jc * 64 + crow) * d + cseg;
      for (int c8 = 0; c8 < cper; c8 += 8) {
        const float4 v0 = *reinterpret_cast<const float4*>(src + c8);
        const float4 v1 = *reinterpret_cast<const float4*>(src + c8 + 4);
        const float x[8] = {v0.x, v0.y, v0.z, v0.w, v1.x, v1.y, v1.z, v1.w};
        uint32_t w0[4], w1[4];
#pragma unroll
        for (int e = 0; e < 4; ++e) {
          const __half2 hi = __floats2half2_rn(x[2 * e], x[2 * e + 1]);
          const float2 hb = __half22float2(hi);
          const __half2 lo = __floats2half2_rn(x[2 * e] - hb.x, x[2 * e + 1] - hb.y);
          w0[e] = *reinterpret_cast<const uint32_t*>(&hi);
          w1[e] = *reinterpret_cast<const uint32_t*>(&lo);
        }
        const int col = cseg + c8;
        const uint32_t off = (uint32_t)(col >> 6) * 8192 + crow * 128 + ((((col & 63) >> 3) ^ (crow & 7)) << 4);
        asm volatile("st.shared.v4.b32 [%0], {%1, %2, %3, %4};" ::"r"(sm_op + off), "r"(w0[0]), "r"(w0[1]), "r"(w0[2]), "r"(w0[3]) : "memory");
        asm volatile("st.shared.v4.b32 [%0], {%1, %2, %3, %4};" ::"r"(sm_op + 16384 + off), "r"(w1[0]), "r"(w1[1]), "r"(w1[2]), "r"(w1[3]) : "memory");
      }
      fence_proxy_async_smem();
      __syncthreads();
      if (tid == 128) {
        tcgen05_fence_after();
        for (int s = 0; s < 2; ++s) {
#pragma unroll
          for (int ks = 0; ks < 4; ++ks) {
            // B: 64-column slabs 8192 B apart, 8-key groups 1024 B apart, 16 keys = 2048 B per step
            const uint64_t bd = make_sdesc(sm_op + s * 16384 + ks * 2048, 8192, 1024, kSwizzle128);
            mma_ts(tmem + kK2OCol, tmem + jc * 32 + ks * 8, bd, idesc2, (jc > 0 || s > 0 || ks > 0) ? 1u : 0u);
          }
        }
        mma_commit(bar_mma);
      }
      ok = __syncthreads_and(mbar_wait(bar_mma, mma_phase, prm.status, &abort_flag)) != 0;
      mma_phase ^= 1;
      tcgen05_fence_after();
    }
  }

  // ---- a_i = accumulator / z_i, stored transposed ([d][p], fp16) for stage 3
  if (warp < 4 && ok) {
    // whole warps are either inside or outside the p features (p is a multiple of 64); the TMEM
    // loads are warp-wide either way, only the stores are predicated
    const uint32_t tb = tmem + ((uint32_t)(warp * 32) << 16) + kK2OCol;
    const float inv = 1.f / zsum;
    __half* dst = prm.aT16 + (size_t)head * d * p + feat;
    for (int c = 0; c < d; c += 32) {
      uint32_t r[32];
      tmem_ld32(tb + c, r);
      tmem_wait_ld();
      if (feat < p) {
#pragma unroll
        for (int e = 0; e < 32; ++e) dst[(size_t)(c + e) * p] = __float2half_rn(__uint_as_float(r[e]) * inv);
      }
    }
  }
  tcgen05_fence_before();
  __syncthreads();
  if (warp == 4) tmem_dealloc(tmem, 512);
}

}  // namespace flurka

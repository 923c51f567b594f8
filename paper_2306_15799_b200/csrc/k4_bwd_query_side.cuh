// Backward of the query side on tensor cores (bf16; PERFORMER with p = 64, 128, 192 or 256 features and
// d = 64 or 128, RNN with d = 64; a last tile of 64 features is padded to 128 with weights that are exactly zero).
//
// The forward's query side (arxiv 2306.15799, Eq. (2) with the normalised weights of Appendix D) is
//     O_n = sum_i P_ni a_i,    P_n. = softmax_i(l_n.),    l_ni = w_i . q_n + b_i.
// The paper trains through it but prints no backward formulas; by the chain rule, given dO,
//     g_ni = dO_n . a_i,   delta_n = sum_i P_ni g_ni,   c_ni = P_ni (g_ni - delta_n),
//     dq_n = sum_i c_ni w_i,   da_i = sum_n P_ni dO_n,   db_i = sum_n c_ni = a_i . da_i - sum_n P_ni delta_n.
// Per tile of 128 query rows every product is a tcgen05 MMA with fp32 accumulators in TMEM:
//     S = Q W^T + 1 b^T  and  G = dO a^T  (a as two bf16 terms, so g is exact to 2^-17),
//     dQ = C W  (C = bf16 c, the A operand read from TMEM),
//     da += P^T dO  and  (P^T delta) += P^T [delta_hi delta_mid delta_lo]  (P = bf16, written to shared memory
//     by the row owners in the canonical 128-byte-swizzled layout, used as an MN-major A operand),
// in two sweeps over the features, 128 at a time: the first gives each row its log-sum-exp and
// delta_n (running maximum, sum and P-weighted sum of g), the second forms P and c, starting with the step
// whose S and G sweep 1 left in TMEM.  da and P^T delta
// stay in TMEM over all the tiles a CTA has of one head and are added to global memory (atomics) when
// the head changes; db comes from them there.  Two threads per query row (8 warps; each takes 64 of the 128
// features of a step), one MMA issuer, one TMA thread; the phases of a tile follow one another (block
// barriers), nothing here waits for another CTA.
// RNN (kPerformer = false): l_ni = log((elu(q_ni) + 1) z_i), so the weights come from the Q tile in shared
// memory without a product or an exponent, and dq_ni = c_ni elu'(q_ni) / (elu(q_ni) + 1) is stored by the row owner.
// d = 128: TMEM cannot hold dQ and da at full width beside S and G, nor shared memory W and both terms of a
// for 256 features, so every tile is visited twice, once per 64-column half of dQ and da (S, G and the weights
// are formed again), and W, a arrive per step of 128 features.
#pragma once

#include <cuda_bf16.h>

#include "tc_common.cuh"

namespace flurka {

struct K4Params {
  int N, p, BH, H;              // H > 0: Q, dO, dQ are [B,N,H,d]; H == 0: [BH,N,d]
  int d;                        // 64, or 128 (PERFORMER only: see the kernel's header)
  int tiles_per_head, total_tiles;
  const float* weight;          // [BH][p]      b_i
  const float* a32;             // [BH][p][d]   a_i (fp32)
  __nv_bfloat16* dQ;
  float* da;                    // [BH][p][d]   added to
  float* db;                    // [BH][p]      added to
  float2* rowstat;              // d = 128: [total_tiles * 128] (log-sum-exp, delta) of every row, kept from a
                                // tile's first visit for its second
  int* status;
};

constexpr int kK4Threads = 320;
// shared memory: W 32 KB | a_hi 32 KB | a_lo 32 KB | 2 x (Q tile 16 KB, dO tile 16 KB) | P tile 32 KB |
// ones 4 KB | bias 8 KB | delta 4 KB | barriers
constexpr uint32_t kK4W = 0, kK4AHi = 32768, kK4ALo = 65536, kK4In = 98304, kK4P = 163840, kK4Ones = 196608,
                   kK4Bias = 200704, kK4Delta = 208896, kK4Bars = 212992;
constexpr int kK4SmemBytes = 212992 + 256 + 1024;
// TMEM columns: S 0..127 (c as bf16 pairs over 0..31 and 64..95), G 128..255, dQ 256..319, da 320..447 (two
// 128-feature tiles of 64 columns), P^T delta 448..479 (two tiles of 16 columns)
constexpr uint32_t kK4ColG = 128, kK4ColDQ = 256, kK4ColDA = 320, kK4ColDD = 448;

__device__ __forceinline__ uint32_t k4_bf16x2(float lo, float hi) {
  uint32_t r;
  asm("cvt.rn.bf16x2.f32 %0, %2, %1;" : "=r"(r) : "f"(lo), "f"(hi));
  return r;
}
__device__ __forceinline__ float k4_ex2(float x) {
  float y;
  asm("ex2.approx.ftz.f32 %0, %1;" : "=f"(y) : "f"(x));
  return y;
}

// a [BH][p][d] fp32 -> two bf16 terms, [BH][2][p][d]
__global__ void k4_split_a(const float* __restrict__ a32, __nv_bfloat16* __restrict__ abf, int BH, int p, int d) {
  const long long per_head = (long long)p * d;
  const long long total = (long long)BH * per_head;
  for (long long i = (long long)blockIdx.x * blockDim.x + threadIdx.x; i < total; i += (long long)gridDim.x * blockDim.x) {
    const long long h = i / per_head, r = i % per_head;
    const float x = a32[i];
    const __nv_bfloat16 hi = __float2bfloat16_rn(x);
    abf[(h * 2) * per_head + r] = hi;
    abf[(h * 2 + 1) * per_head + r] = __float2bfloat16_rn(x - __bfloat162float(hi));
  }
}

template <bool kPerformer, bool kStream>
__global__ void __launch_bounds__(kK4Threads, 1)
k4_bwd_query_side(const __grid_constant__ CUtensorMap tmQ, const __grid_constant__ CUtensorMap tmDO,
                  const __grid_constant__ CUtensorMap tmW, const __grid_constant__ CUtensorMap tmA,
                  const K4Params prm) {
  using namespace tc;
  extern __shared__ uint8_t smem_raw[];
  const uint32_t base = (smem_u32(smem_raw) + 1023u) & ~1023u;
  uint8_t* base_ptr = smem_raw + (base - smem_u32(smem_raw));
  const uint32_t bars = base + kK4Bars;
  const uint32_t bar_w = bars, bar_head = bars + 8, bar_in = bars + 16 /* [2] */, bar_mma = bars + 32,
                 bar_mma2 = bars + 40, tmem_slot = bars + 48;
  __shared__ int abort_flag;
  __shared__ uint32_t tmem_base_shared;
  __shared__ float stat[2][3][128];             // sweep 1: (maximum, sum, weighted sum) of the two threads of a row

  const int tid = threadIdx.x, warp = tid >> 5, lane = tid & 31;
  const int p = prm.p, nh = (p + 127) >> 7;   // feature tiles of 128; rows of W, a past p are zero-filled by TMA
  constexpr int kd = kStream ? 2 : 1;         // 64-column blocks of the head dimension
  constexpr int d = 64 * kd;
  constexpr bool stream = kStream;            // d = 128: see the header
  const uint32_t bar_step = bars + 56;        // d = 128: W, a of the step's 128 features have landed
  const bool owner = warp >= 2;
  const int q4 = warp & 3, row = q4 * 32 + lane;
  const int fh = (warp - 2) >> 2;              // which 64 of a step's 128 features this row owner takes
  // (RNN: 64 features in all, 32 per thread of a row)
  const int c_lo = kPerformer ? fh * 64 : fh * 32, c_hi = kPerformer ? fh * 64 + 64 : fh * 32 + 32;
  const uint32_t lane_off = (uint32_t)(q4 * 32) << 16;

  // d = 128: a CTA walks its tiles twice, once per 64-column half of dQ and da (visit i: half i / nt, tile i % nt)
  const int t_begin = (int)(((long long)blockIdx.x * prm.total_tiles) / gridDim.x);
  const int t_end = (int)(((long long)(blockIdx.x + 1) * prm.total_tiles) / gridDim.x);
  const int nt = t_end - t_begin;
  const int ntiles = nt * kd;

  if (tid == 0) {
    abort_flag = 0;
    mbar_init(bar_w, 1);
    mbar_init(bar_head, 1);
    mbar_init(bar_in, 1);
    mbar_init(bar_in + 8, 1);
    mbar_init(bar_mma, 1);
    mbar_init(bar_mma2, 1);
    mbar_init(bar_step, 1);
    fence_mbar_init();
  }
  if (warp == 1) {
    tmem_alloc(tmem_slot, 512);
    tmem_relinquish();
  }
  if (warp == 2) {
    // the all-ones A operand of the bias step: [128 x 16] bf16, no swizzle, columns 0..2 are 1
    // (element (r, c) at (r/8)*256 + (c/8)*128 + (r%8)*16 + (c%8)*2 bytes)
    __nv_bfloat16* ones = reinterpret_cast<__nv_bfloat16*>(base_ptr + kK4Ones);
    for (int e = lane; e < 128 * 16; e += 32) {
      const int r = e >> 4, c = e & 15;
      ones[(r >> 3) * 128 + (c >> 3) * 64 + (r & 7) * 8 + (c & 7)] = __float2bfloat16_rn(c < 3 ? 1.f : 0.f);
    }
  }
  if (warp == 3) {
    // the delta operand [16 x 128] (K-major, no swizzle): rows 0..2 are rewritten per tile, the rest stays zero
    uint32_t* dz = reinterpret_cast<uint32_t*>(base_ptr + kK4Delta);
    for (int e = lane; e < 1024; e += 32) dz[e] = 0u;
  }
  if (!kPerformer && warp >= 4) {
    // RNN: features 64..127 of the P tile (its second slab) do not exist: zero, once
    uint32_t* pz = reinterpret_cast<uint32_t*>(base_ptr + kK4P + 16384);
    for (int e = threadIdx.x - 128; e < 4096; e += kK4Threads - 128) pz[e] = 0u;
  }
  fence_proxy_async_smem();
  tcgen05_fence_before();
  __syncthreads();
  tcgen05_fence_after();
  if (tid == 0) {
    uint32_t v;
    asm volatile("ld.shared.u32 %0, [%1];" : "=r"(v) : "r"(tmem_slot));
    tmem_base_shared = v;
  }
  __syncthreads();
  const uint32_t tmem = tmem_base_shared;

  auto load_tile = [&](int i) {
    const int tile = t_begin + i % nt;
    const int head = tile / prm.tiles_per_head;
    const int row0 = (tile % prm.tiles_per_head) * 128;
    if (stream) {
      // one stage: Q as two 64-column slabs, then dO as two
      const uint32_t dst = base + kK4In;
      mbar_arrive_expect_tx(bar_in, 65536u);
      for (int kb = 0; kb < 2; ++kb) {
        const int x = (prm.H > 0 ? (head % prm.H) * 128 : 0) + kb * 64, z = prm.H > 0 ? head / prm.H : head;
        tma_load_3d(dst + kb * 16384, &tmQ, bar_in, x, row0, z);
        tma_load_3d(dst + 32768 + kb * 16384, &tmDO, bar_in, x, row0, z);
      }
      return;
    }
    const uint32_t st = (uint32_t)(i & 1);
    const uint32_t dst = base + kK4In + st * 32768u;
    mbar_arrive_expect_tx(bar_in + 8 * st, 32768u);
    if (prm.H > 0) {
      tma_load_3d(dst, &tmQ, bar_in + 8 * st, (head % prm.H) * 64, row0, head / prm.H);
      tma_load_3d(dst + 16384, &tmDO, bar_in + 8 * st, (head % prm.H) * 64, row0, head / prm.H);
    } else {
      tma_load_3d(dst, &tmQ, bar_in + 8 * st, 0, row0, head);
      tma_load_3d(dst + 16384, &tmDO, bar_in + 8 * st, 0, row0, head);
    }
  };

  // da, P^T delta of one head leave TMEM: thread = feature; db from the identity in the header
  auto flush = [&](int hkey) {
    const int head = hkey % prm.BH, dh = hkey / prm.BH;     // dh: which 64 columns of da these accumulators are
    if (!owner || fh >= nh) return;
    tcgen05_fence_after();
    {
      const int hh = fh;                     // the two groups of row owners take one feature tile each
      uint32_t dd[32];                       // columns 0..2 are this tile's P^T delta terms (the load is 32 wide)
      tmem_ld32(tmem + lane_off + kK4ColDD + hh * 16, dd);
      tmem_wait_ld(dd);
      const int feat = hh * 128 + row;
      const bool live = feat < p;            // (the TMEM loads below are warp-wide: every lane takes them)
      const float* arow = prm.a32 + ((size_t)head * p + (live ? feat : 0)) * d + dh * 64;
      float* darow = prm.da + ((size_t)head * p + (live ? feat : 0)) * d + dh * 64;
      float dot = 0.f;
#pragma unroll 1
      for (int c = 0; c < 64; c += 32) {
        uint32_t r[32];
        tmem_ld32(tmem + lane_off + kK4ColDA + hh * 64 + c, r);
        tmem_wait_ld(r);
#pragma unroll
        for (int e = 0; e < 32; e += 4) {
          const float4 av = *reinterpret_cast<const float4*>(arow + c + e);
          dot = fmaf(av.x, __uint_as_float(r[e]), dot);
          dot = fmaf(av.y, __uint_as_float(r[e + 1]), dot);
          dot = fmaf(av.z, __uint_as_float(r[e + 2]), dot);
          dot = fmaf(av.w, __uint_as_float(r[e + 3]), dot);
        }
#pragma unroll
        for (int e = 0; e < 32; ++e)
          if (live) atomicAdd(darow + c + e, __uint_as_float(r[e]));
      }
      // (both column halves accumulate P^T delta; it is subtracted once)
      const float pd = dh == 0 ? __uint_as_float(dd[0]) + __uint_as_float(dd[1]) + __uint_as_float(dd[2]) : 0.f;
      if (live) atomicAdd(prm.db + (size_t)head * p + feat, dot - pd);
    }
    tcgen05_fence_before();
  };

  bool ok = true;
  uint32_t ph_mma = 0, ph_mma2 = 0, ph_head = 0, ph_step = 0;
  int head_prev = -1;
  bool first_of_head = true;
  bool pre_issued = false;        // this tile's first S and G were issued at the end of the previous tile
  const float kLog2e = 1.4426950408889634f;
  const uint32_t idescS = make_idesc(kFmtBF16, 0, 0, 128, 128);   // S, G: both operands K-major
  const uint32_t idescQ = make_idesc(kFmtBF16, 0, 1, 128, 64);    // dQ: A from TMEM, W as an MN-major B
  const uint32_t idescA = make_idesc(kFmtBF16, 1, 1, 128, 64);    // da: P^T (MN-major A) x dO (MN-major B)
  const uint32_t idescD = make_idesc(kFmtBF16, 1, 0, 128, 16);    // P^T delta: delta as a K-major B

  if (ntiles > 0 && tid == 0) {
    prefetch_tmap(&tmQ);
    prefetch_tmap(&tmDO);
    prefetch_tmap(&tmW);
    prefetch_tmap(&tmA);
    if (kPerformer && !stream) {
      mbar_arrive_expect_tx(bar_w, (uint32_t)nh * 16384u);
      tma_load_2d(base + kK4W, &tmW, bar_w, 0, 0);
    }
    if (!stream) load_tile(0);
  }
  if (kPerformer && !stream && ntiles > 0) {
    const bool mine = mbar_wait(bar_w, 0, prm.status, &abort_flag);
    ok = __syncthreads_and(mine) != 0;
  }

  for (int i = 0; i < ntiles && ok; ++i) {
    const int dh = i / nt;                                    // which 64 columns of dQ, da this visit is for (d = 128)
    const int tile = t_begin + i % nt;
    // second visit of a tile: its rows' log-sum-exp and delta are on record, sweep 1 is not done again
    const bool have_stats = stream && dh == 1;
    const int head = tile / prm.tiles_per_head;
    const int hkey = dh * prm.BH + head;
    const int row0 = (tile % prm.tiles_per_head) * 128;
    const uint32_t st = stream ? 0u : (uint32_t)(i & 1);
    const uint32_t sm_q = base + kK4In + st * 32768u, sm_do = sm_q + (stream ? 32768u : 16384u);

    if (hkey != head_prev) {
      // every MMA issued so far has completed (the last wait of the previous tile), so the accumulators
      // of the old head can leave and its operands can be replaced
      if (head_prev >= 0) flush(head_prev);
      __syncthreads();
      if (tid == 0 && !stream) {
        mbar_arrive_expect_tx(bar_head, 2u * (uint32_t)nh * 16384u);
        tma_load_3d(base + kK4AHi, &tmA, bar_head, 0, 0, head * 2);
        tma_load_3d(base + kK4ALo, &tmA, bar_head, 0, 0, head * 2 + 1);
      }
      if (!kPerformer && warp == 1) {
        // RNN: the weight of feature i is (elu(q_ni) + 1) z_i; z_i / max z as floats where the bias operand would be
        const float* wv = prm.weight + (size_t)head * p;
        float mxz = 0.f;
        for (int f = lane; f < p; f += 32) mxz = fmaxf(mxz, wv[f]);
#pragma unroll
        for (int o = 16; o > 0; o >>= 1) mxz = fmaxf(mxz, __shfl_xor_sync(0xffffffffu, mxz, o));
        float* zs = reinterpret_cast<float*>(base_ptr + kK4Bias);
        const float inv = 1.f / mxz;
        for (int f = lane; f < 128; f += 32) zs[f] = f < p ? wv[f] * inv : 0.f;
      }
      if (kPerformer && warp == 1) {
        // bias[f][c], c < 16, no swizzle: b_f - max b as three bf16 terms in columns 0..2
        const float* wv = prm.weight + (size_t)head * p;
        float mx = -INFINITY;
        for (int f = lane; f < p; f += 32) mx = fmaxf(mx, wv[f]);
#pragma unroll
        for (int o = 16; o > 0; o >>= 1) mx = fmaxf(mx, __shfl_xor_sync(0xffffffffu, mx, o));
        __nv_bfloat16* bias = reinterpret_cast<__nv_bfloat16*>(base_ptr + kK4Bias);
        for (int f = lane; f < 256; f += 32) {
          float b = (f < p) ? wv[f] - mx : 0.f;
          const __nv_bfloat16 h0 = __float2bfloat16_rn(b);  b -= __bfloat162float(h0);
          const __nv_bfloat16 h1 = __float2bfloat16_rn(b);  b -= __bfloat162float(h1);
          const __nv_bfloat16 h2 = __float2bfloat16_rn(b);
          __nv_bfloat16* rowp = bias + (f >> 3) * 128 + (f & 7) * 8;
          rowp[0] = h0; rowp[1] = h1; rowp[2] = h2;
#pragma unroll
          for (int c = 3; c < 8; ++c) rowp[c] = __float2bfloat16_rn(0.f);
#pragma unroll
          for (int c = 0; c < 8; ++c) rowp[64 + c] = __float2bfloat16_rn(0.f);
        }
        fence_proxy_async_smem();
      }
      const bool mine = stream ? true : mbar_wait(bar_head, ph_head, prm.status, &abort_flag);
      if (!stream) ph_head ^= 1;
      ok = __syncthreads_and(mine) != 0;
      if (!ok) break;
      head_prev = hkey;
      first_of_head = true;
    }
    // the other stage held tile i-1, which is complete: fetch tile i+1 into it (d = 128: one stage, this tile now)
    if (tid == 0 && !stream && i + 1 < ntiles) load_tile(i + 1);
    if (tid == 0 && stream) load_tile(i);
    {
      const bool mine = mbar_wait(bar_in + 8 * st, (stream ? (uint32_t)i : (uint32_t)(i >> 1)) & 1u, prm.status, &abort_flag);
      ok = __syncthreads_and(mine) != 0;
      if (!ok) break;
    }

    // d = 128: W and the two terms of a for the step's 128 features (96 KB) come in before every step; every
    // product that read the previous step's is complete by then
    uint32_t step_ok = 1;
    auto load_step = [&](int h) {
      if (tid == 0) {
        mbar_arrive_expect_tx(bar_step, 98304u);
        for (int kb = 0; kb < 2; ++kb) {
          tma_load_2d(base + kK4W + kb * 16384, &tmW, bar_step, kb * 64, h * 128);
          tma_load_3d(base + kK4AHi + kb * 16384, &tmA, bar_step, kb * 64, h * 128, head * 2);
          tma_load_3d(base + kK4ALo + kb * 16384, &tmA, bar_step, kb * 64, h * 128, head * 2 + 1);
        }
      }
      const bool mine = mbar_wait(bar_step, ph_step, prm.status, &abort_flag);
      ph_step ^= 1;
      step_ok = __syncthreads_and(mine) != 0;
    };
    auto issue_sg_from = [&](int h, uint32_t sm_q, uint32_t sm_do) {
      tcgen05_fence_after();
      // rows of the step's features: at h * 16384 in the resident tiles (d = 64), at 0 in the step's own (d = 128);
      // 64-column blocks of the head dimension 16384 B apart
      const uint32_t fo = stream ? 0u : (uint32_t)h * 16384u;
      if (kPerformer) {
        for (int kb = 0; kb < kd; ++kb) {
          const uint64_t aq = make_sdesc(sm_q + kb * 16384, 16, 1024, kSwizzle128);
          const uint64_t bw = make_sdesc(base + kK4W + fo + kb * 16384, 16, 1024, kSwizzle128);
          mma_ss_x4(tmem, aq, bw, 2, 2, idescS, kb > 0 ? 1u : 0u);
        }
        const uint64_t a1 = make_sdesc(base + kK4Ones, 128, 256, kSwizzleNone);
        const uint64_t b1 = make_sdesc(base + kK4Bias + h * 4096, 128, 256, kSwizzleNone);
        mma_ss(tmem, a1, b1, idescS, 1u);
      }
      const uint32_t idescG = kPerformer ? idescS : make_idesc(kFmtBF16, 0, 0, 128, 64);   // RNN: 64 features
      for (int kb = 0; kb < kd; ++kb) {
        const uint64_t ag = make_sdesc(sm_do + kb * 16384, 16, 1024, kSwizzle128);
        const uint64_t bh = make_sdesc(base + kK4AHi + fo + kb * 16384, 16, 1024, kSwizzle128);
        const uint64_t bl = make_sdesc(base + kK4ALo + fo + kb * 16384, 16, 1024, kSwizzle128);
        mma_ss_x4(tmem + kK4ColG, ag, bh, 2, 2, idescG, kb > 0 ? 1u : 0u);
        mma_ss_x4(tmem + kK4ColG, ag, bl, 2, 2, idescG, 1u);
      }
      mma_commit(bar_mma);
    };
    auto issue_sg = [&](int h) { issue_sg_from(h, sm_q, sm_do); };

    // RNN: the un-normalised weights (elu(q_ni) + 1) z_i / max z of 32 features (i = c .. c + 31 = columns of
    // this thread's row of the Q tile, which is 128-byte swizzled) and the factor elu'(q) / (elu(q) + 1)
    auto rnn_weights = [&](int c, float (&pv)[32], float (&ratio)[32]) {
      const float* zs = reinterpret_cast<const float*>(base_ptr + kK4Bias);
#pragma unroll
      for (int g = 0; g < 4; ++g) {
        const uint32_t ch = (uint32_t)((c >> 3) + g);
        uint32_t w4[4];
        asm volatile("ld.shared.v4.b32 {%0, %1, %2, %3}, [%4];" : "=r"(w4[0]), "=r"(w4[1]), "=r"(w4[2]), "=r"(w4[3])
                     : "r"(sm_q + (uint32_t)row * 128u + ((ch ^ (uint32_t)(row & 7)) << 4)));
#pragma unroll
        for (int e = 0; e < 4; ++e) {
          const float x0 = __uint_as_float(w4[e] << 16), x1 = __uint_as_float(w4[e] & 0xffff0000u);
          const int f = 8 * g + 2 * e;
          pv[f] = (x0 > 0.f ? x0 + 1.f : __expf(x0)) * zs[c + f];
          pv[f + 1] = (x1 > 0.f ? x1 + 1.f : __expf(x1)) * zs[c + f + 1];
          ratio[f] = x0 > 0.f ? 1.f / (x0 + 1.f) : 1.f;
          ratio[f + 1] = x1 > 0.f ? 1.f / (x1 + 1.f) : 1.f;
        }
      }
    };
    // ------------------------------------------------------------ sweep 1: log-sum-exp and delta of each row
    float mx = -INFINITY, den = 0.f, num = 0.f;     // mx in the base-2 domain
    for (int h = 0; h < nh && ok && !have_stats; ++h) {
      if (stream) {
        load_step(h);
        if (!step_ok) { ok = false; break; }
      }
      if (!(pre_issued && h == 0) && warp == 1 && elect_one()) issue_sg(h);
      bool mine = true;
      if (owner) {
        mine = mbar_wait(bar_mma, ph_mma, prm.status, &abort_flag);
        // (this thread's 64 features of the step lie past p: padding, weight zero; the same for the whole warp)
        if (mine && (!kPerformer || h * 128 + fh * 64 < p)) {
          tcgen05_fence_after();
#pragma unroll 1
          for (int c = c_lo; c < c_hi; c += 32) {
            uint32_t rs[32], rg[32];
            if (!kPerformer) {
              // no exponent to stabilise: the weights are products of bounded factors
              float pv[32], ratio[32];
              tmem_ld32(tmem + lane_off + kK4ColG + c, rg);
              rnn_weights(c, pv, ratio);
              tmem_wait_ld(rg);
              mx = 0.f;
#pragma unroll
              for (int e = 0; e < 32; ++e) {
                den += pv[e];
                num = fmaf(pv[e], __uint_as_float(rg[e]), num);
              }
              continue;
            }
            tmem_ld32(tmem + lane_off + c, rs);
            tmem_ld32(tmem + lane_off + kK4ColG + c, rg);
            tmem_wait_ld(rs);
            tmem_wait_ld(rg);
            float cm = -INFINITY;
#pragma unroll
            for (int e = 0; e < 32; e += 2) cm = fmax3(cm, __uint_as_float(rs[e]), __uint_as_float(rs[e + 1]));
            const float nm = fmaxf(mx, cm * kLog2e);
            const float sc = k4_ex2(mx - nm);
            den *= sc;
            num *= sc;
            mx = nm;
#pragma unroll
            for (int e = 0; e < 32; ++e) {
              const float pe = k4_ex2(fmaf(__uint_as_float(rs[e]), kLog2e, -mx));
              den += pe;
              num = fmaf(pe, __uint_as_float(rg[e]), num);
            }
          }
          tcgen05_fence_before();
        }
      }
      ph_mma ^= 1;
      ok = __syncthreads_and(mine) != 0;          // S, G have been read out
    }
    if (!ok) break;
    // the two threads of a row put their parts together (both in the same order, so they agree to the bit)
    if (owner && !have_stats) { stat[fh][0][row] = mx; stat[fh][1][row] = den; stat[fh][2][row] = num; }
    __syncthreads();
    if (owner && !have_stats) {
      const float m0 = stat[0][0][row], m1 = stat[1][0][row];
      const float nm = fmaxf(m0, m1);
      const float s0 = k4_ex2(m0 - nm), s1 = k4_ex2(m1 - nm);
      mx = nm;
      den = fmaf(stat[0][1][row], s0, stat[1][1][row] * s1);
      num = fmaf(stat[0][2][row], s0, stat[1][2][row] * s1);
    }
    float lse2 = mx + __log2f(den);
    float delta = num / den;
    if (stream && owner) {
      float2* rs2 = prm.rowstat + (size_t)tile * 128 + row;
      if (have_stats) {
        const float2 v = *rs2;
        lse2 = v.x;
        delta = v.y;
      } else if (fh == 0) {
        *rs2 = make_float2(lse2, delta);
      }
    }
    if (owner && fh == 0) {
      // delta_n as three bf16 terms: element (c, n) of the [16 x 128] operand at (n/8)*128 + c*16 + (n%8)*2 bytes
      __nv_bfloat16* dt = reinterpret_cast<__nv_bfloat16*>(base_ptr + kK4Delta) + (row >> 3) * 64 + (row & 7);
      float r = delta;
      const __nv_bfloat16 d0 = __float2bfloat16_rn(r);  r -= __bfloat162float(d0);
      const __nv_bfloat16 d1 = __float2bfloat16_rn(r);  r -= __bfloat162float(d1);
      const __nv_bfloat16 d2 = __float2bfloat16_rn(r);
      dt[0] = d0; dt[8] = d1; dt[16] = d2;
    }

    // ------------------------------------------------------------ sweep 2: P, c and the three products they feed
    // (last step first: its S and G are still in TMEM from sweep 1, and at d = 128 its W is still in shared memory)
    for (int hi = 0; hi < nh && ok; ++hi) {
      const int h = nh - 1 - hi;
      const bool reuse = hi == 0 && !have_stats;
      if (stream && !reuse) {
        load_step(h);
        if (!step_ok) { ok = false; break; }
      }
      if (!reuse && warp == 1 && elect_one()) issue_sg(h);
      bool mine = true;
      if (owner) {
        if (!reuse) mine = mbar_wait(bar_mma, ph_mma, prm.status, &abort_flag);
        if (mine) {
          tcgen05_fence_after();
          const uint32_t prow = base + kK4P + (uint32_t)row * 128u;
#pragma unroll 1
          for (int c = c_lo; c < c_hi; c += 32) {
            uint32_t rs[32], rg[32], cw[16];
            const uint32_t slab = prow + (uint32_t)(c >> 6) * 16384u;
            // features past p (padding of the last tile): P and c exactly zero
            const float keep = (!kPerformer || h * 128 + fh * 64 < p) ? 1.f : 0.f;
            if (!kPerformer) {
              // RNN (p = d = 64): P = weights / their sum; dq_ni = c_ni elu'(q_ni) / (elu(q_ni) + 1) needs no
              // product, so this thread stores its 32 columns of the dQ row here
              float pv[32], ratio[32];
              tmem_ld32(tmem + lane_off + kK4ColG + c, rg);
              rnn_weights(c & 63, pv, ratio);
              tmem_wait_ld(rg);
              const float sc = keep / den;
              const bool store = keep != 0.f && row0 + row < prm.N;
              __nv_bfloat16* orow = prm.H > 0
                  ? prm.dQ + (((size_t)(head / prm.H) * prm.N + row0 + row) * prm.H + (size_t)(head % prm.H)) * 64
                  : prm.dQ + ((size_t)head * prm.N + row0 + row) * 64;
#pragma unroll
              for (int g = 0; g < 4; ++g) {
                uint32_t pw[4], dq[4];
#pragma unroll
                for (int e = 0; e < 4; ++e) {
                  const int j = 8 * g + 2 * e;
                  const float p0 = pv[j] * sc, p1 = pv[j + 1] * sc;
                  pw[e] = k4_bf16x2(p0, p1);
                  dq[e] = k4_bf16x2(p0 * (__uint_as_float(rg[j]) - delta) * ratio[j],
                                    p1 * (__uint_as_float(rg[j + 1]) - delta) * ratio[j + 1]);
                }
                const uint32_t chunk = (uint32_t)(((c & 32) >> 3) + g);
                asm volatile("st.shared.v4.b32 [%0], {%1, %2, %3, %4};" ::"r"(slab + ((chunk ^ (uint32_t)(row & 7)) << 4)),
                             "r"(pw[0]), "r"(pw[1]), "r"(pw[2]), "r"(pw[3]) : "memory");
                if (store) *reinterpret_cast<uint4*>(orow + (c & 63) + 8 * g) = make_uint4(dq[0], dq[1], dq[2], dq[3]);
              }
              continue;
            }
            tmem_ld32(tmem + lane_off + c, rs);
            tmem_ld32(tmem + lane_off + kK4ColG + c, rg);
            tmem_wait_ld(rs);
            tmem_wait_ld(rg);
#pragma unroll
            for (int g = 0; g < 4; ++g) {
              uint32_t pw[4];
#pragma unroll
              for (int e = 0; e < 4; ++e) {
                const int j = 8 * g + 2 * e;
                const float p0 = keep * k4_ex2(fmaf(__uint_as_float(rs[j]), kLog2e, -lse2));
                const float p1 = keep * k4_ex2(fmaf(__uint_as_float(rs[j + 1]), kLog2e, -lse2));
                pw[e] = k4_bf16x2(p0, p1);
                cw[4 * g + e] = k4_bf16x2(p0 * (__uint_as_float(rg[j]) - delta), p1 * (__uint_as_float(rg[j + 1]) - delta));
              }
              const uint32_t chunk = (uint32_t)(((c & 32) >> 3) + g);
              asm volatile("st.shared.v4.b32 [%0], {%1, %2, %3, %4};" ::"r"(slab + ((chunk ^ (uint32_t)(row & 7)) << 4)),
                           "r"(pw[0]), "r"(pw[1]), "r"(pw[2]), "r"(pw[3]) : "memory");
            }
            // over this thread's own (already read) part of S: features 0..63 at columns 0..31, 64..127 at 64..95
            tmem_st16(tmem + lane_off + fh * 64 + ((c & 63) >> 1), cw);
          }
          if (kPerformer) tmem_wait_st();
          fence_proxy_async_smem();
          tcgen05_fence_before();
        }
      }
      if (!reuse) ph_mma ^= 1;
      ok = __syncthreads_and(mine) != 0;
      if (!ok) break;
      if (warp == 1 && elect_one()) {
        tcgen05_fence_after();
        // dQ (+)= c W: 128 features = 8 steps of 16, A 8 columns per step, B 16 rows of W per step
        for (int j = 0; kPerformer && j < 2; ++j) {
          // W rows of the step's features, the 64 columns this visit owns
          const uint64_t bw = make_sdesc(base + kK4W + (stream ? dh : h) * 16384 + j * 8192, 8192, 1024, kSwizzle128);
          mma_ts_x4(tmem + kK4ColDQ, tmem + j * 64, bw, 128, idescQ, (hi > 0 || j > 0) ? 1u : 0u);
        }
        // da_h (+)= P_h^T dO and (P^T delta)_h: 128 rows = 8 steps of 16 rows (2048 B of P and of dO, 256 B of delta)
        for (int j = 0; j < 2; ++j) {
          const uint64_t ap = make_sdesc(base + kK4P + j * 8192, 16384, 1024, kSwizzle128);
          const uint64_t bo = make_sdesc(sm_do + (stream ? dh * 16384 : 0) + j * 8192, 8192, 1024, kSwizzle128);
          mma_ss_x4(tmem + kK4ColDA + h * 64, ap, bo, 128, 128, idescA, (!first_of_head || j > 0) ? 1u : 0u);
          const uint64_t bd = make_sdesc(base + kK4Delta + j * 1024, 128, 2048, kSwizzleNone);
          mma_ss_x4(tmem + kK4ColDD + h * 16, ap, bd, 128, 16, idescD, (!first_of_head || j > 0) ? 1u : 0u);
        }
        mma_commit(bar_mma2);
      }
      // c, P and (after the last half) dQ: wait for these products before anything is overwritten or read
      mine = mbar_wait(bar_mma2, ph_mma2, prm.status, &abort_flag);
      ph_mma2 ^= 1;
      ok = __syncthreads_and(mine) != 0;
    }
    if (!ok) break;
    first_of_head = false;
    // the next tile's first S and G (same head, its Q and dO already fetched) can run under this tile's dQ read-out:
    // every product that used the S and G columns is complete
    pre_issued = false;
    if (!stream && i + 1 < ntiles && (t_begin + i + 1) / prm.tiles_per_head == head) {
      pre_issued = true;
      if (warp == 1) {
        const uint32_t nst = (uint32_t)((i + 1) & 1);
        const bool landed = mbar_wait(bar_in + 8 * nst, (uint32_t)((i + 1) >> 1) & 1u, prm.status, &abort_flag);
        if (__all_sync(0xffffffffu, landed ? 1 : 0) && elect_one()) {
          const uint32_t nq = base + kK4In + nst * 32768u;
          issue_sg_from(0, nq, nq + 16384u);
        }
      }
    }

    // ------------------------------------------------------------ dQ rows (32 columns per thread)
    if (kPerformer && owner) {
      tcgen05_fence_after();
      uint32_t ra[32];
      tmem_ld32(tmem + lane_off + kK4ColDQ + fh * 32, ra);
      tmem_wait_ld(ra);
      tcgen05_fence_before();
      if (row0 + row < prm.N) {
        __nv_bfloat16* orow = prm.H > 0
            ? prm.dQ + (((size_t)(head / prm.H) * prm.N + row0 + row) * prm.H + (size_t)(head % prm.H)) * d
            : prm.dQ + ((size_t)head * prm.N + row0 + row) * d;
        orow += dh * 64 + fh * 32;
#pragma unroll
        for (int g = 0; g < 4; ++g) {
          uint4 v;
          v.x = k4_bf16x2(__uint_as_float(ra[g * 8 + 0]), __uint_as_float(ra[g * 8 + 1]));
          v.y = k4_bf16x2(__uint_as_float(ra[g * 8 + 2]), __uint_as_float(ra[g * 8 + 3]));
          v.z = k4_bf16x2(__uint_as_float(ra[g * 8 + 4]), __uint_as_float(ra[g * 8 + 5]));
          v.w = k4_bf16x2(__uint_as_float(ra[g * 8 + 6]), __uint_as_float(ra[g * 8 + 7]));
          *reinterpret_cast<uint4*>(orow + g * 8) = v;
        }
      }
    }
    __syncthreads();      // dQ has been read: the next tile may overwrite it
  }
  if (ok && head_prev >= 0) flush(head_prev);
  tcgen05_fence_before();
  __syncthreads();
  if (warp == 1) tmem_dealloc(tmem, 512);
}

}  // namespace flurka

// Backward of the down-projection (arxiv 2306.15799, Eq. (2): K' = E K, V' = F V) on tensor cores:
//
//   kMode 0   dK_h = E^T dK'_h,  dV_h = F^T dV'_h        all heads at once: [N x k] x [k x BH d]
//   kMode 1   dE = sum_h dK'_h K_h^T,  dF = sum_h dV'_h V_h^T        [k x BH d] x [BH d x N]
//
// The fp32 dK', dV' of the key side are first split into two bf16 terms (hi + lo, exact to 2^-17), laid
// out as one matrix per projection, `split` = [2][k][2 BH d] (term-major along the row), which is the
// K-major A operand of kMode 1 and, seen through a tensor map with 64-row boxes, the MN-major B operand of
// kMode 0.  E, F are read as they lie ([k][N]: an MN-major A operand for kMode 0), K, V as they lie
// ([.., N, d]: a K-major B operand for kMode 1).  One CTA owns a tile of outputs (K5Shape below) and the
// whole contraction: a TMA ring, one thread issuing tcgen05.mma (M = 128, N = 256, K = 16) into TMEM, four
// warps storing bf16 through swizzled slabs and TMA stores of whole lines.
#pragma once

#include <cuda_bf16.h>

#include "tc_common.cuh"

namespace flurka {

struct K5Params {
  int N, k, d, BH, H;        // H > 0: K, V, dK, dV are [B,N,H,d]
  int row_blocks, col_groups;
  int* status;
};

// kMode 0 has a short contraction (2 k / 64 chunks) and a long epilogue: 128 x 256 outputs per CTA and two
// 48 KB stages, so that two CTAs share an SM and one's epilogue runs under the other's MMAs; kMode 1 has a
// long contraction: 256 x 256 outputs and three 64 KB stages; kMode 2 is kMode 1 with 128 x 256 outputs and four
// 48 KB stages, for shapes whose dE, dF have too few 256 x 256 tiles to occupy the SMs (each CTA is then bound
// by the latency of its ring, so more CTAs with more, smaller stages in flight go faster)
template <int kMode> struct K5Shape {
  static constexpr int kRows = kMode == 1 ? 256 : 128;
  static constexpr int kStages = kMode == 0 ? 2 : (kMode == 1 ? 3 : 4);
  static constexpr int kABytes = kRows * 128;                       // 64 contraction elements per row
  static constexpr int kStageBytes = kABytes + 32768;
  static constexpr int kSmemBytes = kStages * kStageBytes + 1024 + 256;
  static constexpr int kTmemCols = kRows * 2;
  static constexpr int kCtasPerSm = kMode == 0 ? 2 : 1;
};
constexpr int kK5Threads = 192;

// dK', dV' [2][BH][k][d] fp32 -> split [2][k][2][BH][d] bf16 (hi terms of all heads, then lo terms)
__global__ void k5_split_rows(const float* __restrict__ src, __nv_bfloat16* __restrict__ dst, int BH, int k, int d) {
  const long long total = (long long)2 * BH * k * (d >> 2);
  for (long long i = (long long)blockIdx.x * blockDim.x + threadIdx.x; i < total; i += (long long)gridDim.x * blockDim.x) {
    const int c4 = (int)(i % (d >> 2)) * 4;
    long long r = i / (d >> 2);
    const int kk = (int)(r % k); r /= k;
    const int h = (int)(r % BH);
    const int z = (int)(r / BH);
    const float4 x = *reinterpret_cast<const float4*>(src + (((size_t)z * BH + h) * k + kk) * d + c4);
    const float v[4] = {x.x, x.y, x.z, x.w};
    __nv_bfloat16 hi[4], lo[4];
#pragma unroll
    for (int e = 0; e < 4; ++e) {
      hi[e] = __float2bfloat16_rn(v[e]);
      lo[e] = __float2bfloat16_rn(v[e] - __bfloat162float(hi[e]));
    }
    __nv_bfloat16* row = dst + ((size_t)z * k + kk) * ((size_t)2 * BH * d) + (size_t)h * d + c4;
    *reinterpret_cast<uint2*>(row) = *reinterpret_cast<const uint2*>(hi);
    *reinterpret_cast<uint2*>(row + (size_t)BH * d) = *reinterpret_cast<const uint2*>(lo);
  }
}

// tmP0/tmP1: E, F (kMode 0: boxes of 64 n x 64 k) or K, V (kMode 1: boxes of 64 c x 256 n);
// tmS: the split matrix (kMode 0: boxes of 64 x 64; kMode 1: boxes of 64 x 128 rows);
// tmO0/tmO1: dK, dV (boxes of 64 c x 32 n) or dE, dF (boxes of 64 n x 32 k)
template <int kMode>
__global__ void __launch_bounds__(kK5Threads, K5Shape<kMode>::kCtasPerSm)
k5_bwd_projections(const __grid_constant__ CUtensorMap tmP0, const __grid_constant__ CUtensorMap tmP1,
                   const __grid_constant__ CUtensorMap tmS, const __grid_constant__ CUtensorMap tmO0,
                   const __grid_constant__ CUtensorMap tmO1, const K5Params p) {
  using namespace tc;
  extern __shared__ uint8_t smem_raw[];
  const uint32_t smem_base = (smem_u32(smem_raw) + 1023u) & ~1023u;
  constexpr int kK5Stages = K5Shape<kMode>::kStages, kK5StageBytes = K5Shape<kMode>::kStageBytes;
  constexpr int kRows = K5Shape<kMode>::kRows, kABytes = K5Shape<kMode>::kABytes;
  const uint32_t bar_base = smem_base + kK5Stages * kK5StageBytes;
  const uint32_t bar_full = bar_base;                 // [<= 4]
  const uint32_t bar_empty = bar_base + 32;           // [<= 4]
  const uint32_t bar_accum = bar_base + 64;
  const uint32_t tmem_slot = bar_base + 80;
  __shared__ int abort_flag;
  __shared__ uint32_t tmem_base_shared;

  const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
  int idx = blockIdx.x;
  const int cg = idx % p.col_groups; idx /= p.col_groups;
  const int rb = idx % p.row_blocks; idx /= p.row_blocks;
  const int z = idx;                                        // 0: keys / E, 1: values / F
  const int M = kMode == 0 ? p.N : p.k;                     // output rows
  const int NC = kMode == 0 ? p.BH * p.d : p.N;             // output columns
  const int rows = min(kRows, M - rb * kRows);
  const int mt = (rows + 127) >> 7;
  const int ncols = kMode == 0 ? min(256, NC - cg * 256) : 256;   // kMode 1: columns past N are zero and clipped
  const int hd = p.BH * p.d;
  const int per_term = kMode == 0 ? (p.k >> 6) : (hd >> 6); // 64-wide contraction chunks per bf16 term
  const int nchunks = 2 * per_term;
  const CUtensorMap* tmP = z ? &tmP1 : &tmP0;
  const CUtensorMap* tmO = z ? &tmO1 : &tmO0;

  if (threadIdx.x == 0) {
    abort_flag = 0;
    for (int i = 0; i < kK5Stages; ++i) {
      mbar_init(bar_full + 8 * i, 1);
      mbar_init(bar_empty + 8 * i, 1);
    }
    mbar_init(bar_accum, 1);
    fence_mbar_init();
  }
  if (warp == 1) {
    tmem_alloc(tmem_slot, K5Shape<kMode>::kTmemCols);
    tmem_relinquish();
  }
  tcgen05_fence_before();
  __syncthreads();
  tcgen05_fence_after();
  if (threadIdx.x == 0) {
    uint32_t v;
    asm volatile("ld.shared.u32 %0, [%1];" : "=r"(v) : "r"(tmem_slot));
    tmem_base_shared = v;
  }
  __syncthreads();
  const uint32_t tmem = tmem_base_shared;

  if (warp == 0) {
    if (elect_one()) {
      // ------------------------------------------------ TMA producer
      prefetch_tmap(tmP);
      prefetch_tmap(&tmS);
      const uint32_t tx_bytes = kMode == 0 ? (uint32_t)(mt * 16384 + (ncols >> 6) * 8192) : (uint32_t)(mt * 16384 + 32768);
      int issued = 0;
      bool ok = true;
      for (int it = 0; it < nchunks && ok; ++it) {
        const int st = it % kK5Stages;
        if (it >= kK5Stages) ok = mbar_wait(bar_empty + 8 * st, ((it / kK5Stages) - 1) & 1, p.status, &abort_flag);
        if (!ok) break;
        const uint32_t a_dst = smem_base + st * kK5StageBytes;
        const uint32_t b_dst = a_dst + kABytes;
        const uint32_t bar = bar_full + 8 * st;
        const int t = it / per_term, c = it % per_term;
        mbar_arrive_expect_tx(bar, tx_bytes);
        if (kMode == 0) {
          // A: rows n of E^T as two 64-row slabs per M-tile (n contiguous: MN-major); B: 64 rows of the split matrix
          for (int m = 0; m < mt; ++m)
            for (int s = 0; s < 2; ++s)
              tma_load_2d(a_dst + m * 16384 + s * 8192, tmP, bar, rb * kRows + m * 128 + s * 64, c << 6);
          for (int b = 0; b < (ncols >> 6); ++b)
            tma_load_3d(b_dst + b * 8192, &tmS, bar, t * hd + cg * 256 + b * 64, c << 6, z);
        } else {
          // A: 128 rows of the split matrix per M-tile (K-major); B: 256 rows n of one head's K or V (K-major)
          for (int m = 0; m < mt; ++m) tma_load_3d(a_dst + m * 16384, &tmS, bar, t * hd + (c << 6), rb * kRows + m * 128, z);
          const int col = c << 6, head = col / p.d, c0 = col % p.d;
          if (p.H > 0) tma_load_3d(b_dst, tmP, bar, (head % p.H) * p.d + c0, cg * 256, head / p.H);
          else tma_load_3d(b_dst, tmP, bar, c0, cg * 256, head);
        }
        ++issued;
      }
      if (!ok) {
        for (int it = max(0, issued - kK5Stages); it < issued; ++it)
          (void)mbar_wait(bar_full + 8 * (it % kK5Stages), (it / kK5Stages) & 1, p.status, &abort_flag);
      }
    }
  } else if (warp == 1) {
    if (elect_one()) {
      // ------------------------------------------------ MMA issuer
      const uint32_t idesc = kMode == 0 ? make_idesc(kFmtBF16, 1, 1, 128, (uint32_t)ncols) : make_idesc(kFmtBF16, 0, 0, 128, 256);
      bool ok = true;
      for (int it = 0; it < nchunks; ++it) {
        const int st = it % kK5Stages;
        ok = mbar_wait(bar_full + 8 * st, (it / kK5Stages) & 1, p.status, &abort_flag);
        if (!ok) break;
        tcgen05_fence_after();
        const uint32_t a_base = smem_base + st * kK5StageBytes;
        const uint32_t b_base = a_base + kABytes;
        for (int m = 0; m < mt; ++m) {
          if (kMode == 0) {
            // MN-major operands: 64-wide slabs 8192 B apart, 8-row (contraction) groups 1024 B apart, 16 rows per step
            const uint64_t ad = make_sdesc(a_base + m * 16384, 8192, 1024, kSwizzle128);
            const uint64_t bd = make_sdesc(b_base, 8192, 1024, kSwizzle128);
            mma_ss_x4(tmem + m * 256, ad, bd, 128, 128, idesc, it > 0 ? 1u : 0u);
          } else {
            // K-major operands: 128-byte rows, 8-row groups 1024 B apart, 32 B per step
            const uint64_t ad = make_sdesc(a_base + m * 16384, 16, 1024, kSwizzle128);
            const uint64_t bd = make_sdesc(b_base, 16, 1024, kSwizzle128);
            mma_ss_x4(tmem + m * 256, ad, bd, 2, 2, idesc, it > 0 ? 1u : 0u);
          }
        }
        mma_commit(bar_empty + 8 * st);
      }
      if (ok) mma_commit(bar_accum);
    }
  } else {
    // ------------------------------------------------ epilogue: bf16 slabs of [32 rows x 64 columns], one TMA store each
    const int q = warp & 3;
    bool ok = mbar_wait(bar_accum, 0, p.status, &abort_flag);
    if (ok) {
      tcgen05_fence_after();
      const uint32_t stage_buf = smem_base + (warp - 2) * 16384;   // the ring is drained; 4 slabs of 4 KB per warp
      for (int m = 0; m < mt; ++m) {
        const int row0 = rb * kRows + m * 128 + q * 32;
        const int ncc = ncols >> 6;
        for (int cc = 0; cc < ncc; ++cc) {
          uint32_t ra[32], rb2[32];
          tmem_ld32(tmem + ((uint32_t)(q * 32) << 16) + m * 256 + cc * 64, ra);
          tmem_ld32(tmem + ((uint32_t)(q * 32) << 16) + m * 256 + cc * 64 + 32, rb2);
          tmem_wait_ld(ra);
          tmem_wait_ld(rb2);
          const uint32_t row_addr = stage_buf + cc * 4096 + lane * 128;
#pragma unroll
          for (int g = 0; g < 8; ++g) {
            const uint32_t* src = g < 4 ? ra : rb2;
            uint32_t v[4];
#pragma unroll
            for (int e = 0; e < 4; ++e) {
              const __nv_bfloat162 o2 = __floats2bfloat162_rn(__uint_as_float(src[(g & 3) * 8 + 2 * e]),
                                                              __uint_as_float(src[(g & 3) * 8 + 2 * e + 1]));
              v[e] = *reinterpret_cast<const uint32_t*>(&o2);
            }
            asm volatile("st.shared.v4.b32 [%0], {%1, %2, %3, %4};" ::"r"(row_addr + ((g ^ (lane & 7)) << 4)),
                         "r"(v[0]), "r"(v[1]), "r"(v[2]), "r"(v[3]) : "memory");
          }
        }
        fence_proxy_async_smem();
        __syncwarp();
        if (lane == 0) {
          if (row0 < M) {
            for (int cc = 0; cc < ncc; ++cc) {
              const int col = cg * 256 + cc * 64;
              if (col >= NC) break;
              if (kMode == 0) {
                const int head = col / p.d, c0 = col % p.d;
                if (p.H > 0) tma_store_3d(tmO, stage_buf + cc * 4096, (head % p.H) * p.d + c0, row0, head / p.H);
                else tma_store_3d(tmO, stage_buf + cc * 4096, c0, row0, head);
              } else {
                tma_store_2d(tmO, stage_buf + cc * 4096, col, row0);
              }
            }
          }
          bulk_commit_group();
          bulk_wait_group_read0();
        }
        __syncwarp();
      }
      if (lane == 0) bulk_wait_group0();
    }
  }
  tcgen05_fence_before();
  __syncthreads();
  if (warp == 1) tmem_dealloc(tmem, K5Shape<kMode>::kTmemCols);
}

}  // namespace flurka

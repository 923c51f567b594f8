// The per-head linear maps of Eq. (2) (arxiv 2306.15799; Appendix B's step "Linear Transformations")
// on tensor cores, for the entry point that takes un-projected inputs:
//
//   mode 0   K'[b,h] = (E Xk[b]) W^K_h,  V'[b,h] = (F Xv[b]) W^V_h     k rows per batch: the low-rank
//            contraction has already happened, so the maps cost 2 k d_m^2 instead of 2 N d_m^2.  The
//            contracted rows arrive as three bf16 terms side by side along the contraction (hi | mid |
//            lo of the fp32 values, exact to 24 bits), the weight matrix is walked three times, and the
//            fp32 result is added into the K', V' workspace of the key side (partial sums of CTAs that
//            split the contraction meet in L2).
//   mode 1   Q[b] = Xq[b] W^Q                                          N rows per batch, bf16 out, stored
//            as [B,N,H,d] for the query side.
//
// Both are C = A B with A row-major along the contraction (K-major) and B = [d_m, H d] row-major
// (MN-major: the contracted index is the slow one), bf16 operands, fp32 accumulation in TMEM.  One
// CTA owns 256 rows x 256 columns (two 128-row MMA tiles) and a range of 64-wide contraction chunks;
// a three-stage TMA ring feeds one thread that issues tcgen05.mma (M=128, N=256, K=16); four warps
// move the accumulators out: mode 0 through swizzled fp32 slabs and TMA reduce-add, mode 1 through
// swizzled bf16 slabs and TMA stores of whole lines.
#pragma once

#include <cuda_bf16.h>

#include "tc_common.cuh"
#include "k1_down_project_pair.cuh"

namespace flurka {

struct K0Params {
  int mode;          // 0: fp32 reduce-add into [Z*H][M][d]; 1: bf16 store into [M][ncols]
  int M;             // rows of A per z
  int chunks;        // 64-wide contraction chunks of A (mode 0: 3 * d_m / 64)
  int b_chunks;      // 64-row chunks of B (d_m / 64): chunk c of A meets chunk c % b_chunks of B
  int ncols;         // H * d
  int d, H;          // mode 0: output column col belongs to head col / d
  int Z;             // batch count of A (mode 0: 2 * B, keys then values; mode 1: 1)
  int zb_shift;      // mode 0: which B matrix z uses = z / zb_shift (0 = W^K, 1 = W^V)
  int nsplit;        // CTAs along the contraction (mode 1: 1)
  int row_blocks;    // ceil(M / 256)
  int col_groups;    // ceil(ncols / 256)
  int* status;
};

constexpr int kK0Stages = 3;
constexpr int kK0StageBytes = 65536;                  // 32 KB of A rows + 32 KB of B slabs
constexpr int kK0SmemBytes = kK0Stages * kK0StageBytes + 1024 /*alignment*/ + 256 /*barriers*/;
constexpr int kK0Threads = 192;

__global__ void __launch_bounds__(kK0Threads, 1)
k0_linear_map(const __grid_constant__ CUtensorMap tmA, const __grid_constant__ CUtensorMap tmB0,
              const __grid_constant__ CUtensorMap tmB1, const __grid_constant__ CUtensorMap tmOut,
              const K0Params p) {
  using namespace tc;
  extern __shared__ uint8_t smem_raw[];
  const uint32_t smem_base = (smem_u32(smem_raw) + 1023u) & ~1023u;
  const uint32_t bar_base = smem_base + kK0Stages * kK0StageBytes;
  const uint32_t bar_full = bar_base;                 // [3]
  const uint32_t bar_empty = bar_base + 24;           // [3]
  const uint32_t bar_accum = bar_base + 48;
  const uint32_t tmem_slot = bar_base + 64;
  __shared__ int abort_flag;
  __shared__ uint32_t tmem_base_shared;

  const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;

  // ---- which piece of the problem
  int idx = blockIdx.x;
  const int cg = idx % p.col_groups; idx /= p.col_groups;
  const int rb = idx % p.row_blocks; idx /= p.row_blocks;
  const int z = idx % p.Z;           idx /= p.Z;
  const int s = idx;
  const int rows = min(256, p.M - rb * 256);
  const int mt = (rows + 127) >> 7;                         // MMA M-tiles (1 or 2)
  const int ncols = min(256, p.ncols - cg * 256);           // multiple of 64
  const int nb = ncols >> 6;                                // 64-column slabs
  const int c_begin = (int)(((long long)s * p.chunks) / p.nsplit);
  const int c_end = (int)(((long long)(s + 1) * p.chunks) / p.nsplit);
  const int nchunks = c_end - c_begin;
  const uint32_t tmem_cols = mt == 2 ? 512u : 256u;
  const CUtensorMap* tmB = (p.mode == 0 && z / p.zb_shift == 1) ? &tmB1 : &tmB0;

  if (threadIdx.x == 0) {
    abort_flag = 0;
    for (int i = 0; i < kK0Stages; ++i) {
      mbar_init(bar_full + 8 * i, 1);
      mbar_init(bar_empty + 8 * i, 1);
    }
    mbar_init(bar_accum, 1);
    fence_mbar_init();
  }
  if (warp == 1) {
    tmem_alloc(tmem_slot, tmem_cols);
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
  // A (mode 0) is the result of the kernel before this one in the stream
  grid_dependency_wait();

  if (nchunks > 0) {
    if (warp == 0) {
      if (elect_one()) {
        // ------------------------------------------------ TMA producer
        prefetch_tmap(&tmA);
        prefetch_tmap(tmB);
        const uint32_t tx_bytes = (uint32_t)(mt * 16384 + nb * 8192);
        int issued = 0;
        bool ok = true;
        for (int it = 0; it < nchunks && ok; ++it) {
          const int st = it % kK0Stages;
          if (it >= kK0Stages) ok = mbar_wait(bar_empty + 8 * st, ((it / kK0Stages) - 1) & 1, p.status, &abort_flag);
          if (!ok) break;
          const uint32_t a_dst = smem_base + st * kK0StageBytes;
          const uint32_t b_dst = a_dst + 32768;
          const int c = c_begin + it;
          mbar_arrive_expect_tx(bar_full + 8 * st, tx_bytes);
          for (int m = 0; m < mt; ++m) tma_load_3d(a_dst + m * 16384, &tmA, bar_full + 8 * st, c << 6, rb * 256 + m * 128, z);
          for (int b = 0; b < nb; ++b)
            tma_load_2d(b_dst + b * 8192, tmB, bar_full + 8 * st, cg * 256 + b * 64, (c % p.b_chunks) << 6);
          ++issued;
        }
        if (!ok) {
          // loads already in flight still land in this CTA's shared memory: wait for them (bounded)
          for (int it = max(0, issued - kK0Stages); it < issued; ++it)
            (void)mbar_wait(bar_full + 8 * (it % kK0Stages), (it / kK0Stages) & 1, p.status, &abort_flag);
        }
      }
    } else if (warp == 1) {
      if (elect_one()) {
        // ------------------------------------------------ MMA issuer
        const uint32_t idesc = make_idesc(kFmtBF16, /*A K-major*/ 0, /*B MN-major*/ 1, 128, (uint32_t)ncols);
        bool ok = true;
        for (int it = 0; it < nchunks; ++it) {
          const int st = it % kK0Stages;
          ok = mbar_wait(bar_full + 8 * st, (it / kK0Stages) & 1, p.status, &abort_flag);
          if (!ok) break;
          tcgen05_fence_after();
          const uint32_t a_base = smem_base + st * kK0StageBytes;
          const uint32_t b_base = a_base + 32768;
          // A: K-major, 128-byte rows, 8-row groups 1024 B apart; 16 contraction elements = 32 B per step.
          // B: MN-major, 64-column slabs 8192 B apart, 8-row (contraction) groups 1024 B apart;
          //    16 contraction elements = 16 rows = 2048 B per step.
          const uint64_t bd = make_sdesc(b_base, 8192, 1024, kSwizzle128);
          for (int m = 0; m < mt; ++m) {
            const uint64_t ad = make_sdesc(a_base + m * 16384, 16, 1024, kSwizzle128);
            mma_ss_x4(tmem + m * 256, ad, bd, 2, 128, idesc, it > 0 ? 1u : 0u);
          }
          mma_commit(bar_empty + 8 * st);
        }
        if (ok) mma_commit(bar_accum);
      }
    } else {
      // ------------------------------------------------ epilogue (warps 2..5): TMEM -> smem -> global
      const int q = warp & 3;                                // TMEM lane quadrant of this warp
      bool ok = mbar_wait(bar_accum, 0, p.status, &abort_flag);
      if (warp == 2 && lane == 0) grid_launch_dependents();   // only the epilogue is left
      if (ok) {
        tcgen05_fence_after();
        const uint32_t stage_buf = smem_base + (warp - 2) * 32768;   // the pipeline is drained
        for (int m = 0; m < mt; ++m) {
          const int row0 = rb * 256 + m * 128 + q * 32;
          if (p.mode == 0) {
            // fp32 slabs of [32 rows x 32 columns] (128-byte rows, swizzled), one reduce-add each
            const int ncc = ncols >> 5;
            for (int cc = 0; cc < ncc; ++cc) {
              uint32_t r[32];
              tmem_ld32(tmem + ((uint32_t)(q * 32) << 16) + m * 256 + cc * 32, r);
              tmem_wait_ld(r);
              const uint32_t row_addr = stage_buf + cc * 4096 + lane * 128;
#pragma unroll
              for (int c = 0; c < 8; ++c) {
                const uint32_t a = row_addr + ((c ^ (lane & 7)) << 4);
                asm volatile("st.shared.v4.b32 [%0], {%1, %2, %3, %4};" ::"r"(a), "r"(r[4 * c]), "r"(r[4 * c + 1]),
                             "r"(r[4 * c + 2]), "r"(r[4 * c + 3])
                             : "memory");
              }
            }
            fence_proxy_async_smem();
            __syncwarp();
            if (lane == 0) {
              if (row0 < p.M) {
                // z = t * B + b: the heads of this batch's keys (or values) start at z * H
                for (int cc = 0; cc < ncc; ++cc) {
                  const int col = cg * 256 + cc * 32;
                  tma_reduce_add_3d(&tmOut, stage_buf + cc * 4096, col % p.d, row0, z * p.H + col / p.d);
                }
              }
              bulk_commit_group();
              bulk_wait_group_read0();
            }
            __syncwarp();
          } else {
            // bf16 slabs of [32 rows x 64 columns] (128-byte rows, swizzled), one store each
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
              if (row0 < p.M)
                for (int cc = 0; cc < ncc; ++cc) tma_store_2d(&tmOut, stage_buf + cc * 4096, cg * 256 + cc * 64, row0);
              bulk_commit_group();
              bulk_wait_group_read0();
            }
            __syncwarp();
          }
        }
        if (lane == 0) bulk_wait_group0();
      }
    }
  }
  tcgen05_fence_before();
  __syncthreads();
  if (warp == 1) tmem_dealloc(tmem, tmem_cols);
}

// fp32 rows of the contracted keys and values -> three bf16 terms side by side along the contraction.
// `src` is stage 1's output for the un-projected inputs: [2][B][dm/64][k][64] fp32 (64-wide column
// blocks of the k x dm matrices E Xk[b], F Xv[b]); `dst` is [2*B][k][3*dm] bf16: hi | mid | lo.
__global__ void k0_split_rows(const float* __restrict__ src, __nv_bfloat16* __restrict__ dst, int ZB, int k, int dm) {
  tc::grid_dependency_wait();
  const long long total = (long long)ZB * k * (dm >> 2);
  for (long long i = (long long)blockIdx.x * blockDim.x + threadIdx.x; i < total; i += (long long)gridDim.x * blockDim.x) {
    const int c4 = (int)(i % (dm >> 2)) * 4;          // first of four consecutive columns
    const long long zr = i / (dm >> 2);
    const int row = (int)(zr % k);
    const int z = (int)(zr / k);
    const float4 x = *reinterpret_cast<const float4*>(src + (((size_t)z * (dm >> 6) + (c4 >> 6)) * k + row) * 64 + (c4 & 63));
    float v[4] = {x.x, x.y, x.z, x.w};
    __nv_bfloat16 t[3][4];
#pragma unroll
    for (int e = 0; e < 4; ++e) {
      float r = v[e];
#pragma unroll
      for (int s = 0; s < 3; ++s) {
        t[s][e] = __float2bfloat16_rn(r);
        r -= __bfloat162float(t[s][e]);
      }
    }
    __nv_bfloat16* base = dst + ((size_t)z * k + row) * (size_t)(3 * dm) + c4;
#pragma unroll
    for (int s = 0; s < 3; ++s) {
      uint2 w;
      w.x = (uint32_t)__bfloat16_as_ushort(t[s][0]) | ((uint32_t)__bfloat16_as_ushort(t[s][1]) << 16);
      w.y = (uint32_t)__bfloat16_as_ushort(t[s][2]) | ((uint32_t)__bfloat16_as_ushort(t[s][3]) << 16);
      *reinterpret_cast<uint2*>(base + (size_t)s * dm) = w;
    }
  }
  tc::grid_launch_dependents();
}

// ---------------------------------------------------------------------------------------------
// Mode 1 (Q = Xq W^Q, bf16 store) as pairs of CTAs, the way k1_down_project_pair runs stage 1: a
// cluster of two owns 256 rows x 512 columns, each CTA loads its 128 rows of A and its 128-column
// half of each 256-column slab of the weights (48 KB per chunk instead of 64), both CTAs' TMA bytes
// are counted on the even CTA's barrier, one thread of the even CTA issues tcgen05.mma.cta_group::2
// (M = 256 over the pair, N = 256, K = 16), and each CTA stores its own 128 x 512 accumulator.
// Needs ncols (= H d) a multiple of 256; the host uses the one-CTA kernel otherwise.
// ---------------------------------------------------------------------------------------------
constexpr int kK0PStages = 4;
constexpr int kK0PStageBytes = 49152;
constexpr int kK0PSmemBytes = kK0PStages * kK0PStageBytes + 1024 + 256;

namespace tc {
__device__ __forceinline__ void tma_load_2d_pair(uint32_t dst, const CUtensorMap* m, uint32_t bar_cluster_addr, int x,
                                                 int y) {
  asm volatile(
      "cp.async.bulk.tensor.2d.cta_group::2.shared::cluster.global.mbarrier::complete_tx::bytes [%0], [%1, {%3, %4}], [%2];"
      ::"r"(dst), "l"(reinterpret_cast<uint64_t>(m)), "r"(bar_cluster_addr), "r"(x), "r"(y)
      : "memory");
}
}  // namespace tc

__global__ void __cluster_dims__(2, 1, 1) __launch_bounds__(kK0Threads, 1)
k0_query_map_pair(const __grid_constant__ CUtensorMap tmA, const __grid_constant__ CUtensorMap tmB,
                  const __grid_constant__ CUtensorMap tmOut, const K0Params p) {
  using namespace tc;
  extern __shared__ uint8_t smem_raw[];
  const uint32_t smem_base = (smem_u32(smem_raw) + 1023u) & ~1023u;
  const uint32_t bar_base = smem_base + kK0PStages * kK0PStageBytes;
  const uint32_t bar_full = bar_base;                 // [4] even CTA's: the loads of both CTAs have landed
  const uint32_t bar_empty = bar_base + 32;           // [4] the pair's MMAs have read the stage
  const uint32_t bar_accum = bar_base + 96;
  const uint32_t tmem_slot = bar_base + 112;
  __shared__ int abort_flag;
  __shared__ uint32_t tmem_base_shared;

  const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
  const uint32_t rank = cluster_ctarank();
  // ---- which piece of the problem (col_groups here counts 512-column groups)
  int idx = blockIdx.x >> 1;
  const int cg = idx % p.col_groups; idx /= p.col_groups;
  const int rb = idx;
  const int ncols = min(512, p.ncols - cg * 512);           // 256 or 512
  const int nj = ncols >> 8;
  const int nchunks = p.chunks;

  if (threadIdx.x == 0) {
    abort_flag = 0;
    for (int i = 0; i < kK0PStages; ++i) {
      mbar_init(bar_full + 8 * i, 1);
      mbar_init(bar_empty + 8 * i, 1);
    }
    mbar_init(bar_accum, 1);
    fence_mbar_init();
  }
  if (warp == 1) {
    tmem_alloc_pair(tmem_slot, 512);
    tmem_relinquish_pair();
  }
  tcgen05_fence_before();
  __syncthreads();
  tcgen05_fence_after();
  if (threadIdx.x == 0) {
    uint32_t v;
    asm volatile("ld.shared.u32 %0, [%1];" : "=r"(v) : "r"(tmem_slot));
    tmem_base_shared = v;
  }
  cluster_sync_all();
  const uint32_t tmem = tmem_base_shared;
  grid_dependency_wait();

  if (warp == 0) {
    if (elect_one()) {
      // ------------------------------------------------ TMA producer (each CTA feeds its own shared memory)
      prefetch_tmap(&tmA);
      prefetch_tmap(&tmB);
      const uint32_t tx_bytes = (uint32_t)(16384 + nj * 16384);
      bool ok = true;
      int issued = 0;
      for (int it = 0; it < nchunks && ok; ++it) {
        const int st = it % kK0PStages;
        if (it >= kK0PStages) ok = mbar_wait(bar_empty + 8 * st, ((it / kK0PStages) - 1) & 1, p.status, &abort_flag);
        if (!ok) break;
        const uint32_t a_dst = smem_base + st * kK0PStageBytes;
        const uint32_t b_dst = a_dst + 16384;
        const uint32_t fb = map_to_cta(bar_full + 8 * st, 0);
        if (rank == 0) mbar_arrive_expect_tx(bar_full + 8 * st, 2 * tx_bytes);
        tma_load_3d_pair(map_to_cta(a_dst, rank), &tmA, fb, it << 6, rb * 256 + (int)rank * 128, 0);
        for (int j = 0; j < nj; ++j)
          for (int b = 0; b < 2; ++b)
            tma_load_2d_pair(map_to_cta(b_dst + (uint32_t)(j * 2 + b) * 8192u, rank), &tmB, fb,
                             cg * 512 + j * 256 + (int)rank * 128 + b * 64, (it % p.b_chunks) << 6);
        ++issued;
      }
      if (!ok && rank == 0) {
        for (int it = max(0, issued - kK0PStages); it < issued; ++it)
          (void)mbar_wait(bar_full + 8 * (it % kK0PStages), (it / kK0PStages) & 1, p.status, &abort_flag);
      }
    }
  } else if (warp == 1) {
    if (rank == 0 && elect_one()) {
      // ------------------------------------------------ even CTA: MMA issuer for the pair
      const uint32_t idesc = make_idesc(kFmtBF16, /*A K-major*/ 0, /*B MN-major*/ 1, 256, 256);
      bool ok = true;
      for (int it = 0; it < nchunks; ++it) {
        const int st = it % kK0PStages;
        ok = mbar_wait(bar_full + 8 * st, (it / kK0PStages) & 1, p.status, &abort_flag);
        if (!ok) break;
        tcgen05_fence_after();
        const uint32_t a_base = smem_base + st * kK0PStageBytes;
        const uint32_t b_base = a_base + 16384;
        const uint64_t ad = make_sdesc(a_base, 16, 1024, kSwizzle128);
        for (int j = 0; j < nj; ++j) {
          const uint64_t bd = make_sdesc(b_base + j * 16384, 8192, 1024, kSwizzle128);
          mma_ss_x4_pair(tmem + j * 256, ad, bd, 2, 128, idesc, it > 0 ? 1u : 0u);
        }
        mma_commit_pair(bar_empty + 8 * st);
      }
      if (ok) mma_commit_pair(bar_accum);
    }
  } else {
    // ------------------------------------------------ epilogue: this CTA's 128 rows, bf16 slabs of [32 x 64], TMA stores
    const int q = warp & 3;
    bool ok = mbar_wait(bar_accum, 0, p.status, &abort_flag);
    if (warp == 2 && lane == 0) grid_launch_dependents();
    if (ok) {
      tcgen05_fence_after();
      const uint32_t stage_buf = smem_base + (warp - 2) * 32768;
      const int row0 = rb * 256 + (int)rank * 128 + q * 32;
      const int ncc = ncols >> 6;
      for (int cc = 0; cc < ncc; ++cc) {
        uint32_t ra[32], rb2[32];
        tmem_ld32(tmem + ((uint32_t)(q * 32) << 16) + cc * 64, ra);
        tmem_ld32(tmem + ((uint32_t)(q * 32) << 16) + cc * 64 + 32, rb2);
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
        if (row0 < p.M)
          for (int cc = 0; cc < ncc; ++cc) tma_store_2d(&tmOut, stage_buf + cc * 4096, cg * 512 + cc * 64, row0);
        bulk_commit_group();
        bulk_wait_group0();
      }
      __syncwarp();
    }
  }
  tcgen05_fence_before();
  __syncthreads();
  cluster_sync_all();
  if (warp == 1) tmem_dealloc_pair(tmem, 512);
}

}  // namespace flurka

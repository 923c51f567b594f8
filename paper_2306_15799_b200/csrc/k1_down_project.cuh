// Stage 1 on tensor cores: K' = E K and V' = F V (arxiv 2306.15799, Section 2.1 / Eq. (2)),
// a contraction over the sequence axis, split across CTAs along that axis.
//
// One CTA owns: one of the two projections (t), up to 256 rows of the projection matrix (two
// 128-row MMA tiles), 256 output columns = 256/d consecutive heads (one head when every head has its
// own E_i, F_i, as Theorem 1 writes them), and a contiguous range of 64-wide sequence chunks.  Per chunk TMA brings a [rows x 64] slab of E (K-major, the sequence is
// contiguous) and, per 64 columns, a [64 x 64] slab of K or V (MN-major: the head dimension is
// contiguous, the contracted sequence index is the slow one), both 128-byte swizzled.  A single
// thread issues tcgen05.mma (M=128, N=ncols, K=16) into fp32 TMEM accumulators; when the range is
// done four warps move the accumulators to shared memory and add them to the fp32 workspace with
// TMA reduce-add, so partial sums from different CTAs meet in L2.
#pragma once

#include "tc_common.cuh"

namespace flurka {

struct K1Params {
  int N, d, k, BH;
  int H;           // > 0: K, V are [B,N,H,d] (the tensor map has rows of H*d elements); 0: [B,H,N,d]
  int ef_heads;    // > 0: E, F are [ef_heads][k][N], one pair per head (Theorem 1's E_i, F_i); a CTA then owns ONE head
  int group_cols;  // output columns per CTA: 256 (= 256/d heads sharing an E tile), or d with per-head E, F
  int nsplit;      // CTAs along the sequence
  int col_groups;  // ceil(BH * d / group_cols)
  int k_halves;    // ceil(k / 256)
  int* status;
};

constexpr int kK1Stages = 3;
constexpr int kK1StageBytes = 65536;                  // 32 KB of E rows + 32 KB of K/V slabs
constexpr int kK1SmemBytes = kK1Stages * kK1StageBytes + 1024 /*alignment*/ + 256 /*barriers*/;
constexpr int kK1Threads = 192;

__global__ void __launch_bounds__(kK1Threads, 1)
k1_down_project(const __grid_constant__ CUtensorMap tmE, const __grid_constant__ CUtensorMap tmF,
                const __grid_constant__ CUtensorMap tmK, const __grid_constant__ CUtensorMap tmV,
                const __grid_constant__ CUtensorMap tmOut, const K1Params p) {
  using namespace tc;
  extern __shared__ uint8_t smem_raw[];
  const uint32_t smem_base = (smem_u32(smem_raw) + 1023u) & ~1023u;
  const uint32_t bar_base = smem_base + kK1Stages * kK1StageBytes;
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
  const int kh = idx % p.k_halves;   idx /= p.k_halves;
  const int t = idx & 1;
  const int s = idx >> 1;
  const int rows = min(256, p.k - kh * 256);
  const int mt = (rows + 127) >> 7;                         // MMA M-tiles (1 or 2)
  const int total_cols = p.BH * p.d;
  const int ncols = min(p.group_cols, total_cols - cg * p.group_cols);   // multiple of 64
  const int nb = ncols >> 6;                                // 64-column slabs
  const int chunks_total = (p.N + 63) >> 6;                 // a ragged last chunk is zero-filled by TMA
  const int c_begin = (int)(((long long)s * chunks_total) / p.nsplit);
  const int c_end = (int)(((long long)(s + 1) * chunks_total) / p.nsplit);
  const int nchunks = c_end - c_begin;
  const uint32_t tmem_cols = mt == 2 ? 512u : 256u;

  if (threadIdx.x == 0) {
    abort_flag = 0;
    for (int i = 0; i < kK1Stages; ++i) {
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

  if (nchunks > 0) {
    if (warp == 0 && lane == 0) {
      // ------------------------------------------------ TMA producer
      const CUtensorMap* tmP = t ? &tmF : &tmE;
      const CUtensorMap* tmX = t ? &tmV : &tmK;
      prefetch_tmap(tmP);
      prefetch_tmap(tmX);
      const uint32_t tx_bytes = (uint32_t)(mt * 16384 + nb * 8192);
      const int dblocks = p.d >> 6;                         // 64-column slabs per head
      int issued = 0;
      bool ok = true;
      for (int it = 0; it < nchunks && ok; ++it) {
        const int st = it % kK1Stages;
        if (it >= kK1Stages) ok = mbar_wait(bar_empty + 8 * st, ((it / kK1Stages) - 1) & 1, p.status, &abort_flag);
        if (!ok) break;
        const uint32_t a_dst = smem_base + st * kK1StageBytes;
        const uint32_t b_dst = a_dst + 32768;
        const int n0 = (c_begin + it) << 6;
        mbar_arrive_expect_tx(bar_full + 8 * st, tx_bytes);
        // with per-head E, F this CTA's head is cg (its group is one head wide); E_i is shared over the batch
        const int ez = p.ef_heads > 0 ? cg % p.ef_heads : 0;
        for (int m = 0; m < mt; ++m) tma_load_3d(a_dst + m * 16384, tmP, bar_full + 8 * st, n0, kh * 256 + m * 128, ez);
        for (int b = 0; b < nb; ++b) {
          const int slab = cg * (p.group_cols >> 6) + b;     // global 64-column slab index
          const int head = slab / dblocks, dc = slab % dblocks;
          if (p.H > 0) tma_load_3d(b_dst + b * 8192, tmX, bar_full + 8 * st, (head % p.H) * p.d + dc * 64, n0, head / p.H);
          else tma_load_3d(b_dst + b * 8192, tmX, bar_full + 8 * st, dc * 64, n0, head);
        }
        ++issued;
      }
      if (!ok) {
        // loads already in flight still land in this CTA's shared memory: wait for them (bounded)
        for (int it = max(0, issued - kK1Stages); it < issued; ++it)
          (void)mbar_wait(bar_full + 8 * (it % kK1Stages), (it / kK1Stages) & 1, p.status, &abort_flag);
      }
    } else if (warp == 1 && lane == 0) {
      // ------------------------------------------------ MMA issuer
      const uint32_t idesc = make_idesc(kFmtBF16, /*A K-major*/ 0, /*B MN-major*/ 1, 128, (uint32_t)ncols);
      bool ok = true;
      for (int it = 0; it < nchunks; ++it) {
        const int st = it % kK1Stages;
        ok = mbar_wait(bar_full + 8 * st, (it / kK1Stages) & 1, p.status, &abort_flag);
        if (!ok) break;
        tcgen05_fence_after();
        const uint32_t a_base = smem_base + st * kK1StageBytes;
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
    } else if (warp >= 2) {
      // ------------------------------------------------ epilogue: TMEM -> smem -> TMA reduce-add
      const int q = warp & 3;                                // TMEM lane quadrant of this warp
      bool ok = mbar_wait(bar_accum, 0, p.status, &abort_flag);
      if (warp == 2 && lane == 0) grid_launch_dependents();   // only the epilogue is left
      if (ok) {
        tcgen05_fence_after();
        const uint32_t stage_buf = smem_base + (warp - 2) * 32768;   // 8 x 4 KB, pipeline is drained
        for (int m = 0; m < mt; ++m) {
          const int row0 = kh * 256 + m * 128 + q * 32;
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
            if (row0 < p.k) {
              for (int cc = 0; cc < ncc; ++cc) {
                const int col = cg * p.group_cols + cc * 32;
                const int head = col / p.d, c0 = col % p.d;
                tma_reduce_add_3d(&tmOut, stage_buf + cc * 4096, c0, row0, t * p.BH + head);
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
  }
  tcgen05_fence_before();
  __syncthreads();
  if (warp == 1) tmem_dealloc(tmem, tmem_cols);
}

}  // namespace flurka

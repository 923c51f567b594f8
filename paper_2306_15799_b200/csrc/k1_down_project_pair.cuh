// Stage 1 on tensor cores, two CTAs per output tile (tcgen05.mma.cta_group::2): K' = E K and
// V' = F V (arxiv 2306.15799, Section 2.1 / Eq. (2)), a contraction over the sequence axis split
// across CTA pairs along that axis.
//
// The one-CTA kernel (k1_down_project.cuh) takes 64 KB from L2 per 64-wide chunk for 1024 cycles of
// MMA, and all SMs together then ask L2 for about 10 TB/s, which is what bounds it.  Here a pair of
// CTAs (a cluster of two) owns 256 rows of the projection matrix and 512 output columns: each CTA
// loads ITS 128 rows of the E slab and ITS half of every 256-column K/V slab (48 KB per chunk for the
// same 1024 cycles of MMA per CTA), the tensor cores of the pair read both halves of B, and each CTA
// accumulates its 128 rows x 512 columns in its own TMEM.  The TMA loads of both CTAs count their
// bytes on the even CTA's barrier (the data itself goes to the loading CTA only, every load has one
// destination); one thread of the even CTA issues the MMAs for both, and its commits arrive on the
// barriers of both CTAs.  Measured against the one-CTA kernel: c4 205 -> 180 us, k = 512 of the
// sweep 114 -> 97 us, c3 75 -> 71.5 us, c2 41 -> 39.7 us.  The epilogue is the one-CTA
// kernel's: TMEM -> registers -> swizzled shared memory -> TMA reduce-add into the fp32 workspace.
//
// Needs k a multiple of 256 and B*H*d a multiple of 256 (the host falls back to the one-CTA kernel
// otherwise, and when every head has its own E_i, F_i).
#pragma once

#include "tc_common.cuh"

namespace flurka {

struct K1PairParams {
  int N, d, k, BH;
  int H;           // > 0: K, V are [B,N,H,d]; 0: [B,H,N,d]
  int nsplit;      // CTA pairs along the sequence
  int col_groups;  // ceil(BH * d / 512)
  int k_halves;    // k / 256
  int* status;
};

constexpr int kK1PStages = 4;
constexpr int kK1PStageBytes = 49152;                 // 16 KB of E rows + 32 KB of K/V half-slabs
constexpr int kK1PSmemBytes = kK1PStages * kK1PStageBytes + 1024 /*alignment*/ + 256 /*barriers*/;
constexpr int kK1PThreads = 192;

namespace tc {
__device__ __forceinline__ uint32_t cluster_ctarank() {
  uint32_t r;
  asm volatile("mov.u32 %0, %%cluster_ctarank;" : "=r"(r));
  return r;
}
// all threads of both CTAs
__device__ __forceinline__ void cluster_sync_all() {
  asm volatile("barrier.cluster.arrive.release.aligned;" ::: "memory");
  asm volatile("barrier.cluster.wait.acquire.aligned;" ::: "memory");
}
__device__ __forceinline__ void tmem_alloc_pair(uint32_t smem_result, uint32_t cols) {
  asm volatile("tcgen05.alloc.cta_group::2.sync.aligned.shared::cta.b32 [%0], %1;" ::"r"(smem_result), "r"(cols)
               : "memory");
}
__device__ __forceinline__ void tmem_relinquish_pair() {
  asm volatile("tcgen05.relinquish_alloc_permit.cta_group::2.sync.aligned;" ::: "memory");
}
__device__ __forceinline__ void tmem_dealloc_pair(uint32_t taddr, uint32_t cols) {
  asm volatile("tcgen05.dealloc.cta_group::2.sync.aligned.b32 %0, %1;" ::"r"(taddr), "r"(cols) : "memory");
}
// four 16-wide contraction steps of a two-CTA MMA (M = 256 over the pair, A and D split by rows, B by columns)
__device__ __forceinline__ void mma_ss_x4_pair(uint32_t d_tmem, uint64_t a_desc, uint64_t b_desc, uint32_t a_step,
                                               uint32_t b_step, uint32_t idesc, uint32_t accumulate) {
  asm volatile(
      "{\n\t.reg .pred p, q;\n\t.reg .b64 a1, a2, a3, b1, b2, b3, sa, sb;\n\t"
      "setp.ne.b32 p, %6, 0;\n\t"
      "setp.eq.b32 q, 0, 0;\n\t"
      "cvt.u64.u32 sa, %3;\n\t"
      "cvt.u64.u32 sb, %4;\n\t"
      "add.u64 a1, %1, sa;\n\t add.u64 a2, a1, sa;\n\t add.u64 a3, a2, sa;\n\t"
      "add.u64 b1, %2, sb;\n\t add.u64 b2, b1, sb;\n\t add.u64 b3, b2, sb;\n\t"
      "tcgen05.mma.cta_group::2.kind::f16 [%0], %1, %2, %5, p;\n\t"
      "tcgen05.mma.cta_group::2.kind::f16 [%0], a1, b1, %5, q;\n\t"
      "tcgen05.mma.cta_group::2.kind::f16 [%0], a2, b2, %5, q;\n\t"
      "tcgen05.mma.cta_group::2.kind::f16 [%0], a3, b3, %5, q;\n\t}"
      ::"r"(d_tmem), "l"(a_desc), "l"(b_desc), "r"(a_step), "r"(b_step), "r"(idesc), "r"(accumulate)
      : "memory");
}
// arrives on the barrier at this shared-memory offset in BOTH CTAs of the pair once every MMA issued so
// far by this thread has completed
__device__ __forceinline__ void mma_commit_pair(uint32_t bar) {
  asm volatile(
      "tcgen05.commit.cta_group::2.mbarrier::arrive::one.shared::cluster.multicast::cluster.b64 [%0], %1;"
      ::"r"(bar), "h"((unsigned short)3)
      : "memory");
}
// TMA load into THIS CTA's shared memory whose bytes are counted on a barrier given as a shared::cluster
// address (it may belong to the other CTA of the pair); the data has one destination, this CTA
__device__ __forceinline__ void tma_load_3d_pair(uint32_t dst, const CUtensorMap* m, uint32_t bar_cluster_addr, int x,
                                                 int y, int z) {
  asm volatile(
      "cp.async.bulk.tensor.3d.cta_group::2.shared::cluster.global.mbarrier::complete_tx::bytes [%0], [%1, {%3, %4, %5}], [%2];"
      ::"r"(dst), "l"(reinterpret_cast<uint64_t>(m)), "r"(bar_cluster_addr), "r"(x), "r"(y), "r"(z)
      : "memory");
}
__device__ __forceinline__ uint32_t map_to_cta(uint32_t addr, uint32_t rank) {
  uint32_t r;
  asm volatile("mapa.shared::cluster.u32 %0, %1, %2;" : "=r"(r) : "r"(addr), "r"(rank));
  return r;
}
}  // namespace tc

__global__ void __cluster_dims__(2, 1, 1) __launch_bounds__(kK1PThreads, 1)
k1_down_project_pair(const __grid_constant__ CUtensorMap tmE, const __grid_constant__ CUtensorMap tmF,
                     const __grid_constant__ CUtensorMap tmK, const __grid_constant__ CUtensorMap tmV,
                     const __grid_constant__ CUtensorMap tmOut, const K1PairParams p) {
  using namespace tc;
  extern __shared__ uint8_t smem_raw[];
  const uint32_t smem_base = (smem_u32(smem_raw) + 1023u) & ~1023u;
  const uint32_t bar_base = smem_base + kK1PStages * kK1PStageBytes;
  const uint32_t bar_full = bar_base;                 // [4] even CTA's: the loads of BOTH CTAs of a stage have landed
  const uint32_t bar_empty = bar_base + 32;           // [4] the pair's MMAs have read the stage (both CTAs get the arrival)
  const uint32_t bar_accum = bar_base + 96;
  const uint32_t tmem_slot = bar_base + 112;
  __shared__ int abort_flag;
  __shared__ uint32_t tmem_base_shared;

  const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
  const uint32_t rank = cluster_ctarank();            // 0: issues the MMAs; 1: its peer

  // ---- which piece of the problem (the same for both CTAs of a pair)
  int idx = blockIdx.x >> 1;
  const int cg = idx % p.col_groups; idx /= p.col_groups;
  const int kh = idx % p.k_halves;   idx /= p.k_halves;
  const int t = idx & 1;
  const int s = idx >> 1;
  const int total_cols = p.BH * p.d;
  const int ncols = min(512, total_cols - cg * 512);        // 256 or 512
  const int nj = ncols >> 8;                                // 256-column MMAs per contraction step
  const int chunks_total = (p.N + 63) >> 6;                 // a ragged last chunk is zero-filled by TMA
  const int c_begin = (int)(((long long)s * chunks_total) / p.nsplit);
  const int c_end = (int)(((long long)(s + 1) * chunks_total) / p.nsplit);
  const int nchunks = c_end - c_begin;

  if (threadIdx.x == 0) {
    abort_flag = 0;
    for (int i = 0; i < kK1PStages; ++i) {
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
  // both CTAs have initialised their barriers and hold their TMEM before anything crosses between them
  cluster_sync_all();
  const uint32_t tmem = tmem_base_shared;

  if (nchunks > 0) {
    if (warp == 0) {
      if (elect_one()) {
        // ------------------------------------------------ TMA producer (each CTA feeds its own shared memory)
        const CUtensorMap* tmP = t ? &tmF : &tmE;
        const CUtensorMap* tmX = t ? &tmV : &tmK;
        prefetch_tmap(tmP);
        prefetch_tmap(tmX);
        const uint32_t tx_bytes = (uint32_t)(16384 + nj * 16384);
        const int dblocks = p.d >> 6;                         // 64-column slabs per head
        int issued = 0;
        bool ok = true;
        for (int it = 0; it < nchunks && ok; ++it) {
          const int st = it % kK1PStages;
          if (it >= kK1PStages) ok = mbar_wait(bar_empty + 8 * st, ((it / kK1PStages) - 1) & 1, p.status, &abort_flag);
          if (!ok) break;
          const uint32_t a_dst = smem_base + st * kK1PStageBytes;
          const uint32_t b_dst = a_dst + 16384;
          const int n0 = (c_begin + it) << 6;
          // the bytes of BOTH CTAs are counted on the even CTA's barrier, which alone posts the expectation
          const uint32_t fb = map_to_cta(bar_full + 8 * st, 0);
          const uint32_t dst_a = map_to_cta(a_dst, rank);
          if (rank == 0) mbar_arrive_expect_tx(bar_full + 8 * st, 2 * tx_bytes);
          // this CTA's 128 rows of the E slab
          tma_load_3d_pair(dst_a, tmP, fb, n0, kh * 256 + (int)rank * 128, 0);
          // this CTA's 128-column half of each 256-column slab of K / V: two 64-column pieces
          for (int j = 0; j < nj; ++j) {
            for (int b = 0; b < 2; ++b) {
              const int slab = cg * 8 + j * 4 + (int)rank * 2 + b;   // global 64-column slab index
              const int head = slab / dblocks, dc = slab % dblocks;
              const uint32_t dst = map_to_cta(b_dst + (uint32_t)(j * 2 + b) * 8192u, rank);
              if (p.H > 0) tma_load_3d_pair(dst, tmX, fb, (head % p.H) * p.d + dc * 64, n0, head / p.H);
              else tma_load_3d_pair(dst, tmX, fb, dc * 64, n0, head);
            }
          }
          ++issued;
        }
        if (!ok && rank == 0) {
          for (int it = max(0, issued - kK1PStages); it < issued; ++it)
            (void)mbar_wait(bar_full + 8 * (it % kK1PStages), (it / kK1PStages) & 1, p.status, &abort_flag);
        }
      }
    } else if (warp == 1) {
      if (elect_one()) {
        if (rank == 0) {
          // ------------------------------------------------ even CTA: MMA issuer for the pair
          const uint32_t idesc = make_idesc(kFmtBF16, /*A K-major*/ 0, /*B MN-major*/ 1, 256, 256);
          bool ok = true;
          for (int it = 0; it < nchunks; ++it) {
            const int st = it % kK1PStages;
            ok = mbar_wait(bar_full + 8 * st, (it / kK1PStages) & 1, p.status, &abort_flag);
            if (!ok) break;
            tcgen05_fence_after();
            const uint32_t a_base = smem_base + st * kK1PStageBytes;
            const uint32_t b_base = a_base + 16384;
            // A: K-major, 128-byte rows, 8-row groups 1024 B apart; 16 contraction elements = 32 B per step.
            // B: MN-major, this CTA's two 64-column pieces of a slab 8192 B apart, 8-row (contraction)
            //    groups 1024 B apart; 16 contraction elements = 16 rows = 2048 B per step.
            const uint64_t ad = make_sdesc(a_base, 16, 1024, kSwizzle128);
            for (int j = 0; j < nj; ++j) {
              const uint64_t bd = make_sdesc(b_base + j * 16384, 8192, 1024, kSwizzle128);
              mma_ss_x4_pair(tmem + j * 256, ad, bd, 2, 128, idesc, it > 0 ? 1u : 0u);
            }
            mma_commit_pair(bar_empty + 8 * st);
          }
          if (ok) mma_commit_pair(bar_accum);
        }
      }
    } else {
      // ------------------------------------------------ epilogue: TMEM -> smem -> TMA reduce-add (this CTA's 128 rows)
      const int q = warp & 3;                                // TMEM lane quadrant of this warp
      bool ok = mbar_wait(bar_accum, 0, p.status, &abort_flag);
      if (warp == 2 && lane == 0) grid_launch_dependents();   // only the epilogue is left
      if (ok) {
        tcgen05_fence_after();
        const uint32_t stage_buf = smem_base + (warp - 2) * 32768;   // 8 x 4 KB per warp, the pipeline is drained
        const int row0 = kh * 256 + (int)rank * 128 + q * 32;
        for (int j = 0; j < nj; ++j) {
          for (int cc = 0; cc < 8; ++cc) {
            uint32_t r[32];
            tmem_ld32(tmem + ((uint32_t)(q * 32) << 16) + j * 256 + cc * 32, r);
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
            for (int cc = 0; cc < 8; ++cc) {
              const int col = cg * 512 + j * 256 + cc * 32;
              const int head = col / p.d, c0 = col % p.d;
              tma_reduce_add_3d(&tmOut, stage_buf + cc * 4096, c0, row0, t * p.BH + head);
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
  // neither CTA gives its TMEM back while the other may still be part of an MMA or of its commits
  tcgen05_fence_before();
  __syncthreads();
  cluster_sync_all();
  if (warp == 1) tmem_dealloc_pair(tmem, 512);
}

}  // namespace flurka

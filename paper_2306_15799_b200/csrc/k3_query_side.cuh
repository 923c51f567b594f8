// Stage 3 on tensor cores: the query feature map, the associative product and the row division
// (arxiv 2306.15799, Eq. (2); normalisation as in Appendix D), one pass over Q.
//
//   PERFORMER   S = Q W^T + 1 b^T      (tcgen05, bf16 x bf16 -> fp32 in TMEM; b_i rides along as
//                                        three bf16 terms in one extra 16-wide contraction step)
//               p = exp(S - rowmax S)   (two passes over TMEM by the thread that owns the row)
//               O = (p a) / sum_i p_i   (p as fp16 back into TMEM, tcgen05 with A from TMEM,
//                                        a^T resident in shared memory)
//   RNN         p = (elu(q) + 1) z / max z  straight from the Q tile, then the same second product.
//
// The per-feature summaries a_i, b_i (or z_i) come from stage 2.  A persistent CTA walks a
// contiguous range of 128-row tiles; warp 0 feeds Q tiles by TMA, warps 1 and 3 issue the first and the second
// products, warp 2 reloads a^T and rebuilds the bias operand when the head changes, and two groups of four warps
// alternate tiles.  TMEM holds S/p and O of the tiles in flight: two 256-column buffers in general, four
// 128-column buffers when d = 64 and p <= 128.  p overwrites S at half the width, block by block of 64
// features, and the row owners hand every finished block to the second product.  With d = 64, O sits in
// columns 64..127 of its buffer, which pass 2 has consumed after the first 128 features (blocks 2 and 3 of
// p go to columns 128.. instead), so at m = 256 the second product of a tile runs under the second half
// of its pass 2 and only its last block is left when the row owners start waiting for O.  With four
// buffers each group has two tiles in flight and reads tile i-2 out after it has handed tile i to the
// second product.  Every thread of a group owns one output row and writes it with 32-byte stores.
#pragma once

#include <cuda_bf16.h>
#include <cuda_fp16.h>

#include "tc_common.cuh"

namespace flurka {

struct K3Params {
  int N, d, p, BH;          // p = feature dimension (m, or d for RNN)
  int H;                    // > 0: Q and out are [B,N,H,d] (the Q tensor map has rows of H*d elements); 0: [B,H,N,d]
  int tiles_per_head;       // ceil(N / 128): TMA zero-fills the rows of a ragged last tile, their outputs are not stored
  int total_tiles;
  const float* weight;      // [BH][p]  b_i or z_i
  __nv_bfloat16* out;       // [BH][N][d]
  int* status;
};

constexpr int kK3Threads = 384;
constexpr int kK3MaxQStages = 4;

__device__ __forceinline__ float ex2_approx(float x) {
  float y;
  asm("ex2.approx.ftz.f32 %0, %1;" : "=f"(y) : "f"(x));
  return y;
}

// shared-memory plan (byte offsets from a 1024-aligned base)
struct K3Smem {
  uint32_t w, ones, bias, aT, q, ostage, scale, bars, total;
  int q_stages;
};

__host__ __device__ inline K3Smem k3_smem_plan(int d, int p, bool performer) {
  K3Smem s;
  uint32_t off = 0;
  s.w = off;    off += performer ? (uint32_t)p * d * 2 : 0;        // W: d/64 K-blocks of [p rows x 128 B]
  s.ones = off; off += performer ? 4096 : 0;                       // [128 x 16] bf16, no swizzle
  s.bias = off; off += performer ? 8192 : 0;                       // [256 x 16] bf16, no swizzle
  off = (off + 1023u) & ~1023u;
  s.aT = off;   off += (uint32_t)d * p * 2;                        // a^T: p/64 K-blocks of [d rows x 128 B]
  off = (off + 1023u) & ~1023u;
  s.q_stages = (d == 64) ? 4 : 2;
  s.q = off;    off += (uint32_t)s.q_stages * 128 * d * 2;
  s.ostage = off; off += (d == 64) ? 8 * 4096 : 0;                 // d = 64: a [32 x 64] bf16 output slab per row-owner warp
  s.scale = off; off += 1024;                                      // RNN: z_i / max z as floats
  s.bars = off; off += 512;
  s.total = off + 1024;                                            // alignment slack
  return s;
}

template <bool kPerformer>
__global__ void __launch_bounds__(kK3Threads, 1)
k3_query_side(const __grid_constant__ CUtensorMap tmQ, const __grid_constant__ CUtensorMap tmW,
              const __grid_constant__ CUtensorMap tmAT, const __grid_constant__ CUtensorMap tmO,
              const K3Params prm) {
  using namespace tc;
  extern __shared__ uint8_t smem_raw[];
  const uint32_t base = (smem_u32(smem_raw) + 1023u) & ~1023u;
  uint8_t* base_ptr = smem_raw + (base - smem_u32(smem_raw));
  const int d = prm.d, p = prm.p;
  const K3Smem L = k3_smem_plan(d, p, kPerformer);
  const int NS = L.q_stages;
  const uint32_t q_stage_bytes = 128u * d * 2u;

  // barriers
  const uint32_t bars = base + L.bars;
  const uint32_t bar_qfull = bars;            // [4]   Q tile landed
  const uint32_t bar_qempty = bars + 32;      // [4]   Q tile consumed (MMA commit, or 128 readers for RNN)
  const uint32_t bar_sfull = bars + 64;       // [4]   S ready in TMEM (PERFORMER)
  const uint32_t bar_ofull = bars + 96;       // [4]   O ready in TMEM
  const uint32_t bar_sfree = bars + 128;      // [4]   TMEM buffer read out, may be overwritten
  const uint32_t bar_pfull = bars + 160;      // [4][4] a block of 64 features of p written to TMEM by the 128 row owners
  const uint32_t bar_wfull = bars + 288;      //       W resident
  const uint32_t bar_drained = bars + 296;    //       every MMA of the previous head is complete
  const uint32_t bar_atfull = bars + 304;     //       a^T of the new head resident
  const uint32_t bar_biasready = bars + 312;  //       bias operand / scale vector of the new head built
  const uint32_t tmem_slot = bars + 320;
  __shared__ int abort_flag;
  __shared__ uint32_t tmem_base_shared;
  // RNN: how many heads' scale vectors have been built so far.  A count, not an mbarrier: a row-owner group
  // whose first tile already belongs to the CTA's second head has never waited for the first head's phase, and a
  // parity wait cannot tell "phase 1 complete" from "nothing complete yet".
  __shared__ volatile int scale_epoch;

  const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;

  // contiguous range of tiles for this CTA
  const int t_begin = (int)(((long long)blockIdx.x * prm.total_tiles) / gridDim.x);
  const int t_end = (int)(((long long)(blockIdx.x + 1) * prm.total_tiles) / gridDim.x);
  const int ntiles = t_end - t_begin;

  if (threadIdx.x == 0) {
    abort_flag = 0;
    scale_epoch = 0;
    for (int i = 0; i < kK3MaxQStages; ++i) {
      mbar_init(bar_qfull + 8 * i, 1);
      mbar_init(bar_qempty + 8 * i, kPerformer ? 1 : 128);
    }
    for (int i = 0; i < 4; ++i) {
      mbar_init(bar_sfull + 8 * i, 1);
      for (int q = 0; q < 4; ++q) mbar_init(bar_pfull + 8 * (4 * i + q), 128);
      mbar_init(bar_ofull + 8 * i, 1);
      mbar_init(bar_sfree + 8 * i, 128);
    }
    mbar_init(bar_wfull, 1);
    mbar_init(bar_drained, 1);
    mbar_init(bar_atfull, 1);
    mbar_init(bar_biasready, 32);
    fence_mbar_init();
  }
  if (warp == 1) {
    tmem_alloc(tmem_slot, 512);
    tmem_relinquish();
  }
  if (kPerformer && warp == 2) {
    // the all-ones A operand of the bias step: row r, column c (c < 16), no swizzle:
    // offset = (r/8)*256 + (c/8)*128 + (r%8)*16 + (c%8)*2; columns 0..2 are 1, the rest 0
    __nv_bfloat16* ones = reinterpret_cast<__nv_bfloat16*>(base_ptr + L.ones);
    for (int e = lane; e < 128 * 16; e += 32) {
      const int r = e >> 4, c = e & 15;
      const int off = (r >> 3) * 128 + (c >> 3) * 64 + (r & 7) * 8 + (c & 7);
      ones[off] = __float2bfloat16_rn(c < 3 ? 1.f : 0.f);
    }
    fence_proxy_async_smem();
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

  const int kq = d >> 6;      // 64-wide K-blocks of the Q / W tiles
  const int kp = p >> 6;      // 64-wide K-blocks of a^T
  // TMEM buffers: tile i uses buffer i % NB, its barriers flip once per NB tiles
  const int NB = (d == 64 && p <= 128) ? 4 : 2;
  const int nb_shift = NB == 4 ? 2 : 1;
  const uint32_t buf_cols = 512u / NB;
  const uint32_t o_col = d == 64 ? 64u : 128u;
  // O occupies columns [o_col, o_col + d) of the buffer.  Where that range overlaps S (PERFORMER), the
  // second product may start only when pass 2 has consumed those columns: q_first is the first block
  // of 64 features whose completion its issuer waits for (the blocks before it need no signal).
  int q_first = 0;
  if (kPerformer && (int)o_col < p) q_first = (min(p, (int)o_col + d) - 1) >> 6;
  // p's block kb of 64 features (32 columns of fp16 pairs) sits at column pcol(kb): side by side from
  // column 0, except that with d = 64 blocks 2 and 3 skip over O to columns 128 and 160
  auto pcol = [&](int kb) -> uint32_t { return (uint32_t)(32 * kb + ((d == 64 && kb >= 2) ? 64 : 0)); };

  if (ntiles > 0 && warp == 0 && lane == 0) {
    // W is an input, not a result of stage 2: its load starts before the dependency wait
    prefetch_tmap(&tmQ);
    prefetch_tmap(&tmAT);
    if (kPerformer) {
      prefetch_tmap(&tmW);
      mbar_arrive_expect_tx(bar_wfull, (uint32_t)p * d * 2);
      for (int kb = 0; kb < kq; ++kb) tma_load_2d(base + L.w + kb * (p * 128), &tmW, bar_wfull, kb * 64, 0);
    }
  }
  grid_dependency_wait();

  if (ntiles > 0) {
    if (warp == 0 && elect_one()) {
      // ============================================================ TMA producer
      // Q tiles only: they do not depend on the head's operands, so the ring keeps running ahead
      // across a change of head (a^T is reloaded by the operand builder, which waits for the drain)
      bool ok = true;
      int issued = 0;
      for (int i = 0; i < ntiles && ok; ++i) {
        const int tile = t_begin + i;
        const int head = tile / prm.tiles_per_head;
        const int row0 = (tile % prm.tiles_per_head) * 128;
        const int st = i % NS;
        if (i >= NS) ok = mbar_wait(bar_qempty + 8 * st, ((i / NS) - 1) & 1, prm.status, &abort_flag);
        if (!ok) break;
        mbar_arrive_expect_tx(bar_qfull + 8 * st, q_stage_bytes);
        for (int kb = 0; kb < kq; ++kb)
          if (prm.H > 0)
            tma_load_3d(base + L.q + st * q_stage_bytes + kb * 16384, &tmQ, bar_qfull + 8 * st,
                        (head % prm.H) * d + kb * 64, row0, head / prm.H);
          else
            tma_load_3d(base + L.q + st * q_stage_bytes + kb * 16384, &tmQ, bar_qfull + 8 * st, kb * 64, row0, head);
        ++issued;
      }
      if (!ok) {
        for (int i = max(0, issued - NS); i < issued; ++i)
          (void)mbar_wait(bar_qfull + 8 * (i % NS), (i / NS) & 1, prm.status, &abort_flag);
      }
    } else if (warp == 1 && elect_one()) {
      // ============================================================ issuer of the first products
      // S_i = Q_i W^T + 1 b^T (PERFORMER only).  A new head's bias operand is ready once
      // bar_biasready flips, which also means every MMA of the old head has completed.
      if (kPerformer) {
        const uint32_t idesc1 = make_idesc(kFmtBF16, 0, 0, 128, (uint32_t)p);
        bool ok = mbar_wait(bar_wfull, 0, prm.status, &abort_flag);
        int head_prev = -1, events = 0;
        for (int i = 0; i < ntiles && ok; ++i) {
          const int head = (t_begin + i) / prm.tiles_per_head;
          const int buf = i & (NB - 1), st = i % NS;
          if (head != head_prev) {
            ok = mbar_wait(bar_biasready, events & 1, prm.status, &abort_flag);
            if (!ok) break;
            head_prev = head;
            ++events;
          }
          // TMEM half `buf` must have been read out by the row owners of tile i-2
          if (i >= NB) ok = mbar_wait(bar_sfree + 8 * buf, ((i >> nb_shift) - 1) & 1, prm.status, &abort_flag);
          if (ok) ok = mbar_wait(bar_qfull + 8 * st, (i / NS) & 1, prm.status, &abort_flag);
          if (!ok) break;
          tcgen05_fence_after();
          const uint32_t tb = tmem + buf * buf_cols;
          const uint32_t qb = base + L.q + st * q_stage_bytes;
          for (int kb = 0; kb < kq; ++kb) {
            const uint64_t ad = make_sdesc(qb + kb * 16384, 16, 1024, kSwizzle128);
            const uint64_t bd = make_sdesc(base + L.w + kb * (p * 128), 16, 1024, kSwizzle128);
            mma_ss_x4(tb, ad, bd, 2, 2, idesc1, kb > 0 ? 1u : 0u);
          }
          {
            // bias step: ones[128 x 16] (columns 0..2 = 1) times bias[p x 16] (b split in three bf16)
            const uint64_t ad = make_sdesc(base + L.ones, 128, 256, kSwizzleNone);
            const uint64_t bd = make_sdesc(base + L.bias, 128, 256, kSwizzleNone);
            mma_ss(tb, ad, bd, idesc1, 1u);
          }
          mma_commit(bar_sfull + 8 * buf);
          mma_commit(bar_qempty + 8 * st);         // the Q tile is free once these MMAs have read it
        }
      }
    } else if (warp == 3 && lane == 0) {
      // (lane 0 rather than an elected lane: with the slower issue code the compiler makes for a lane it
      // cannot prove to be alone, the second products of one tile interleave better with the first
      // products of the next: measured 5 % faster at m = 128 and 3 % at d = 128)
      // ============================================================ issuer of the second products
      // O_j = p_j a once the 128 row owners of tile j have written p_j.  Before the first tile of a
      // new head it waits for that head's a^T; after the last tile of a head it commits to
      // bar_drained, which therefore flips when every MMA that used the old operands is complete
      // (a tile's second product completes after its first product).
      const uint32_t idesc2 = make_idesc(kFmtF16, 0, 0, 128, (uint32_t)d);
      bool ok = true;
      int head_prev = -1, events = 0;
      for (int j = 0; j < ntiles && ok; ++j) {
        const int head = (t_begin + j) / prm.tiles_per_head;
        const int buf = j & (NB - 1);
        if (head != head_prev) {
          ok = mbar_wait(bar_atfull, events & 1, prm.status, &abort_flag);
          if (!ok) break;
          head_prev = head;
          ++events;
        }
        const uint32_t tb = tmem + buf * buf_cols;
        // block by block of 64 features as the row owners hand them over (the blocks before q_first
        // go together with block q_first); four 16-wide steps per call
        for (int kb = q_first; kb < kp && ok; ++kb) {
          ok = mbar_wait(bar_pfull + 8 * (4 * buf + kb), (j >> nb_shift) & 1, prm.status, &abort_flag);
          if (!ok) break;
          tcgen05_fence_after();
          for (int kk = (kb == q_first ? 0 : kb); kk <= kb; ++kk) {
            const uint64_t bd = make_sdesc(base + L.aT + kk * (d * 128), 16, 1024, kSwizzle128);
            mma_ts_x4(tb + o_col, tb + pcol(kk), bd, 2, idesc2, kk > 0 ? 1u : 0u);
          }
        }
        if (!ok) break;
        mma_commit(bar_ofull + 8 * buf);
        const bool last_of_head = (j + 1 < ntiles) && ((t_begin + j + 1) / prm.tiles_per_head != head);
        if (last_of_head) mma_commit(bar_drained);
      }
    } else if (warp == 2) {
      // ============================================================ per-head operand builder
      int head_prev = -1, events = 0;
      bool ok = true;
      for (int i = 0; i < ntiles && ok; ++i) {
        const int head = (t_begin + i) / prm.tiles_per_head;
        if (head == head_prev) continue;
        if (events > 0) ok = mbar_wait(bar_drained, (events - 1) & 1, prm.status, &abort_flag);
        if (!ok) break;
        if (lane == 0) {
          // a^T of the new head, the resident B operand of the second product
          mbar_arrive_expect_tx(bar_atfull, (uint32_t)d * p * 2);
          for (int kb = 0; kb < kp; ++kb) tma_load_3d(base + L.aT + kb * (d * 128), &tmAT, bar_atfull, kb * 64, 0, head);
        }
        const float* wv = prm.weight + (size_t)head * p;
        float mx = -INFINITY;
        for (int f = lane; f < p; f += 32) mx = fmaxf(mx, wv[f]);
#pragma unroll
        for (int o = 16; o > 0; o >>= 1) mx = fmaxf(mx, __shfl_xor_sync(0xffffffffu, mx, o));
        if (kPerformer) {
          // bias[f][c], c < 16, no swizzle: offset = (f/8)*256 + (c/8)*128 + (f%8)*16 + (c%8)*2 bytes
          __nv_bfloat16* bias = reinterpret_cast<__nv_bfloat16*>(base_ptr + L.bias);
          for (int f = lane; f < 256; f += 32) {
            float b = (f < p) ? wv[f] - mx : 0.f;
            const __nv_bfloat16 h0 = __float2bfloat16_rn(b);  b -= __bfloat162float(h0);
            const __nv_bfloat16 h1 = __float2bfloat16_rn(b);  b -= __bfloat162float(h1);
            const __nv_bfloat16 h2 = __float2bfloat16_rn(b);
            __nv_bfloat16* row = bias + (f >> 3) * 128 + (f & 7) * 8;
            row[0] = h0; row[1] = h1; row[2] = h2;
#pragma unroll
            for (int c = 3; c < 8; ++c) row[c] = __float2bfloat16_rn(0.f);
#pragma unroll
            for (int c = 0; c < 8; ++c) row[64 + c] = __float2bfloat16_rn(0.f);
          }
          fence_proxy_async_smem();
        } else {
          float* sc = reinterpret_cast<float*>(base_ptr + L.scale);
          const float inv = 1.f / mx;
          for (int f = lane; f < p; f += 32) sc[f] = wv[f] * inv;
          __syncwarp();
          if (lane == 0) {
            __threadfence_block();
            scale_epoch = events + 1;
          }
        }
        mbar_arrive(bar_biasready);
        head_prev = head;
        ++events;
      }
    } else if (warp >= 4) {
      // ============================================================ row owners (two groups of 4 warps)
      const int grp = (warp - 4) >> 2;                 // tiles with (i & 1) == grp
      const int q4 = warp & 3;                         // TMEM lane quadrant
      const int row = q4 * 32 + lane;                  // row of the tile this thread owns
      const uint32_t lane_off = (uint32_t)(q4 * 32) << 16;
      const float kLog2e = 1.4426950408889634f;
      int events = 0;
      bool ok = true;
      // read-out of tile j: O / sum -> bf16 -> the output rows
      // (head and first row of the tile are tracked by the caller: no divisions on this path)
      const uint32_t slab = base + L.ostage + (uint32_t)(warp - 4) * 4096u;
      auto read_out = [&](int j, float inv, int head, int row0) -> bool {
        const int buf = j & (NB - 1);
        const uint32_t tb = tmem + buf * buf_cols + lane_off + o_col;
        if (!mbar_wait(bar_ofull + 8 * buf, (j >> nb_shift) & 1, prm.status, &abort_flag)) return false;
        tcgen05_fence_after();
        if (d == 64) {
          // d = 64: the warp's 32 rows go through a 4 KB slab of shared memory (128-byte rows, 16-byte
          // chunks swizzled like the tensor map expects, so the stores do not collide) and leave as one
          // TMA store of whole lines; rows past the end of the sequence are clipped by the tensor map
          if (lane == 0) bulk_wait_group_read0();          // the slab's previous store has been read
          __syncwarp();
          uint32_t ra[32], rb[32];
          tmem_ld32(tb, ra);
          tmem_ld32(tb + 32, rb);
          tmem_wait_ld(ra);
          tmem_wait_ld(rb);
          tcgen05_fence_before();
          mbar_arrive(bar_sfree + 8 * buf);                 // the buffer goes back before the rows are packed
#pragma unroll
          for (int g = 0; g < 8; ++g) {
            const uint32_t* src = g < 4 ? ra : rb;
            uint32_t v[4];
#pragma unroll
            for (int e = 0; e < 4; ++e) {
              const __nv_bfloat162 o2 = __floats2bfloat162_rn(__uint_as_float(src[(g & 3) * 8 + 2 * e]) * inv,
                                                              __uint_as_float(src[(g & 3) * 8 + 2 * e + 1]) * inv);
              v[e] = *reinterpret_cast<const uint32_t*>(&o2);
            }
            asm volatile("st.shared.v4.b32 [%0], {%1, %2, %3, %4};" ::"r"(slab + lane * 128 + ((g ^ (lane & 7)) << 4)),
                         "r"(v[0]), "r"(v[1]), "r"(v[2]), "r"(v[3]) : "memory");
          }
          fence_proxy_async_smem();
          __syncwarp();
          if (lane == 0 && row0 + q4 * 32 < prm.N) {
            if (prm.H > 0) tma_store_3d(&tmO, slab, (head % prm.H) * d, row0 + q4 * 32, head / prm.H);
            else tma_store_3d(&tmO, slab, 0, row0 + q4 * 32, head);
            bulk_commit_group();
          }
          return true;
        }
        __nv_bfloat16* orow = prm.H > 0
            ? prm.out + (((size_t)(head / prm.H) * prm.N + row0 + row) * prm.H + (size_t)(head % prm.H)) * d
            : prm.out + ((size_t)head * prm.N + row0 + row) * d;
        const bool in_range = row0 + row < prm.N;        // rows past the end of the sequence exist only in the tile
        for (int c = 0; c < d; c += 64) {
          uint32_t ra[32], rb[32];
          tmem_ld32(tb + c, ra);
          tmem_ld32(tb + c + 32, rb);
          tmem_wait_ld(ra);
          tmem_wait_ld(rb);
          if (c + 64 >= d) {
            // everything this tile needs from TMEM is in registers: hand the buffer back before storing
            tcgen05_fence_before();
            mbar_arrive(bar_sfree + 8 * buf);
          }
#pragma unroll
          for (int g8 = 0; g8 < 4; ++g8) {
            const uint32_t* src = g8 < 2 ? ra : rb;
            uint32_t v[8];
#pragma unroll
            for (int e = 0; e < 8; ++e) {
              const __nv_bfloat162 o2 = __floats2bfloat162_rn(__uint_as_float(src[(g8 & 1) * 16 + 2 * e]) * inv,
                                                              __uint_as_float(src[(g8 & 1) * 16 + 2 * e + 1]) * inv);
              v[e] = *reinterpret_cast<const uint32_t*>(&o2);
            }
            if (in_range)
            asm volatile("st.global.v8.b32 [%0], {%1, %2, %3, %4, %5, %6, %7, %8};" ::"l"(orow + c + g8 * 16),
                         "r"(v[0]), "r"(v[1]), "r"(v[2]), "r"(v[3]), "r"(v[4]), "r"(v[5]), "r"(v[6]), "r"(v[7])
                         : "memory");
          }
        }
        return true;
      };
      // a block of 64 features of p is complete: every row owner waits for its own TMEM stores and
      // tells the issuer of the second product
      auto hand_over = [&](int buf, int kb) {
        tmem_wait_st();
        tcgen05_fence_before();
        mbar_arrive(bar_pfull + 8 * (4 * buf + kb));
      };
      float inv_prev = 0.f;                            // four buffers: 1 / sum of the group's previous tile
      // head and tile-within-head of this group's current tile, advanced by two tiles per iteration;
      // the previous tile's pair is kept for the late read-out
      const int head_first = t_begin / prm.tiles_per_head;
      int head_i = (t_begin + grp) / prm.tiles_per_head, tih = (t_begin + grp) % prm.tiles_per_head;
      int head_o = head_i, row0_o = 0;
      const int ns_mask = NS - 1, ns_shift = NS == 4 ? 2 : 1;   // NS is 2 or 4
      for (int i = grp; i < ntiles && ok; i += 2) {
        const int buf = i & (NB - 1), st = i & ns_mask;
        const uint32_t tb = tmem + buf * buf_cols + lane_off;
        float denom = 0.f, denom1 = 0.f;
        const int head = head_i, row0 = tih * 128;
        events = head - head_first + 1;                // heads met so far, the way the other roles count them
        if (kPerformer) {
          ok = mbar_wait(bar_sfull + 8 * buf, (i >> nb_shift) & 1, prm.status, &abort_flag);
          if (!ok) break;
          tcgen05_fence_after();
          // Two passes over the row with double-buffered TMEM loads: while one 32-column chunk is
          // being worked on, the next one is already in flight.
          // pass 1: row maximum
          float mx = -INFINITY, mx1 = -INFINITY, mx2 = -INFINITY, mx3 = -INFINITY;
          uint32_t ra[32], rb[32];
          tmem_ld32(tb, ra);
          for (int c = 0; c < p; c += 64) {
            tmem_wait_ld(ra);
            tmem_ld32(tb + c + 32, rb);
#pragma unroll
            for (int e = 0; e < 32; e += 8) {      // four independent chains
              mx = fmax3(mx, __uint_as_float(ra[e]), __uint_as_float(ra[e + 1]));
              mx1 = fmax3(mx1, __uint_as_float(ra[e + 2]), __uint_as_float(ra[e + 3]));
              mx2 = fmax3(mx2, __uint_as_float(ra[e + 4]), __uint_as_float(ra[e + 5]));
              mx3 = fmax3(mx3, __uint_as_float(ra[e + 6]), __uint_as_float(ra[e + 7]));
            }
            tmem_wait_ld(rb);
            tmem_ld32(tb + ((c + 64 < p) ? c + 64 : 0), ra);      // last round: first chunk of pass 2
#pragma unroll
            for (int e = 0; e < 32; e += 8) {
              mx = fmax3(mx, __uint_as_float(rb[e]), __uint_as_float(rb[e + 1]));
              mx1 = fmax3(mx1, __uint_as_float(rb[e + 2]), __uint_as_float(rb[e + 3]));
              mx2 = fmax3(mx2, __uint_as_float(rb[e + 4]), __uint_as_float(rb[e + 5]));
              mx3 = fmax3(mx3, __uint_as_float(rb[e + 6]), __uint_as_float(rb[e + 7]));
            }
          }
          mx = fmaxf(fmax3(mx, mx1, mx2), mx3);
          const float shift = mx * kLog2e;
          // pass 2: p = 2^(S log2e - shift), fp16 pairs back into the buffer at half the width.  Scale and
          // shift and the row sums run two-wide; three pairs in eight take their exponential as a cubic on
          // the FMA pipe, the others on the special-function unit, which is the busiest unit of this kernel
          // (an all-MUFU loop of two warps per scheduler takes 8.9 cycles per warp-wide ex2; this mix 7.1).
          const uint64_t l2 = pack2(kLog2e, kLog2e), ms2 = pack2(-shift, -shift);
          uint64_t den2 = pack2(0.f, 0.f);
          auto exp_block = [&](const uint32_t (&r)[32], uint32_t (&h)[16]) {
#pragma unroll
            for (int e = 0; e < 16; ++e) {
              uint64_t x2 = fma2(pack2u(r[2 * e], r[2 * e + 1]), l2, ms2);
              float e0, e1;
              if ((e & 7) == 1 || (e & 7) == 4 || (e & 7) == 6) {
                float x0, x1;
                unpack2(x2, x0, x1);
                // far below what fp16 can hold the result is 0 either way; the cubic needs its exponent in range
                exp2_cubic2(pack2(fmaxf(x0, -60.f), fmaxf(x1, -60.f)), e0, e1);
              } else {
                float x0, x1;
                unpack2(x2, x0, x1);
                e0 = ex2_approx(x0);
                e1 = ex2_approx(x1);
              }
              den2 = add2(den2, pack2(e0, e1));
              const __half2 hh = __floats2half2_rn(e0, e1);
              h[e] = *reinterpret_cast<const uint32_t*>(&hh);
            }
          };
          for (int c = 0; c < p; c += 64) {
            uint32_t h[16];
            tmem_wait_ld(ra);
            tmem_ld32(tb + c + 32, rb);
            exp_block(ra, h);
            const uint32_t pc = pcol(c >> 6);
            tmem_st16(tb + pc, h);
            tmem_wait_ld(rb);
            if (c + 64 < p) tmem_ld32(tb + c + 64, ra);
            exp_block(rb, h);
            tmem_st16(tb + pc + 16, h);
            if ((c >> 6) >= q_first && c + 64 < p) hand_over(buf, c >> 6);
          }
          unpack2(den2, denom, denom1);
        } else {
          // RNN: p_f = (elu(q_f) + 1) * z_f / max z, features = the d entries of the Q row
          // (no wait for the buffer: this thread has itself read out the tile that used it before, and
          // the second product starts only when all 128 owners have said so)
          // this head's scale vector is in place (it is replaced only after every product of this head, hence
          // every row owner's use of it, is complete)
          if (scale_epoch < events) {
            const uint64_t t0 = global_timer_ns();
            uint32_t spins = 0;
            while (scale_epoch < events) {
              if ((++spins & 63u) == 0) {
                if (abort_flag) { ok = false; break; }
                if (global_timer_ns() - t0 > kWaitLimitNs) {
                  atomicOr(prm.status, 1);
                  abort_flag = 1;
                  ok = false;
                  break;
                }
              }
            }
          }
          __threadfence_block();
          if (ok) ok = mbar_wait(bar_qfull + 8 * st, (i >> ns_shift) & 1, prm.status, &abort_flag);
          if (!ok) break;
          const uint32_t qb = base + L.q + st * q_stage_bytes;
          const float* sc = reinterpret_cast<const float*>(base_ptr + L.scale);
          for (int c = 0; c < d; c += 32) {
            uint32_t h[16];
#pragma unroll
            for (int ch = 0; ch < 4; ++ch) {
              const int col = c + ch * 8;
              const uint32_t a = qb + (col >> 6) * 16384 + row * 128 + ((((col & 63) >> 3) ^ (row & 7)) << 4);
              uint32_t v[4];
              asm volatile("ld.shared.v4.b32 {%0, %1, %2, %3}, [%4];"
                           : "=r"(v[0]), "=r"(v[1]), "=r"(v[2]), "=r"(v[3]) : "r"(a));
              // the eight scale factors of these features: two 16-byte loads (every lane reads the same words)
              const float4 s0 = *reinterpret_cast<const float4*>(sc + col);
              const float4 s1 = *reinterpret_cast<const float4*>(sc + col + 4);
              const float scv[8] = {s0.x, s0.y, s0.z, s0.w, s1.x, s1.y, s1.z, s1.w};
#pragma unroll
              for (int e = 0; e < 4; ++e) {
                // a bf16 is the upper half of an fp32
                const float x0 = __uint_as_float(v[e] << 16), x1 = __uint_as_float(v[e] & 0xffff0000u);
                // elu(x) + 1 = max(x, 0) + exp(min(x, 0))
                const float f0 = (fmaxf(x0, 0.f) + ex2_approx(fminf(x0, 0.f) * kLog2e)) * scv[2 * e];
                const float f1 = (fmaxf(x1, 0.f) + ex2_approx(fminf(x1, 0.f) * kLog2e)) * scv[2 * e + 1];
                denom += f0;
                denom1 += f1;
                const __half2 hh = __floats2half2_rn(f0, f1);
                h[ch * 4 + e] = *reinterpret_cast<const uint32_t*>(&hh);
              }
            }
            tmem_st16(tb + (c >> 1), h);
            if ((c & 32) != 0 && c + 32 < d) hand_over(buf, c >> 6);
          }
          mbar_arrive(bar_qempty + 8 * st);             // this thread is done with the Q tile
        }
        hand_over(buf, kp - 1);                         // the last block of the tile

        const float inv = 1.f / fmaxf(denom + denom1, 1.17549435e-38f);
        if (NB == 4) {
          // two tiles of this group are in flight: read out the previous one, whose second product
          // has had this tile's passes to finish
          if (i >= 2) ok = read_out(i - 2, inv_prev, head_o, row0_o);
          inv_prev = inv;
          head_o = head;
          row0_o = row0;
        } else {
          ok = read_out(i, inv, head, row0);
        }
        tih += 2;
        while (tih >= prm.tiles_per_head) { tih -= prm.tiles_per_head; ++head_i; }
      }
      if (NB == 4 && ok && ntiles > grp) (void)read_out(grp + 2 * ((ntiles - 1 - grp) / 2), inv_prev, head_o, row0_o);
      if (lane == 0) bulk_wait_group0();                // this warp's output stores are complete
    }
  }
  tcgen05_fence_before();
  __syncthreads();
  if (warp == 1) tmem_dealloc(tmem, 512);
}

}  // namespace flurka

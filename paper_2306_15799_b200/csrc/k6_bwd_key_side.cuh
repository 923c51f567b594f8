// Backward of the key side on tensor cores (PERFORMER, d = 64; k a multiple of 64 up to 512, p = 64 .. 256).
//
// Forward (arxiv 2306.15799, Eq. (2) with Appendix D's normaliser, per feature i in the log domain):
//     L_ij = w_i . k'_j - |k'_j|^2 / 2,   b_i = log sum_j exp(L_ij),   A_ij = exp(L_ij - b_i),   a_i = sum_j A_ij v'_j.
// Given da_i, db_i (from the query side), by the chain rule
//     g_ij = da_i . v'_j + e_i  with  e_i = db_i - da_i . a_i,        dL_ij = A_ij g_ij,
//     dv'_j = sum_i A_ij da_i,        dk'_j = sum_i dL_ij w_i - k'_j sum_i dL_ij.
// One CTA owns 128 projected keys of one head and walks the features 128 at a time; every product is a
// tcgen05 MMA with fp32 accumulators in TMEM:
//     L = W K'^T + 1 n^T (K' as three bf16 terms and n_j = -|k'_j|^2/2 as three more: the exponent needs fp32),
//     T = da V'^T (both as two bf16 terms),
//     dV' += A^T da,   dK' += dL^T W,   s += dL^T 1      (A, dL as bf16 tiles the feature owners write into
//     shared memory in the canonical 128-byte-swizzled layout, read as MN-major A operands),
// and the key owners finish with dk'_j = (dL^T W)_j - k'_j s_j.  Nothing is shared between CTAs: dK', dV' rows
// are written once, with plain stores.
#pragma once

#include <cuda_bf16.h>

#include "tc_common.cuh"

namespace flurka {

struct K6Params {
  int k, p, BH;                 // d = 64
  const float* kpvp;            // [2][BH][k][64]  K', V'
  const float* weight;          // [BH][p]         b_i
  const float* a32;             // [BH][p][64]
  const float* da;              // [BH][p][64]
  const float* db;              // [BH][p]
  float* dkpvp;                 // [2][BH][k][64]  dK', dV'
  int* status;
};

constexpr int kK6Threads = 256;
// shared memory: W tile 16 KB | K' three terms 48 KB | n operand 4 KB | ones 4 KB | V' two terms 32 KB |
// da two terms 32 KB | A tile 32 KB | dL tile 32 KB | ones-column operand 4 KB | barriers
constexpr uint32_t kK6W = 0, kK6K3 = 16384, kK6Nrm = 65536, kK6Ones = 69632, kK6V2 = 73728, kK6Da2 = 106496,
                   kK6A = 139264, kK6DL = 172032, kK6One16 = 204800, kK6Bars = 208896;
constexpr int kK6SmemBytes = 208896 + 256 + 1024;
// TMEM columns: L 0..127, T 128..255, dV' 256..319, dK' 320..383, s 384..399
constexpr uint32_t kK6ColT = 128, kK6ColDV = 256, kK6ColDK = 320, kK6ColS = 384;

__device__ __forceinline__ uint32_t k6_bf16x2(float lo, float hi) {
  uint32_t r;
  asm("cvt.rn.bf16x2.f32 %0, %2, %1;" : "=r"(r) : "f"(lo), "f"(hi));
  return r;
}
__device__ __forceinline__ float k6_ex2(float x) {
  float y;
  asm("ex2.approx.ftz.f32 %0, %1;" : "=f"(y) : "f"(x));
  return y;
}

// four fp32 values of a row -> `terms` bf16 terms, each into its own K-major 128-byte-swizzled [128 x 64] tile
// (tiles 16384 B apart): row r, columns c4 .. c4 + 3
template <int kTerms>
__device__ __forceinline__ void k6_split_store(uint32_t tile0, int r, int c4, float4 x) {
  float a = x.x, b = x.y, c = x.z, e = x.w;
  const uint32_t off = tile0 + (uint32_t)r * 128u + ((((uint32_t)c4 >> 3) ^ ((uint32_t)r & 7u)) << 4) + (((uint32_t)c4 & 4u) << 1);
#pragma unroll
  for (int t = 0; t < kTerms; ++t) {
    const uint32_t h0 = k6_bf16x2(a, b), h1 = k6_bf16x2(c, e);
    asm volatile("st.shared.v2.b32 [%0], {%1, %2};" ::"r"(off + (uint32_t)t * 16384u), "r"(h0), "r"(h1) : "memory");
    a -= __uint_as_float(h0 << 16); b -= __uint_as_float(h0 & 0xffff0000u);
    c -= __uint_as_float(h1 << 16); e -= __uint_as_float(h1 & 0xffff0000u);
  }
}

__global__ void __launch_bounds__(kK6Threads, 1)
k6_bwd_key_side(const __grid_constant__ CUtensorMap tmW, const K6Params prm) {
  using namespace tc;
  extern __shared__ uint8_t smem_raw[];
  const uint32_t base = (smem_u32(smem_raw) + 1023u) & ~1023u;
  uint8_t* base_ptr = smem_raw + (base - smem_u32(smem_raw));
  const uint32_t bars = base + kK6Bars;
  const uint32_t bar_w = bars, bar_mma = bars + 8, bar_mma2 = bars + 16, tmem_slot = bars + 24;
  __shared__ int abort_flag;
  __shared__ uint32_t tmem_base_shared;

  const int tid = threadIdx.x, warp = tid >> 5, lane = tid & 31;
  const int k = prm.k, p = prm.p;
  const int nkc = (k + 127) >> 7;                       // key chunks per head
  const int head = blockIdx.x / nkc, jc = blockIdx.x % nkc;
  const int j0 = jc * 128, keys = min(128, k - j0);     // 64 or 128 live keys
  const int nft = (p + 127) >> 7;                       // feature tiles
  const float* __restrict__ Kp = prm.kpvp + ((size_t)head * k + j0) * 64;
  const float* __restrict__ Vp = prm.kpvp + (((size_t)prm.BH + head) * k + j0) * 64;

  if (tid == 0) {
    abort_flag = 0;
    mbar_init(bar_w, 1);
    mbar_init(bar_mma, 1);
    mbar_init(bar_mma2, 1);
    fence_mbar_init();
  }
  if (warp == 4) {
    tmem_alloc(tmem_slot, 512);
    tmem_relinquish();
  }
  if (warp == 5) {
    // A operand of the bias step: [128 x 16] bf16, no swizzle, columns 0..2 are 1
    // (element (r, c) at (r/8)*256 + (c/8)*128 + (r%8)*16 + (c%8)*2 bytes)
    __nv_bfloat16* ones = reinterpret_cast<__nv_bfloat16*>(base_ptr + kK6Ones);
    for (int e = lane; e < 128 * 16; e += 32) {
      const int r = e >> 4, c = e & 15;
      ones[(r >> 3) * 128 + (c >> 3) * 64 + (r & 7) * 8 + (c & 7)] = __float2bfloat16_rn(c < 3 ? 1.f : 0.f);
    }
  }
  if (warp == 6) {
    // B operand of the column sums: [16 x 128] (K-major, no swizzle), row 0 all ones:
    // element (c, n) at (c/8)*2048 + (n/8)*128 + (c%8)*16 + (n%8)*2 bytes
    __nv_bfloat16* o16 = reinterpret_cast<__nv_bfloat16*>(base_ptr + kK6One16);
    for (int e = lane; e < 2048; e += 32) {
      const int n = ((e >> 6) & 15) * 8 + (e & 7), c = ((e >> 3) & 7) + (e >> 10) * 8;
      o16[e] = __float2bfloat16_rn(c == 0 && n < 128 ? 1.f : 0.f);
    }
  }
  // ---- K' and V' of the chunk, once: fp32 rows from the workspace -> bf16 terms; n_j = -|k'_j|^2 / 2
  {
    const int ccol = (lane & 15) * 4;                   // 16 lanes per row of 64 floats
    for (int r = warp * 2 + (lane >> 4); r < 128; r += 16) {
      const bool live = r < keys;
      const float4 xk = live ? *reinterpret_cast<const float4*>(Kp + (size_t)r * 64 + ccol) : make_float4(0.f, 0.f, 0.f, 0.f);
      const float4 xv = live ? *reinterpret_cast<const float4*>(Vp + (size_t)r * 64 + ccol) : make_float4(0.f, 0.f, 0.f, 0.f);
      k6_split_store<3>(base + kK6K3, r, ccol, xk);
      k6_split_store<2>(base + kK6V2, r, ccol, xv);
      float sq = fmaf(xk.x, xk.x, fmaf(xk.y, xk.y, fmaf(xk.z, xk.z, xk.w * xk.w)));
#pragma unroll
      for (int o = 8; o > 0; o >>= 1) sq += __shfl_xor_sync(0xffffffffu, sq, o);
      if ((lane & 15) == 0) {
        float bb = -0.5f * sq;
        const __nv_bfloat16 g0 = __float2bfloat16_rn(bb);  bb -= __bfloat162float(g0);
        const __nv_bfloat16 g1 = __float2bfloat16_rn(bb);  bb -= __bfloat162float(g1);
        const __nv_bfloat16 g2 = __float2bfloat16_rn(bb);
        const uint32_t na = base + kK6Nrm + (uint32_t)(r >> 3) * 256u + (uint32_t)(r & 7) * 16u;
        const uint32_t z = 0;
        asm volatile("st.shared.v4.b32 [%0], {%1, %2, %3, %4};" ::"r"(na),
                     "r"((uint32_t)__bfloat16_as_ushort(g0) | ((uint32_t)__bfloat16_as_ushort(g1) << 16)),
                     "r"((uint32_t)__bfloat16_as_ushort(g2)), "r"(z), "r"(z) : "memory");
        asm volatile("st.shared.v4.b32 [%0], {%1, %2, %3, %4};" ::"r"(na + 128), "r"(z), "r"(z), "r"(z), "r"(z) : "memory");
      }
    }
  }
  fence_proxy_async_smem();
  tcgen05_fence_before();
  __syncthreads();
  tcgen05_fence_after();
  if (tid == 0) {
    uint32_t v;
    asm volatile("ld.shared.u32 %0, [%1];" : "=r"(v) : "r"(tmem_slot));
    tmem_base_shared = v;
    prefetch_tmap(&tmW);
  }
  __syncthreads();
  const uint32_t tmem = tmem_base_shared;
  const uint32_t lane_off = (uint32_t)((warp & 3) * 32) << 16;
  const float kLog2e = 1.4426950408889634f;
  const uint32_t idescL = make_idesc(kFmtBF16, 0, 0, 128, 128);    // L, T: both operands K-major
  const uint32_t idescO = make_idesc(kFmtBF16, 1, 1, 128, 64);     // dV', dK': MN-major A (A / dL tile) and B (da / W tile)
  const uint32_t idescS = make_idesc(kFmtBF16, 1, 0, 128, 16);     // s: MN-major A, K-major ones column
  bool ok = true;
  uint32_t ph_w = 0, ph_mma = 0, ph_mma2 = 0;

  for (int ft = 0; ft < nft && ok; ++ft) {
    const int i0 = ft * 128;
    // (the products of the previous feature tile that read W, da, A and dL are complete: waited for below)
    if (tid == 0) {
      mbar_arrive_expect_tx(bar_w, 16384u);
      tma_load_2d(base + kK6W, &tmW, bar_w, 0, i0);       // rows past p read as zero
    }
    // da of the tile -> two bf16 terms (rows past p: zero)
    {
      const int ccol = (lane & 15) * 4;
      for (int r = warp * 2 + (lane >> 4); r < 128; r += 16) {
        const float4 x = (i0 + r < p) ? *reinterpret_cast<const float4*>(prm.da + ((size_t)head * p + i0 + r) * 64 + ccol)
                                      : make_float4(0.f, 0.f, 0.f, 0.f);
        k6_split_store<2>(base + kK6Da2, r, ccol, x);
      }
    }
    // this feature's scalars (threads 0..127: feature = thread)
    float b_i = 0.f, e_i = 0.f;
    const int feat = i0 + (warp & 3) * 32 + lane;
    const bool feat_live = warp < 4 && feat < p;
    if (feat_live) {
      const float4* dr = reinterpret_cast<const float4*>(prm.da + ((size_t)head * p + feat) * 64);
      const float4* ar = reinterpret_cast<const float4*>(prm.a32 + ((size_t)head * p + feat) * 64);
      float dot = 0.f;
#pragma unroll 4
      for (int c = 0; c < 16; ++c) {
        const float4 x = dr[c], y = ar[c];
        dot = fmaf(x.x, y.x, fmaf(x.y, y.y, fmaf(x.z, y.z, fmaf(x.w, y.w, dot))));
      }
      e_i = prm.db[(size_t)head * p + feat] - dot;
      b_i = prm.weight[(size_t)head * p + feat];
    }
    fence_proxy_async_smem();
    {
      const bool mine = mbar_wait(bar_w, ph_w, prm.status, &abort_flag);
      ph_w ^= 1;
      ok = __syncthreads_and(mine) != 0;
      if (!ok) break;
    }
    if (warp == 4 && elect_one()) {
      tcgen05_fence_after();
      const uint64_t aw = make_sdesc(base + kK6W, 16, 1024, kSwizzle128);
      for (int t = 0; t < 3; ++t) {
        const uint64_t bk = make_sdesc(base + kK6K3 + t * 16384, 16, 1024, kSwizzle128);
        mma_ss_x4(tmem, aw, bk, 2, 2, idescL, t > 0 ? 1u : 0u);
      }
      const uint64_t a1 = make_sdesc(base + kK6Ones, 128, 256, kSwizzleNone);
      const uint64_t b1 = make_sdesc(base + kK6Nrm, 128, 256, kSwizzleNone);
      mma_ss(tmem, a1, b1, idescL, 1u);
      // T = da V'^T: hi hi + hi lo + lo hi
      const uint64_t dh = make_sdesc(base + kK6Da2, 16, 1024, kSwizzle128);
      const uint64_t dl = make_sdesc(base + kK6Da2 + 16384, 16, 1024, kSwizzle128);
      const uint64_t vh = make_sdesc(base + kK6V2, 16, 1024, kSwizzle128);
      const uint64_t vl = make_sdesc(base + kK6V2 + 16384, 16, 1024, kSwizzle128);
      mma_ss_x4(tmem + kK6ColT, dh, vh, 2, 2, idescL, 0u);
      mma_ss_x4(tmem + kK6ColT, dh, vl, 2, 2, idescL, 1u);
      mma_ss_x4(tmem + kK6ColT, dl, vh, 2, 2, idescL, 1u);
      mma_commit(bar_mma);
    }
    // ---- feature owners: A_ij and dL_ij of their row, 32 keys at a time, into the two tiles
    bool mine = true;
    if (warp < 4) {
      mine = mbar_wait(bar_mma, ph_mma, prm.status, &abort_flag);
      if (mine) {
        tcgen05_fence_after();
        const int row = (warp & 3) * 32 + lane;
        const float keep = feat_live ? 1.f : 0.f;
        const float bs = b_i * kLog2e;
#pragma unroll 1
        for (int c = 0; c < 128; c += 32) {
          uint32_t rl[32], rt[32];
          tmem_ld32(tmem + lane_off + c, rl);
          tmem_ld32(tmem + lane_off + kK6ColT + c, rt);
          tmem_wait_ld(rl);
          tmem_wait_ld(rt);
          const uint32_t slab = (uint32_t)(c >> 6) * 16384u + (uint32_t)row * 128u;
#pragma unroll
          for (int g = 0; g < 4; ++g) {
            uint32_t aw4[4], lw4[4];
#pragma unroll
            for (int e = 0; e < 4; ++e) {
              const int j = 8 * g + 2 * e;
              const float a0 = keep * k6_ex2(fmaf(__uint_as_float(rl[j]), kLog2e, -bs));
              const float a1 = keep * k6_ex2(fmaf(__uint_as_float(rl[j + 1]), kLog2e, -bs));
              aw4[e] = k6_bf16x2(a0, a1);
              lw4[e] = k6_bf16x2(a0 * (__uint_as_float(rt[j]) + e_i), a1 * (__uint_as_float(rt[j + 1]) + e_i));
            }
            const uint32_t off = slab + (((uint32_t)(((c & 32) >> 3) + g) ^ (uint32_t)(row & 7)) << 4);
            asm volatile("st.shared.v4.b32 [%0], {%1, %2, %3, %4};" ::"r"(base + kK6A + off), "r"(aw4[0]), "r"(aw4[1]),
                         "r"(aw4[2]), "r"(aw4[3]) : "memory");
            asm volatile("st.shared.v4.b32 [%0], {%1, %2, %3, %4};" ::"r"(base + kK6DL + off), "r"(lw4[0]), "r"(lw4[1]),
                         "r"(lw4[2]), "r"(lw4[3]) : "memory");
          }
        }
        fence_proxy_async_smem();
        tcgen05_fence_before();
      }
    }
    ph_mma ^= 1;
    ok = __syncthreads_and(mine) != 0;
    if (!ok) break;
    if (warp == 4 && elect_one()) {
      tcgen05_fence_after();
      const uint32_t acc = ft > 0 ? 1u : 0u;
      // 128 features = 8 steps of 16 rows: 2048 B of the A / dL tile, of the da / W tile, 256 B of the ones column
      for (int j = 0; j < 2; ++j) {
        const uint64_t aa = make_sdesc(base + kK6A + j * 8192, 16384, 1024, kSwizzle128);
        const uint64_t al = make_sdesc(base + kK6DL + j * 8192, 16384, 1024, kSwizzle128);
        const uint64_t bh = make_sdesc(base + kK6Da2 + j * 8192, 8192, 1024, kSwizzle128);
        const uint64_t bl = make_sdesc(base + kK6Da2 + 16384 + j * 8192, 8192, 1024, kSwizzle128);
        const uint64_t bw = make_sdesc(base + kK6W + j * 8192, 8192, 1024, kSwizzle128);
        const uint64_t bo = make_sdesc(base + kK6One16 + j * 1024, 128, 2048, kSwizzleNone);
        mma_ss_x4(tmem + kK6ColDV, aa, bh, 128, 128, idescO, (acc || j > 0) ? 1u : 0u);
        mma_ss_x4(tmem + kK6ColDV, aa, bl, 128, 128, idescO, 1u);
        mma_ss_x4(tmem + kK6ColDK, al, bw, 128, 128, idescO, (acc || j > 0) ? 1u : 0u);
        mma_ss_x4(tmem + kK6ColS, al, bo, 128, 16, idescS, (acc || j > 0) ? 1u : 0u);
      }
      mma_commit(bar_mma2);
    }
    {
      const bool m2 = mbar_wait(bar_mma2, ph_mma2, prm.status, &abort_flag);
      ph_mma2 ^= 1;
      ok = __syncthreads_and(m2) != 0;
    }
  }

  // ---- key owners: dv'_j and dk'_j = (dL^T W)_j - k'_j s_j, one row of 64 floats each
  if (ok && warp < 4) {
    tcgen05_fence_after();
    const int j = (warp & 3) * 32 + lane;
    uint32_t rs[32];
    tmem_ld32(tmem + lane_off + kK6ColS, rs);             // column 0 of 16 (the load is 32 wide)
    tmem_wait_ld(rs);
    const float sj = __uint_as_float(rs[0]);
    const bool live = j < keys;
    float* dk = prm.dkpvp + ((size_t)head * k + j0 + (live ? j : 0)) * 64;
    float* dv = prm.dkpvp + (((size_t)prm.BH + head) * k + j0 + (live ? j : 0)) * 64;
    const float* kr = Kp + (size_t)(live ? j : 0) * 64;
#pragma unroll 1
    for (int c = 0; c < 64; c += 32) {
      uint32_t r1[32], r2[32];
      tmem_ld32(tmem + lane_off + kK6ColDK + c, r1);
      tmem_ld32(tmem + lane_off + kK6ColDV + c, r2);
      tmem_wait_ld(r1);
      tmem_wait_ld(r2);
      if (live) {
#pragma unroll
        for (int e = 0; e < 32; e += 4) {
          const float4 kv = *reinterpret_cast<const float4*>(kr + c + e);
          *reinterpret_cast<float4*>(dk + c + e) =
              make_float4(fmaf(-kv.x, sj, __uint_as_float(r1[e])), fmaf(-kv.y, sj, __uint_as_float(r1[e + 1])),
                          fmaf(-kv.z, sj, __uint_as_float(r1[e + 2])), fmaf(-kv.w, sj, __uint_as_float(r1[e + 3])));
          *reinterpret_cast<float4*>(dv + c + e) = make_float4(__uint_as_float(r2[e]), __uint_as_float(r2[e + 1]),
                                                               __uint_as_float(r2[e + 2]), __uint_as_float(r2[e + 3]));
        }
      }
    }
  }
  tcgen05_fence_before();
  __syncthreads();
  if (warp == 4) tmem_dealloc(tmem, 512);
}

}  // namespace flurka

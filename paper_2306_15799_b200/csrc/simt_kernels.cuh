// CUDA-core (fp32 FFMA) kernels for the three stages of the FLuRKA forward pass
// (arxiv 2306.15799, Eq. (2)).  They serve the float32 I/O configuration, every shape the
// tensor-core kernels do not cover, and the key-side stage of both paths.
//
// Stage 1  down-projection   K' = E K, V' = F V          (Section 2.1; sequence contraction)
// Stage 2  key side          per feature i:  b_i = log sum_j exp(L_ji),  a_i = softmax_j(L_.i)^T V'
//                            with L_ji = w_i.k'_j - |k'_j|^2/2            (PERFORMER)
//                            or  z_i = sum_j (elu(k'_ji)+1),  a_i = sum_j (elu(k'_ji)+1) v'_j / z_i  (RNN)
// Stage 3  query side        O_n = sum_i p_ni a_i / sum_i p_ni,  p_ni = exp(w_i.q_n + b_i - r_n)  (PERFORMER)
//                            or  p_ni = (elu(q_ni)+1) z_i                                          (RNN)
//
// Stage 2 + 3 are Eq. (2)'s phi(Q)(phi(K')^T V') / phi(Q)(phi(K')^T 1): phi(K')^T V' = diag(e^b) a and
// phi(K')^T 1 = e^b, so every per-feature scale e^{b_i} moves into the query-side exponent.  The
// 1/sqrt(m), exp(-|q|^2/2) and any per-row r_n cancel in the ratio.
#pragma once

#include <cuda_bf16.h>
#include <cuda_fp16.h>
#include <cuda_runtime.h>
#include <math.h>

namespace flurka {

// Where head bh of a [B,H,N,d] tensor (H == 0) or of a [B,N,H,d] tensor (H = number of heads) starts,
// and the distance between consecutive sequence positions of that head, in elements.
struct HeadView {
  size_t base, row_stride;
};
__host__ __device__ __forceinline__ HeadView head_view(int bh, int H, int N, int d) {
  HeadView v;
  if (H > 0) {
    v.base = ((size_t)(bh / H) * N * H + (size_t)(bh % H)) * d;
    v.row_stride = (size_t)H * d;
  } else {
    v.base = (size_t)bh * N * d;
    v.row_stride = (size_t)d;
  }
  return v;
}

__device__ __forceinline__ float to_f32(float x) { return x; }
__device__ __forceinline__ float to_f32(__nv_bfloat16 x) { return __bfloat162float(x); }
__device__ __forceinline__ void store_out(float* p, float v) { *p = v; }
__device__ __forceinline__ void store_out(__nv_bfloat16* p, float v) { *p = __float2bfloat16_rn(v); }

// ---------------------------------------------------------------------------------------------
// Stage 1.  grid = (ceil(k/32), B*H, 2*nsplit); block = 256.
// blockIdx.z = t*nsplit + s: t = 0 projects K with E, t = 1 projects V with F; split s covers the
// sequence range [s*chunk, min(N,(s+1)*chunk)).  Partial sums are added into KpVp (zeroed before).
// KpVp layout: [2][B*H][k][d] fp32.  E, F: [k][N] shared by all heads, or [H][k][N] (ef_heads = H).
// ---------------------------------------------------------------------------------------------
template <typename T>
__global__ void __launch_bounds__(256)
simt_down_project(const T* __restrict__ Kin, const T* __restrict__ Vin, const T* __restrict__ E,
                  const T* __restrict__ F, float* __restrict__ KpVp, int BH, int N, int d, int k,
                  int nsplit, int chunk, int seq_major_heads, int ef_heads) {
  constexpr int TJ = 32, TN = 32;
  __shared__ float Ps[TJ][TN + 1];
  __shared__ float Xs[TN][128];

  const int t = blockIdx.z / nsplit;
  const int s = blockIdx.z % nsplit;
  const int bh = blockIdx.y;
  const int j0 = blockIdx.x * TJ;
  // ef_heads > 0: E and F are [ef_heads][k][N], one pair per head (head = bh % ef_heads)
  const T* __restrict__ P = (t ? F : E) + (ef_heads > 0 ? (size_t)(bh % ef_heads) * k * N : 0);
  const HeadView hv = head_view(bh, seq_major_heads, N, d);
  const T* __restrict__ X = (t ? Vin : Kin) + hv.base;
  float* __restrict__ out = KpVp + ((size_t)t * BH + bh) * (size_t)k * d;

  const int n_begin = s * chunk;
  const int n_end = min(N, n_begin + chunk);
  const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;

  float acc[4][4];
#pragma unroll
  for (int a = 0; a < 4; ++a)
#pragma unroll
    for (int b = 0; b < 4; ++b) acc[a][b] = 0.f;

  for (int n0 = n_begin; n0 < n_end; n0 += TN) {
    // stage the projection tile [32 j][32 n] and the input tile [32 n][d]
    for (int idx = threadIdx.x; idx < TJ * TN; idx += 256) {
      const int jj = idx / TN, nn = idx % TN;
      const int j = j0 + jj, n = n0 + nn;
      Ps[jj][nn] = (j < k && n < n_end) ? to_f32(P[(size_t)j * N + n]) : 0.f;
    }
    for (int idx = threadIdx.x; idx < TN * 128; idx += 256) {
      const int nn = idx >> 7, c = idx & 127;
      const int n = n0 + nn;
      Xs[nn][c] = (n < n_end && c < d) ? to_f32(X[(size_t)n * hv.row_stride + c]) : 0.f;
    }
    __syncthreads();
#pragma unroll 4
    for (int nn = 0; nn < TN; ++nn) {
      float p[4], x[4];
#pragma unroll
      for (int a = 0; a < 4; ++a) p[a] = Ps[warp * 4 + a][nn];
#pragma unroll
      for (int b = 0; b < 4; ++b) x[b] = Xs[nn][lane + 32 * b];
#pragma unroll
      for (int a = 0; a < 4; ++a)
#pragma unroll
        for (int b = 0; b < 4; ++b) acc[a][b] = fmaf(p[a], x[b], acc[a][b]);
    }
    __syncthreads();
  }
#pragma unroll
  for (int a = 0; a < 4; ++a) {
    const int j = j0 + warp * 4 + a;
    if (j >= k) continue;
#pragma unroll
    for (int b = 0; b < 4; ++b) {
      const int c = lane + 32 * b;
      if (c < d) atomicAdd(out + (size_t)j * d + c, acc[a][b]);
    }
  }
}

// ---------------------------------------------------------------------------------------------
// Stage 2.  grid = (ceil(p/8), B*H); block = 256 (8 warps, one feature each); p = m or d.
// Dynamic shared memory: 8*k floats (the exponents / feature values of this block's features)
// followed by 32*(d+1) floats (one chunk of K' rows).
// Outputs: weight[bh][i] (b_i or z_i), a32[bh][i][c] fp32, aT16[bh][c][i] fp16 (either may be NULL).
// ---------------------------------------------------------------------------------------------
template <typename T, bool kPerformer>
__global__ void __launch_bounds__(256)
simt_key_side(const float* __restrict__ KpVp, const T* __restrict__ W, float* __restrict__ weight,
              float* __restrict__ a32, __half* __restrict__ aT16, int BH, int d, int k, int p) {
  extern __shared__ float smem[];
  float* Ls = smem;                 // [8][k]
  float* Ks = smem + 8 * k;         // [32][d+1]
  __shared__ float nrm[32];
  __shared__ float wrow[8][128];

  const int bh = blockIdx.y;
  const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
  const int i = blockIdx.x * 8 + warp;          // this warp's feature
  const bool live = i < p;
  const float* __restrict__ Kp = KpVp + (size_t)bh * k * d;
  const float* __restrict__ Vp = KpVp + ((size_t)BH + bh) * (size_t)k * d;

  if (kPerformer) {
    for (int c = lane; c < d; c += 32) wrow[warp][c] = live ? to_f32(W[(size_t)i * d + c]) : 0.f;
  }
  // pass 1: exponents L_ji (PERFORMER) or feature values elu(k'_ji)+1 (RNN), all keys j
  for (int j0 = 0; j0 < k; j0 += 32) {
    __syncthreads();
    for (int idx = threadIdx.x; idx < 32 * d; idx += 256) {
      const int jj = idx / d, c = idx % d;
      Ks[jj * (d + 1) + c] = (j0 + jj < k) ? Kp[(size_t)(j0 + jj) * d + c] : 0.f;
    }
    __syncthreads();
    if (kPerformer) {
      if (warp == 0) {
        float s = 0.f;
        for (int c = 0; c < d; ++c) { const float v = Ks[lane * (d + 1) + c]; s = fmaf(v, v, s); }
        nrm[lane] = 0.5f * s;
      }
      __syncthreads();
      float dot = 0.f;
      for (int c = 0; c < d; ++c) dot = fmaf(wrow[warp][c], Ks[lane * (d + 1) + c], dot);
      if (j0 + lane < k) Ls[warp * k + j0 + lane] = dot - nrm[lane];
    } else {
      if (j0 + lane < k) {
        const float x = live ? Ks[lane * (d + 1) + i] : 0.f;
        Ls[warp * k + j0 + lane] = x > 0.f ? x + 1.f : expf(x);
      }
    }
  }
  __syncwarp();
  // per-feature maximum (PERFORMER); RNN needs none
  float cmax = 0.f;
  if (kPerformer) {
    cmax = -INFINITY;
    for (int j = lane; j < k; j += 32) cmax = fmaxf(cmax, Ls[warp * k + j]);
#pragma unroll
    for (int o = 16; o > 0; o >>= 1) cmax = fmaxf(cmax, __shfl_xor_sync(0xffffffffu, cmax, o));
    for (int j = lane; j < k; j += 32) Ls[warp * k + j] = expf(Ls[warp * k + j] - cmax);
    __syncwarp();
  }
  // pass 2: z_i and the weighted sum of V' rows; lane owns columns lane, lane+32, ...
  float z = 0.f, acc[4] = {0.f, 0.f, 0.f, 0.f};
  for (int j = 0; j < k; ++j) {
    const float e = Ls[warp * k + j];
    z += e;
#pragma unroll
    for (int b = 0; b < 4; ++b) {
      const int c = lane + 32 * b;
      if (c < d) acc[b] = fmaf(e, Vp[(size_t)j * d + c], acc[b]);
    }
  }
  if (!live) return;
  const float inv = 1.f / z;
  if (lane == 0) weight[(size_t)bh * p + i] = kPerformer ? cmax + logf(z) : z;
#pragma unroll
  for (int b = 0; b < 4; ++b) {
    const int c = lane + 32 * b;
    if (c < d) {
      const float a = acc[b] * inv;
      if (a32) a32[((size_t)bh * p + i) * d + c] = a;
      if (aT16) aT16[((size_t)bh * d + c) * p + i] = __float2half_rn(a);
    }
  }
}

// ---------------------------------------------------------------------------------------------
// Stage 3.  grid = (ceil(N/32), B*H); block = 256: warp w owns rows 4w..4w+3 of the 32-row tile,
// lane owns feature (i0 + lane) while scoring and columns lane + 32t while accumulating.
// Features are streamed in chunks of 32 with an online (running-maximum) normalisation.
// Dynamic shared memory: 32*(d+1) floats (W chunk) + 32*d floats (a chunk).
// ---------------------------------------------------------------------------------------------
template <typename T, bool kPerformer>
__global__ void __launch_bounds__(256)
simt_query_side(const T* __restrict__ Q, const T* __restrict__ W, const float* __restrict__ weight,
                const float* __restrict__ a32, T* __restrict__ out, int N, int d, int p, int seq_major_heads) {
  extern __shared__ float smem[];
  float* Ws = smem;                  // [32][d+1]
  float* As = smem + 32 * (d + 1);   // [32][d]
  __shared__ float qs[32][128];
  __shared__ float ws[32];

  const int bh = blockIdx.y;
  const int n0 = blockIdx.x * 32;
  const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
  const HeadView hv = head_view(bh, seq_major_heads, N, d);
  const T* __restrict__ Qh = Q + hv.base;
  const float* __restrict__ ah = a32 + (size_t)bh * p * d;
  const float* __restrict__ wh = weight + (size_t)bh * p;

  for (int idx = threadIdx.x; idx < 32 * d; idx += 256) {
    const int r = idx / d, c = idx % d;
    qs[r][c] = (n0 + r < N) ? to_f32(Qh[(size_t)(n0 + r) * hv.row_stride + c]) : 0.f;
  }
  float run_max[4], run_sum[4], acc[4][4];
#pragma unroll
  for (int r = 0; r < 4; ++r) {
    run_max[r] = -INFINITY;
    run_sum[r] = 0.f;
#pragma unroll
    for (int b = 0; b < 4; ++b) acc[r][b] = 0.f;
  }

  for (int i0 = 0; i0 < p; i0 += 32) {
    __syncthreads();
    if (kPerformer) {
      for (int idx = threadIdx.x; idx < 32 * d; idx += 256) {
        const int ii = idx / d, c = idx % d;
        Ws[ii * (d + 1) + c] = (i0 + ii < p) ? to_f32(W[(size_t)(i0 + ii) * d + c]) : 0.f;
      }
    }
    for (int idx = threadIdx.x; idx < 32 * d; idx += 256) {
      const int ii = idx / d, c = idx % d;
      As[ii * d + c] = (i0 + ii < p) ? ah[(size_t)(i0 + ii) * d + c] : 0.f;
    }
    if (threadIdx.x < 32) ws[threadIdx.x] = (i0 + threadIdx.x < p) ? wh[i0 + threadIdx.x] : 0.f;
    __syncthreads();
    const bool feat_live = (i0 + lane) < p;
#pragma unroll
    for (int r = 0; r < 4; ++r) {
      const int row = warp * 4 + r;
      float pv;
      if (kPerformer) {
        float s = 0.f;
        for (int c = 0; c < d; ++c) s = fmaf(qs[row][c], Ws[lane * (d + 1) + c], s);
        s = feat_live ? s + ws[lane] : -INFINITY;
        float cm = s;
#pragma unroll
        for (int o = 16; o > 0; o >>= 1) cm = fmaxf(cm, __shfl_xor_sync(0xffffffffu, cm, o));
        const float new_max = fmaxf(run_max[r], cm);
        const float rescale = expf(run_max[r] - new_max);   // exp(-inf) = 0 on the first chunk
        run_max[r] = new_max;
        run_sum[r] *= rescale;
#pragma unroll
        for (int b = 0; b < 4; ++b) acc[r][b] *= rescale;
        pv = feat_live ? expf(s - new_max) : 0.f;
      } else {
        const float x = feat_live ? qs[row][i0 + lane] : 0.f;
        pv = feat_live ? (x > 0.f ? x + 1.f : expf(x)) * ws[lane] : 0.f;
      }
      float psum = pv;
#pragma unroll
      for (int o = 16; o > 0; o >>= 1) psum += __shfl_xor_sync(0xffffffffu, psum, o);
      run_sum[r] += psum;
      for (int ii = 0; ii < 32; ++ii) {
        const float pi = __shfl_sync(0xffffffffu, pv, ii);
#pragma unroll
        for (int b = 0; b < 4; ++b) {
          const int c = lane + 32 * b;
          if (c < d) acc[r][b] = fmaf(pi, As[ii * d + c], acc[r][b]);
        }
      }
    }
  }
#pragma unroll
  for (int r = 0; r < 4; ++r) {
    const int n = n0 + warp * 4 + r;
    if (n >= N) continue;
    const float inv = 1.f / fmaxf(run_sum[r], 1.17549435e-38f);
#pragma unroll
    for (int b = 0; b < 4; ++b) {
      const int c = lane + 32 * b;
      if (c < d) store_out(out + hv.base + (size_t)n * hv.row_stride + c, acc[r][b] * inv);
    }
  }
}

// ---------------------------------------------------------------------------------------------
// The linear maps of Eq. (2) and the contraction of un-projected inputs on CUDA cores: a plain
// batched C = A B with fp32 accumulation.  A: [Z][M][K] (batch stride a_stride, 0 = shared),
// B: [Z][K][ncols] (b_stride likewise), both row-major.  grid = (ceil(ncols/32), ceil(M/32), Z),
// block = 256 (a 32 x 32 tile of C, four rows per thread).
// head_d == 0: C is [Z][M][ncols] row-major.  head_d > 0: C is the K', V' workspace, fp32
// [(z0 + z) * ncols/head_d + col/head_d][M][head_d]: column block h of the product is head h's.
// ---------------------------------------------------------------------------------------------
template <typename TA, typename TB, typename TC>
__global__ void __launch_bounds__(256)
simt_linear_map(const TA* __restrict__ A, const TB* __restrict__ Bm, TC* __restrict__ C, int M, int K, int ncols,
                size_t a_stride, size_t b_stride, int head_d, int z0) {
  __shared__ float sa[32][33];
  __shared__ float sb[32][33];
  const int z = blockIdx.z;
  const TA* Az = A + (size_t)z * a_stride;
  const TB* Bz = Bm + (size_t)z * b_stride;
  const int tx = threadIdx.x & 31, ty = threadIdx.x >> 5;      // ty: 0..7
  const int row0 = blockIdx.y * 32, col0 = blockIdx.x * 32;
  float acc[4] = {0.f, 0.f, 0.f, 0.f};
  for (int k0 = 0; k0 < K; k0 += 32) {
#pragma unroll
    for (int r = 0; r < 4; ++r) {
      const int ar = row0 + ty + 8 * r, ak = k0 + tx;
      sa[ty + 8 * r][tx] = (ar < M && ak < K) ? to_f32(Az[(size_t)ar * K + ak]) : 0.f;
      const int bk = k0 + ty + 8 * r, bc = col0 + tx;
      sb[ty + 8 * r][tx] = (bk < K && bc < ncols) ? to_f32(Bz[(size_t)bk * ncols + bc]) : 0.f;
    }
    __syncthreads();
#pragma unroll 8
    for (int kk = 0; kk < 32; ++kk) {
      const float b = sb[kk][tx];
#pragma unroll
      for (int r = 0; r < 4; ++r) acc[r] = fmaf(sa[ty + 8 * r][kk], b, acc[r]);
    }
    __syncthreads();
  }
  const int col = col0 + tx;
  if (col >= ncols) return;
#pragma unroll
  for (int r = 0; r < 4; ++r) {
    const int row = row0 + ty + 8 * r;
    if (row >= M) continue;
    if (head_d > 0) {
      const size_t head = (size_t)(z0 + z) * (ncols / head_d) + col / head_d;
      store_out(C + (head * M + row) * head_d + col % head_d, acc[r]);
    } else {
      store_out(C + ((size_t)z * M + row) * ncols + col, acc[r]);
    }
  }
}

}  // namespace flurka

// Backward pass of the FLuRKA forward (arxiv 2306.15799, Eq. (2); the paper trains these models but
// prints no backward formulas: this is the chain rule through the three stages, CUDA cores, fp32).
//
// With the forward's per-feature summaries  a_i (a d-vector) and b_i = log z_i,  the output is
//     O_n = sum_i P_ni a_i,     P_n. = softmax_i(l_ni),   l_ni = w_i.q_n + b_i          (PERFORMER)
//                                                          l_ni = log(elu(q_ni)+1) + b_i  (RNN)
// and   a_i = sum_j A_ij v'_j,  b_i = log sum_j exp(L_ji),  A_i. = softmax_j(L_.i),
//     L_ji = w_i.k'_j - |k'_j|^2/2  (PERFORMER),   L_ji = log(elu(k'_ji)+1)  (RNN).
// Given dO:
//   query side   c_ni = P_ni (a_i.dO_n - O_n.dO_n)   (sums to zero over i)
//                dq_n = sum_i c_ni w_i  (PERFORMER; the -q_n sum_i c_ni term vanishes),
//                dq_ni = c_ni elu'(q_ni)/(elu(q_ni)+1)  (RNN)
//                da_i = sum_n P_ni dO_n,   db_i = sum_n c_ni
//   key side     g_ij = da_i.(v'_j - a_i) + db_i,   dL_ji = A_ij g_ij,   dv'_j = sum_i A_ij da_i,
//                dk'_j = sum_i dL_ji (w_i - k'_j)  (PERFORMER),  dk'_ji = dL_ji elu'(k'_ji)/(elu(k'_ji)+1)  (RNN)
//   projections  dK = E^T dK',  dV = F^T dV',  dE = sum_heads dK' K^T,  dF = sum_heads dV' V^T.
#pragma once

#include "simt_kernels.cuh"

namespace flurka {

__device__ __forceinline__ float elu1(float x) { return x > 0.f ? x + 1.f : expf(x); }
__device__ __forceinline__ float elu1_slope(float x) { return x > 0.f ? 1.f : expf(x); }

// ---------------------------------------------------------------------------------------------
// Query side.  grid = (ceil(N/32), B*H); block = 256: warp w owns rows 4w..4w+3 of the tile.
// Two sweeps over the features in chunks of 32: the first is the forward (running maximum, sum,
// O_n); the second forms c_ni and accumulates dq_n, da_i, db_i.  da, db (fp32, zeroed before) are
// added to with atomics: every row tile of a head contributes.
// Dynamic shared memory: 2 * 32 * (d+1) floats (W chunk, a chunk) + 32 * 33 (P tile) + 32 * d (dO tile).
// ---------------------------------------------------------------------------------------------
template <typename T, bool kPerformer>
__global__ void __launch_bounds__(256)
simt_bwd_query_side(const T* __restrict__ Q, const T* __restrict__ W, const T* __restrict__ dO,
                    const float* __restrict__ weight, const float* __restrict__ a32, T* __restrict__ dQ,
                    float* __restrict__ da, float* __restrict__ db, int N, int d, int p, int seq_major_heads) {
  extern __shared__ float smem[];
  float* Ws = smem;                          // [32][d+1]
  float* As = Ws + 32 * (d + 1);             // [32][d+1]
  float* Ps = As + 32 * (d + 1);             // [32 rows][33]
  float* Gs = Ps + 32 * 33;                  // [32 rows][d]   dO tile
  __shared__ float qs[32][128];
  __shared__ float ws[32];
  __shared__ float dbs[8][32];

  const int bh = blockIdx.y;
  const int n0 = blockIdx.x * 32;
  const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
  const HeadView hv = head_view(bh, seq_major_heads, N, d);
  const float* __restrict__ ah = a32 + (size_t)bh * p * d;
  const float* __restrict__ wh = weight + (size_t)bh * p;

  for (int idx = threadIdx.x; idx < 32 * d; idx += 256) {
    const int r = idx / d, c = idx % d;
    const bool in = n0 + r < N;
    qs[r][c] = in ? to_f32(Q[hv.base + (size_t)(n0 + r) * hv.row_stride + c]) : 0.f;
    Gs[r * d + c] = in ? to_f32(dO[hv.base + (size_t)(n0 + r) * hv.row_stride + c]) : 0.f;
  }
  float run_max[4], run_sum[4], acc[4][4];
#pragma unroll
  for (int r = 0; r < 4; ++r) {
    run_max[r] = kPerformer ? -INFINITY : 0.f;
    run_sum[r] = 0.f;
#pragma unroll
    for (int b = 0; b < 4; ++b) acc[r][b] = 0.f;
  }
  auto stage_chunk = [&](int i0) {
    __syncthreads();
    for (int idx = threadIdx.x; idx < 32 * d; idx += 256) {
      const int ii = idx / d, c = idx % d;
      const bool in = i0 + ii < p;
      if (kPerformer) Ws[ii * (d + 1) + c] = in ? to_f32(W[(size_t)(i0 + ii) * d + c]) : 0.f;
      As[ii * (d + 1) + c] = in ? ah[(size_t)(i0 + ii) * d + c] : 0.f;
    }
    if (threadIdx.x < 32) ws[threadIdx.x] = (i0 + threadIdx.x < p) ? wh[i0 + threadIdx.x] : 0.f;
    __syncthreads();
  };
  // unnormalised weight of (row, feature lane) and its logit: PERFORMER exp(s - max) with s = q.w + b
  auto logit = [&](int row, int i0, bool live) -> float {
    if (kPerformer) {
      float s = 0.f;
      for (int c = 0; c < d; ++c) s = fmaf(qs[row][c], Ws[lane * (d + 1) + c], s);
      return live ? s + ws[lane] : -INFINITY;
    }
    return live ? elu1(qs[row][i0 + lane]) * ws[lane] : 0.f;     // RNN: the weight itself, no exponent
  };

  // ---- sweep 1: the forward (O_n, the row maximum and sum)
  for (int i0 = 0; i0 < p; i0 += 32) {
    stage_chunk(i0);
    const bool live = (i0 + lane) < p;
#pragma unroll
    for (int r = 0; r < 4; ++r) {
      const int row = warp * 4 + r;
      float pv = logit(row, i0, live);
      if (kPerformer) {
        float cm = pv;
#pragma unroll
        for (int o = 16; o > 0; o >>= 1) cm = fmaxf(cm, __shfl_xor_sync(0xffffffffu, cm, o));
        const float new_max = fmaxf(run_max[r], cm);
        const float rescale = expf(run_max[r] - new_max);
        run_max[r] = new_max;
        run_sum[r] *= rescale;
#pragma unroll
        for (int b = 0; b < 4; ++b) acc[r][b] *= rescale;
        pv = live ? expf(pv - new_max) : 0.f;
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
          if (c < d) acc[r][b] = fmaf(pi, As[ii * (d + 1) + c], acc[r][b]);
        }
      }
    }
  }
  // t_r = O_r . dO_r
  float inv_sum[4], t[4], dq[4][4];
#pragma unroll
  for (int r = 0; r < 4; ++r) {
    inv_sum[r] = 1.f / fmaxf(run_sum[r], 1.17549435e-38f);
    float s = 0.f;
#pragma unroll
    for (int b = 0; b < 4; ++b) {
      const int c = lane + 32 * b;
      if (c < d) s = fmaf(acc[r][b] * inv_sum[r], Gs[(warp * 4 + r) * d + c], s);
      dq[r][b] = 0.f;
    }
#pragma unroll
    for (int o = 16; o > 0; o >>= 1) s += __shfl_xor_sync(0xffffffffu, s, o);
    t[r] = s;
  }

  // ---- sweep 2: c_ni, dq_n, da_i, db_i
  for (int i0 = 0; i0 < p; i0 += 32) {
    stage_chunk(i0);
    const bool live = (i0 + lane) < p;
    float db_part = 0.f;
#pragma unroll
    for (int r = 0; r < 4; ++r) {
      const int row = warp * 4 + r;
      const bool row_live = n0 + row < N;
      float pv = logit(row, i0, live);
      if (kPerformer) pv = live ? expf(pv - run_max[r]) : 0.f;
      const float P = row_live ? pv * inv_sum[r] : 0.f;
      float u = 0.f;
      for (int c = 0; c < d; ++c) u = fmaf(As[lane * (d + 1) + c], Gs[row * d + c], u);
      const float cv = P * (u - t[r]);
      db_part += cv;
      Ps[row * 33 + lane] = P;
      if (kPerformer) {
        for (int ii = 0; ii < 32; ++ii) {
          const float ci = __shfl_sync(0xffffffffu, cv, ii);
#pragma unroll
          for (int b = 0; b < 4; ++b) {
            const int c = lane + 32 * b;
            if (c < d) dq[r][b] = fmaf(ci, Ws[ii * (d + 1) + c], dq[r][b]);
          }
        }
      } else if (live && row_live) {
        // feature i is column i of the row: d log(elu(x)+1)/dx = elu'(x)/(elu(x)+1)
        const float x = qs[row][i0 + lane];
        store_out(dQ + hv.base + (size_t)(n0 + row) * hv.row_stride + i0 + lane, cv * elu1_slope(x) / elu1(x));
      }
    }
    dbs[warp][lane] = db_part;
    __syncthreads();
    // da_i[c] += sum over the tile's rows of P_ri dO_r[c]: warp w takes features 4w..4w+3 of the chunk
#pragma unroll
    for (int f = 0; f < 4; ++f) {
      const int ii = warp * 4 + f;
      if (i0 + ii >= p) continue;
      float s4[4] = {0.f, 0.f, 0.f, 0.f};
      for (int r = 0; r < 32; ++r) {
        const float pr = Ps[r * 33 + ii];
#pragma unroll
        for (int b = 0; b < 4; ++b) {
          const int c = lane + 32 * b;
          if (c < d) s4[b] = fmaf(pr, Gs[r * d + c], s4[b]);
        }
      }
#pragma unroll
      for (int b = 0; b < 4; ++b) {
        const int c = lane + 32 * b;
        if (c < d) atomicAdd(da + ((size_t)bh * p + i0 + ii) * d + c, s4[b]);
      }
    }
    if (warp == 0 && live) {
      float s = 0.f;
#pragma unroll
      for (int w8 = 0; w8 < 8; ++w8) s += dbs[w8][lane];
      atomicAdd(db + (size_t)bh * p + i0 + lane, s);
    }
  }
  if (kPerformer) {
#pragma unroll
    for (int r = 0; r < 4; ++r) {
      const int n = n0 + warp * 4 + r;
      if (n >= N) continue;
#pragma unroll
      for (int b = 0; b < 4; ++b) {
        const int c = lane + 32 * b;
        if (c < d) store_out(dQ + hv.base + (size_t)n * hv.row_stride + c, dq[r][b]);
      }
    }
  }
}

// ---------------------------------------------------------------------------------------------
// Key side.  grid = (ceil(k/32), B*H); block = 256: a warp owns four projected keys, so that every
// chunk of W, a, da a block brings into shared memory (32 features at a time) serves 32 keys and every
// value read from it in the inner loops serves four.  Lane = feature for the scalar parts (A_ij, g_ij),
// lane = column for the sums over features; A and dL of a chunk go through shared memory so that the
// column loop reads the four keys' values of a feature with one 16-byte broadcast load each.
// Inputs: K', V' (KpVp), W, a, b (weight), da, db.  Outputs: dKpVp [2][B*H][k][d] fp32 (dK' then dV').
// Dynamic shared memory: 3 * 32 * (d+1) floats (W, a, da chunks) + 2 * 32 * d floats (the block's keys, values).
// ---------------------------------------------------------------------------------------------
constexpr int kBwdKeysPerWarp = 4;
template <typename T, bool kPerformer>
__global__ void __launch_bounds__(256, 4)
simt_bwd_key_side(const float* __restrict__ KpVp, const T* __restrict__ W, const float* __restrict__ weight,
                  const float* __restrict__ a32, const float* __restrict__ da, const float* __restrict__ db,
                  float* __restrict__ dKpVp, int BH, int d, int k, int p) {
  constexpr int KW = kBwdKeysPerWarp;
  extern __shared__ float smem[];
  float* Ws = smem;                          // [32][d+1]
  float* As = Ws + 32 * (d + 1);             // [32][d+1]
  float* Ds = As + 32 * (d + 1);             // [32][d+1]  da chunk
  // the block's 8 * KW keys and values, rows of d floats (dynamic: d = 64 leaves room for a fourth block per SM)
  float* ks = Ds + 32 * (d + 1);             // [8 * KW][d]
  float* vs = ks + 8 * KW * d;               // [8 * KW][d]
  __shared__ __align__(16) float sA[8][32][KW], sdL[8][32][KW];
  __shared__ float bs[32], dbs[32];

  const int bh = blockIdx.y;
  const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
  const int j0 = (blockIdx.x * 8 + warp) * KW;                 // this warp's keys j0 .. j0 + KW - 1
  const float* __restrict__ Kp = KpVp + (size_t)bh * k * d;
  const float* __restrict__ Vp = KpVp + ((size_t)BH + bh) * (size_t)k * d;
  float half_sq[KW];
#pragma unroll
  for (int q = 0; q < KW; ++q) {
    const bool key_live = j0 + q < k;
    float hs = 0.f;
    for (int c = lane; c < d; c += 32) {
      const float x = key_live ? Kp[(size_t)(j0 + q) * d + c] : 0.f;
      ks[(warp * KW + q) * d + c] = x;
      vs[(warp * KW + q) * d + c] = key_live ? Vp[(size_t)(j0 + q) * d + c] : 0.f;
      hs = fmaf(x, x, hs);
    }
#pragma unroll
    for (int o = 16; o > 0; o >>= 1) hs += __shfl_xor_sync(0xffffffffu, hs, o);
    half_sq[q] = 0.5f * hs;
  }
  float dk[KW][4], dv[KW][4], dl_sum[KW];
#pragma unroll
  for (int q = 0; q < KW; ++q) {
    dl_sum[q] = 0.f;
#pragma unroll
    for (int b = 0; b < 4; ++b) dk[q][b] = dv[q][b] = 0.f;
  }
  for (int i0 = 0; i0 < p; i0 += 32) {
    __syncthreads();
    for (int idx = threadIdx.x; idx < 32 * d; idx += 256) {
      const int ii = idx / d, c = idx % d;
      const bool in = i0 + ii < p;
      const size_t g = ((size_t)bh * p + i0 + ii) * d + c;
      if (kPerformer) Ws[ii * (d + 1) + c] = in ? to_f32(W[(size_t)(i0 + ii) * d + c]) : 0.f;
      As[ii * (d + 1) + c] = in ? a32[g] : 0.f;
      Ds[ii * (d + 1) + c] = in ? da[g] : 0.f;
    }
    if (threadIdx.x < 32) {
      const bool in = i0 + threadIdx.x < p;
      bs[threadIdx.x] = in ? weight[(size_t)bh * p + i0 + threadIdx.x] : 0.f;
      dbs[threadIdx.x] = in ? db[(size_t)bh * p + i0 + threadIdx.x] : 0.f;
    }
    __syncthreads();
    const bool feat_live = (i0 + lane) < p;
    // A_ij and g_ij for feature i = i0 + lane and the warp's four keys
    float e1[KW], wk[KW];
#pragma unroll
    for (int q = 0; q < KW; ++q) e1[q] = wk[q] = 0.f;
    for (int c = 0; c < d; ++c) {
      const float dsv = Ds[lane * (d + 1) + c], asv = As[lane * (d + 1) + c];
      const float wsv = kPerformer ? Ws[lane * (d + 1) + c] : 0.f;
#pragma unroll
      for (int q = 0; q < KW; ++q) {
        e1[q] = fmaf(dsv, vs[(warp * KW + q) * d + c] - asv, e1[q]);
        if (kPerformer) wk[q] = fmaf(wsv, ks[(warp * KW + q) * d + c], wk[q]);
      }
    }
#pragma unroll
    for (int q = 0; q < KW; ++q) {
      const bool live = feat_live && (j0 + q < k);
      float A = 0.f, g = 0.f;
      if (live) {
        g = e1[q] + dbs[lane];
        if (kPerformer) A = expf(wk[q] - half_sq[q] - bs[lane]);     // b_i = log sum_j exp(L_ji): A <= 1
        else A = elu1(ks[(warp * KW + q) * d + i0 + lane]) / bs[lane];      // weight holds z_i for RNN
      }
      const float dL = A * g;
      dl_sum[q] += dL;
      if (!kPerformer && live) {
        const float x = ks[(warp * KW + q) * d + i0 + lane];
        dKpVp[((size_t)bh * k + j0 + q) * d + i0 + lane] = dL * elu1_slope(x) / elu1(x);
      }
      sA[warp][lane][q] = A;
      sdL[warp][lane][q] = dL;
    }
    __syncwarp();
    for (int ii = 0; ii < 32; ++ii) {
      const float4 A4 = *reinterpret_cast<const float4*>(&sA[warp][ii][0]);
      const float4 L4 = *reinterpret_cast<const float4*>(&sdL[warp][ii][0]);
      const float Aq[KW] = {A4.x, A4.y, A4.z, A4.w}, Lq[KW] = {L4.x, L4.y, L4.z, L4.w};
#pragma unroll
      for (int b = 0; b < 4; ++b) {
        const int c = lane + 32 * b;
        if (c < d) {
          const float dsv = Ds[ii * (d + 1) + c];
          const float wsv = kPerformer ? Ws[ii * (d + 1) + c] : 0.f;
#pragma unroll
          for (int q = 0; q < KW; ++q) {
            dv[q][b] = fmaf(Aq[q], dsv, dv[q][b]);
            if (kPerformer) dk[q][b] = fmaf(Lq[q], wsv, dk[q][b]);
          }
        }
      }
    }
    __syncwarp();
  }
#pragma unroll
  for (int q = 0; q < KW; ++q) {
    if (j0 + q >= k) continue;
    float ds = dl_sum[q];
#pragma unroll
    for (int o = 16; o > 0; o >>= 1) ds += __shfl_xor_sync(0xffffffffu, ds, o);
#pragma unroll
    for (int b = 0; b < 4; ++b) {
      const int c = lane + 32 * b;
      if (c < d) {
        if (kPerformer) dKpVp[((size_t)bh * k + j0 + q) * d + c] = dk[q][b] - ks[(warp * KW + q) * d + c] * ds;
        dKpVp[(((size_t)BH + bh) * k + j0 + q) * d + c] = dv[q][b];
      }
    }
  }
}

// ---------------------------------------------------------------------------------------------
// dK = E^T dK', dV = F^T dV'.  grid = (ceil(N/32), B*H, 2); block = 256: warp w owns positions
// 4w..4w+3 of the tile, lane owns columns lane + 32 b.  E, F: [k][N] (or [H][k][N], ef_heads = H).
// ---------------------------------------------------------------------------------------------
template <typename T>
__global__ void __launch_bounds__(256)
simt_bwd_inputs(const T* __restrict__ E, const T* __restrict__ F, const float* __restrict__ dKpVp,
                T* __restrict__ dK, T* __restrict__ dV, int BH, int N, int d, int k, int seq_major_heads,
                int ef_heads) {
  __shared__ float Ps[32][33];     // [j][n]
  __shared__ float Gs[32][128];    // [j][c]
  const int t = blockIdx.z, bh = blockIdx.y, n0 = blockIdx.x * 32;
  const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
  const T* __restrict__ P = (t ? F : E) + (ef_heads > 0 ? (size_t)(bh % ef_heads) * k * N : 0);
  const float* __restrict__ G = dKpVp + ((size_t)t * BH + bh) * (size_t)k * d;
  const HeadView hv = head_view(bh, seq_major_heads, N, d);
  T* __restrict__ out = (t ? dV : dK) + hv.base;
  float acc[4][4];
#pragma unroll
  for (int r = 0; r < 4; ++r)
#pragma unroll
    for (int b = 0; b < 4; ++b) acc[r][b] = 0.f;
  for (int j0 = 0; j0 < k; j0 += 32) {
    __syncthreads();
    for (int idx = threadIdx.x; idx < 32 * 32; idx += 256) {
      const int jj = idx >> 5, nn = idx & 31;
      Ps[jj][nn] = (j0 + jj < k && n0 + nn < N) ? to_f32(P[(size_t)(j0 + jj) * N + n0 + nn]) : 0.f;
    }
    for (int idx = threadIdx.x; idx < 32 * 128; idx += 256) {
      const int jj = idx >> 7, c = idx & 127;
      Gs[jj][c] = (j0 + jj < k && c < d) ? G[(size_t)(j0 + jj) * d + c] : 0.f;
    }
    __syncthreads();
    for (int jj = 0; jj < 32; ++jj) {
#pragma unroll
      for (int r = 0; r < 4; ++r) {
        const float e = Ps[jj][warp * 4 + r];
#pragma unroll
        for (int b = 0; b < 4; ++b) acc[r][b] = fmaf(e, Gs[jj][lane + 32 * b], acc[r][b]);
      }
    }
  }
#pragma unroll
  for (int r = 0; r < 4; ++r) {
    const int n = n0 + warp * 4 + r;
    if (n >= N) continue;
#pragma unroll
    for (int b = 0; b < 4; ++b) {
      const int c = lane + 32 * b;
      if (c < d) store_out(out + (size_t)n * hv.row_stride + c, acc[r][b]);
    }
  }
}

// ---------------------------------------------------------------------------------------------
// dE = sum over heads of dK' K^T, dF = sum over heads of dV' V^T.  grid = (ceil(N/32), ceil(k/32),
// 2 * max(ef_heads, 1)); block = 256 (a 32 x 32 tile of dE, four rows per thread).  With shared E, F
// the sum runs over all B*H heads; with one pair per head over the batch only.
// ---------------------------------------------------------------------------------------------
template <typename T>
__global__ void __launch_bounds__(256)
simt_bwd_projections(const T* __restrict__ Kin, const T* __restrict__ Vin, const float* __restrict__ dKpVp,
                     T* __restrict__ dE, T* __restrict__ dF, int BH, int N, int d, int k, int seq_major_heads,
                     int ef_heads) {
  __shared__ float Gs[32][129];    // [j][c]
  __shared__ float Xs[32][129];    // [n][c]
  const int groups = ef_heads > 0 ? ef_heads : 1;
  const int t = blockIdx.z / groups, eh = blockIdx.z % groups;
  const int n0 = blockIdx.x * 32, j0 = blockIdx.y * 32;
  const int tx = threadIdx.x & 31, ty = threadIdx.x >> 5;
  float acc[4] = {0.f, 0.f, 0.f, 0.f};
  for (int bh = eh; bh < BH; bh += groups) {
    const float* __restrict__ G = dKpVp + ((size_t)t * BH + bh) * (size_t)k * d;
    const HeadView hv = head_view(bh, seq_major_heads, N, d);
    const T* __restrict__ X = (t ? Vin : Kin) + hv.base;
    __syncthreads();
    for (int idx = threadIdx.x; idx < 32 * 128; idx += 256) {
      const int rr = idx >> 7, c = idx & 127;
      Gs[rr][c] = (j0 + rr < k && c < d) ? G[(size_t)(j0 + rr) * d + c] : 0.f;
      Xs[rr][c] = (n0 + rr < N && c < d) ? to_f32(X[(size_t)(n0 + rr) * hv.row_stride + c]) : 0.f;
    }
    __syncthreads();
    for (int c = 0; c < d; ++c) {
      const float x = Xs[tx][c];
#pragma unroll
      for (int r = 0; r < 4; ++r) acc[r] = fmaf(Gs[ty + 8 * r][c], x, acc[r]);
    }
  }
  T* __restrict__ out = (t ? dF : dE) + (size_t)eh * k * N;
#pragma unroll
  for (int r = 0; r < 4; ++r) {
    const int j = j0 + ty + 8 * r;
    if (j < k && n0 + tx < N) store_out(out + (size_t)j * N + n0 + tx, acc[r]);
  }
}

}  // namespace flurka

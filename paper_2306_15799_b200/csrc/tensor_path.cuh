// Host side of the tensor-core (tcgen05 / TMEM / TMA) kernels: tensor-map encoding and launches.
#pragma once

#include <cuda.h>
#include <cuda_fp16.h>
#include <cuda_runtime.h>
#include <string.h>

#include "k0_linear_maps.cuh"
#include "k1_down_project.cuh"
#include "k1_down_project_pair.cuh"
#include "k2_key_side.cuh"
#include "k3_query_side.cuh"
#include "k4_bwd_query_side.cuh"
#include "k5_bwd_projections.cuh"
#include "k6_bwd_key_side.cuh"

namespace flurka {

// Optional per-stage timing: events recorded on the launch stream around the three stages.
struct StageTimer {
  bool on = false;
  bool have = false;
  cudaEvent_t ev[4] = {nullptr, nullptr, nullptr, nullptr};
  // creates the events on the current device on first use; returns a cudaError_t as int
  int create() {
    for (int i = 0; i < 4; ++i) {
      if (!ev[i]) {
        cudaError_t e = cudaEventCreate(&ev[i]);
        if (e != cudaSuccess) return (int)e;
      }
    }
    return 0;
  }
  void mark(int i, cudaStream_t st) {
    if (on && ev[i]) cudaEventRecord(ev[i], st);
  }
};

// ---------------------------------------------------------------------------------------------
// cuTensorMapEncodeTiled is fetched from the driver at run time, so the library links against
// the CUDA runtime only and still loads on machines without a driver.
// ---------------------------------------------------------------------------------------------
typedef CUresult (*EncodeTiledFn)(CUtensorMap*, CUtensorMapDataType, cuuint32_t, void*, const cuuint64_t*,
                                  const cuuint64_t*, const cuuint32_t*, const cuuint32_t*, CUtensorMapInterleave,
                                  CUtensorMapSwizzle, CUtensorMapL2promotion, CUtensorMapFloatOOBfill);

inline EncodeTiledFn encode_tiled_fn() {
  static EncodeTiledFn fn = nullptr;
  if (!fn) {
    void* ptr = nullptr;
    cudaDriverEntryPointQueryResult qres;
    if (cudaGetDriverEntryPoint("cuTensorMapEncodeTiled", &ptr, cudaEnableDefault, &qres) != cudaSuccess ||
        qres != cudaDriverEntryPointSuccess) {
      (void)cudaGetLastError();
      return nullptr;
    }
    fn = reinterpret_cast<EncodeTiledFn>(ptr);
  }
  return fn;
}

// A tensor map together with the arguments it was built from (re-encoded only when they change).
struct CachedMap {
  CUtensorMap map;
  const void* ptr = nullptr;
  unsigned long long key[8] = {0, 0, 0, 0, 0, 0, 0, 0};
  bool valid = false;
};

// rank <= 3; dims/box in elements (innermost first); 128-byte swizzle; out-of-range reads give zero.
inline bool encode_map(CachedMap* cm, CUtensorMapDataType dt, int esize, int rank, const void* ptr,
                       const unsigned long long* dims, const unsigned* box) {
  unsigned long long key[8] = {(unsigned long long)dt, (unsigned long long)rank, dims[0], dims[1],
                               rank > 2 ? dims[2] : 1ull, box[0], box[1], rank > 2 ? box[2] : 1u};
  if (cm->valid && cm->ptr == ptr && memcmp(key, cm->key, sizeof(key)) == 0) return true;
  EncodeTiledFn fn = encode_tiled_fn();
  if (!fn) return false;
  cuuint64_t gdim[3] = {dims[0], dims[1], rank > 2 ? dims[2] : 1};
  cuuint64_t gstride[2] = {dims[0] * (cuuint64_t)esize, dims[0] * dims[1] * (cuuint64_t)esize};
  cuuint32_t bdim[3] = {box[0], box[1], rank > 2 ? box[2] : 1};
  cuuint32_t estr[3] = {1, 1, 1};
  CUresult r = fn(&cm->map, dt, (cuuint32_t)rank, const_cast<void*>(ptr), gdim, gstride, bdim, estr,
                  CU_TENSOR_MAP_INTERLEAVE_NONE, CU_TENSOR_MAP_SWIZZLE_128B, CU_TENSOR_MAP_L2_PROMOTION_L2_256B,
                  CU_TENSOR_MAP_FLOAT_OOB_FILL_NONE);
  if (r != CUDA_SUCCESS) { cm->valid = false; return false; }
  cm->ptr = ptr;
  memcpy(cm->key, key, sizeof(key));
  cm->valid = true;
  return true;
}

struct TensorMaps {
  CachedMap E, F, K, V, kpvp, Q, W, W2, aT, O;
  CachedMap dO, abf;                            // backward of the query side
  CachedMap bE, bF, bK, bV, split64, split128, gK, gV, gE, gF;   // backward of the down-projection
  CachedMap A3, Wk, Wv, Xq, Wq, Qp, kpvp2;      // the linear maps of the entry point with un-projected inputs
};

// Per-device context of the tensor-core kernels: the cached tensor maps (their pointers are device
// addresses), the SM count, and whether the kernels' shared-memory limits have been raised there.
struct TensorContext {
  TensorMaps maps;
  int sms = 0;
  bool k1_attr = false;
  bool k1p_attr = false;
  bool k0_attr = false;
  bool k0p_attr = false;
  bool k5_attr = false;
  int sm_total() {
    if (!sms) {
      int dev = 0;
      cudaGetDevice(&dev);
      cudaDeviceGetAttribute(&sms, cudaDevAttrMultiProcessorCount, dev);
      if (sms <= 0) sms = 148;
    }
    return sms;
  }
  // SMs the persistent kernels may use (the test knob caps it)
  int sm_count();
};

// whether stage 1 may run as pairs of CTAs (tcgen05.mma.cta_group::2) where the shape allows
inline int& stage1_pairs() {
  static int on = 1;
  return on;
}

// 0 = use every SM; otherwise the persistent kernels are launched with at most this many CTAs
inline int& cta_limit() {
  static int limit = 0;
  return limit;
}

inline int TensorContext::sm_count() {
  const int n = sm_total();
  const int lim = cta_limit();
  return (lim > 0 && lim < n) ? lim : n;
}

// Sequence splits of stage 1: as few as fill the machine once.  Every split adds a full copy of
// the output to the fp32 reduction (measured: the reduce-add traffic of all CTAs drains at about
// 2.5 TB/s after the last MMA, so more, shorter CTAs lose more in that tail than they gain).
inline int k1_choose_nsplit(int sms, int units, int chunks) {
  int ns = sms / units;
  if (ns < 1) ns = 1;
  if (ns > chunks) ns = chunks;
  return ns;
}

// ---- stage 1: K' = E K, V' = F V into kpvp (already zeroed) ----------------------------------
// H > 0: K, V are [B,N,H,d] (H heads merged into the row); H == 0: [B,H,N,d]
// ef_heads > 0: E, F are [ef_heads][k][N] (one pair per head; head index = bh % ef_heads)
inline int launch_k1(TensorContext& tc, const void* K, const void* V, const void* E, const void* F, float* kpvp,
                     int BH, int H, int N, int d, int k, int* status, cudaStream_t st, int* cuda_err,
                     int ef_heads = 0) {
  TensorMaps& tm = tc.maps;
  const unsigned long long dE[3] = {(unsigned long long)N, (unsigned long long)k,
                                    (unsigned long long)(ef_heads > 0 ? ef_heads : 1)};
  const unsigned bE[3] = {64, 128, 1};
  // [B,N,H,d] is a 3-D tensor too: rows of H*d elements, head h at columns h*d .. h*d+d-1
  const unsigned long long dX[3] = {(unsigned long long)(H > 0 ? H * d : d), (unsigned long long)N,
                                    (unsigned long long)(H > 0 ? BH / H : BH)};
  const unsigned bX[3] = {64, 64, 1};
  const unsigned long long dO[3] = {(unsigned long long)d, (unsigned long long)k, (unsigned long long)2 * BH};
  const unsigned bO[3] = {32, 32, 1};
  if (!encode_map(&tm.E, CU_TENSOR_MAP_DATA_TYPE_BFLOAT16, 2, 3, E, dE, bE) ||
      !encode_map(&tm.F, CU_TENSOR_MAP_DATA_TYPE_BFLOAT16, 2, 3, F, dE, bE) ||
      !encode_map(&tm.K, CU_TENSOR_MAP_DATA_TYPE_BFLOAT16, 2, 3, K, dX, bX) ||
      !encode_map(&tm.V, CU_TENSOR_MAP_DATA_TYPE_BFLOAT16, 2, 3, V, dX, bX) ||
      !encode_map(&tm.kpvp, CU_TENSOR_MAP_DATA_TYPE_FLOAT32, 4, 3, kpvp, dO, bO)) {
    *cuda_err = (int)cudaErrorInvalidValue;
    return -6;
  }
  if (stage1_pairs() && ef_heads == 0 && k % 256 == 0 && (BH * d) % 256 == 0) {
    // two CTAs per output tile: 256 projection rows x 512 columns per pair
    K1PairParams pp;
    pp.N = N; pp.d = d; pp.k = k; pp.BH = BH; pp.H = H;
    pp.col_groups = (BH * d + 511) / 512;
    pp.k_halves = k / 256;
    pp.nsplit = k1_choose_nsplit(tc.sm_count() / 2, 2 * pp.col_groups * pp.k_halves, (N + 63) / 64);
    pp.status = status;
    if (!tc.k1p_attr) {
      cudaError_t e = cudaFuncSetAttribute(k1_down_project_pair, cudaFuncAttributeMaxDynamicSharedMemorySize, kK1PSmemBytes);
      if (e != cudaSuccess) { *cuda_err = (int)e; (void)cudaGetLastError(); return -6; }
      tc.k1p_attr = true;
    }
    const int pairs = 2 * pp.k_halves * pp.col_groups * pp.nsplit;
    k1_down_project_pair<<<2 * pairs, kK1PThreads, kK1PSmemBytes, st>>>(tm.E.map, tm.F.map, tm.K.map, tm.V.map,
                                                                        tm.kpvp.map, pp);
    cudaError_t e = cudaGetLastError();
    if (e != cudaSuccess) { *cuda_err = (int)e; return -6; }
    return 0;
  }
  K1Params p;
  p.N = N; p.d = d; p.k = k; p.BH = BH; p.H = H;
  p.ef_heads = ef_heads;
  p.group_cols = ef_heads > 0 ? d : 256;
  p.col_groups = (BH * d + p.group_cols - 1) / p.group_cols;
  p.k_halves = (k + 255) / 256;
  p.nsplit = k1_choose_nsplit(tc.sm_count(), 2 * p.col_groups * p.k_halves, (N + 63) / 64);
  p.status = status;
  if (!tc.k1_attr) {
    cudaError_t e = cudaFuncSetAttribute(k1_down_project, cudaFuncAttributeMaxDynamicSharedMemorySize, kK1SmemBytes);
    if (e != cudaSuccess) { *cuda_err = (int)e; (void)cudaGetLastError(); return -6; }
    tc.k1_attr = true;
  }
  const int grid = 2 * p.k_halves * p.col_groups * p.nsplit;
  k1_down_project<<<grid, kK1Threads, kK1SmemBytes, st>>>(tm.E.map, tm.F.map, tm.K.map, tm.V.map, tm.kpvp.map, p);
  cudaError_t e = cudaGetLastError();
  if (e != cudaSuccess) { *cuda_err = (int)e; return -6; }
  return 0;
}

// Forward declaration (defined below).
template <typename... KArgs, typename... Args>
inline cudaError_t launch_after_predecessor(void (*fn)(KArgs...), int grid, int block, size_t smem, cudaStream_t st,
                                            Args... args);

inline int k0_set_attr(TensorContext& tc, int* cuda_err) {
  if (!tc.k0_attr) {
    cudaError_t e = cudaFuncSetAttribute(k0_linear_map, cudaFuncAttributeMaxDynamicSharedMemorySize, kK0SmemBytes);
    if (e != cudaSuccess) { *cuda_err = (int)e; (void)cudaGetLastError(); return -6; }
    tc.k0_attr = true;
  }
  return 0;
}

// ---- the linear maps on the k contracted rows: K', V' (fp32, [2][B*H][k][d], already zeroed) from
//      kt = stage 1's output for the un-projected inputs ([2][B][dm/64][k][64] fp32)
inline int launch_k0_key_value_maps(TensorContext& tc, const float* kt, __nv_bfloat16* a3, const void* Wk,
                                    const void* Wv, float* kpvp, int B, int H, int dm, int d, int k, int* status,
                                    cudaStream_t st, int* cuda_err) {
  TensorMaps& tm = tc.maps;
  {
    const long long total = (long long)2 * B * k * (dm >> 2);
    int grid = (int)((total + 255) / 256);
    if (grid > tc.sm_total() * 8) grid = tc.sm_total() * 8;
    cudaError_t e = launch_after_predecessor(k0_split_rows, grid, 256, 0, st, kt, a3, 2 * B, k, dm);
    if (e != cudaSuccess) { *cuda_err = (int)e; (void)cudaGetLastError(); return -6; }
  }
  const unsigned long long dA[3] = {(unsigned long long)3 * dm, (unsigned long long)k, (unsigned long long)2 * B};
  const unsigned bA[3] = {64, 128, 1};
  const unsigned long long dB[2] = {(unsigned long long)H * d, (unsigned long long)dm};
  const unsigned bB[2] = {64, 64};
  const unsigned long long dO[3] = {(unsigned long long)d, (unsigned long long)k, (unsigned long long)2 * B * H};
  const unsigned bO[3] = {32, 32, 1};
  if (!encode_map(&tm.A3, CU_TENSOR_MAP_DATA_TYPE_BFLOAT16, 2, 3, a3, dA, bA) ||
      !encode_map(&tm.Wk, CU_TENSOR_MAP_DATA_TYPE_BFLOAT16, 2, 2, Wk, dB, bB) ||
      !encode_map(&tm.Wv, CU_TENSOR_MAP_DATA_TYPE_BFLOAT16, 2, 2, Wv, dB, bB) ||
      !encode_map(&tm.kpvp2, CU_TENSOR_MAP_DATA_TYPE_FLOAT32, 4, 3, kpvp, dO, bO)) {
    *cuda_err = (int)cudaErrorInvalidValue;
    return -6;
  }
  K0Params p;
  p.mode = 0; p.M = k; p.chunks = 3 * dm / 64; p.b_chunks = dm / 64; p.ncols = H * d; p.d = d; p.H = H;
  p.Z = 2 * B; p.zb_shift = B;
  p.row_blocks = (k + 255) / 256;
  p.col_groups = (H * d + 255) / 256;
  const int units = p.row_blocks * p.col_groups * p.Z;
  p.nsplit = k1_choose_nsplit(tc.sm_count(), units, p.chunks);
  p.status = status;
  int rc = k0_set_attr(tc, cuda_err);
  if (rc) return rc;
  cudaError_t e = launch_after_predecessor(k0_linear_map, units * p.nsplit, kK0Threads, kK0SmemBytes, st, tm.A3.map,
                                           tm.Wk.map, tm.Wv.map, tm.kpvp2.map, p);
  if (e != cudaSuccess) { *cuda_err = (int)e; (void)cudaGetLastError(); return -6; }
  return 0;
}

// ---- the query map: Qp [B*N][H*d] bf16 = Xq [B*N][dm] Wq [dm][H*d]
inline int launch_k0_query_map(TensorContext& tc, const void* Xq, const void* Wq, void* Qp, int B, int N, int H, int dm,
                               int d, int* status, cudaStream_t st, int* cuda_err) {
  TensorMaps& tm = tc.maps;
  const unsigned long long dA[3] = {(unsigned long long)dm, (unsigned long long)B * N, 1ull};
  const unsigned bA[3] = {64, 128, 1};
  const unsigned long long dB[2] = {(unsigned long long)H * d, (unsigned long long)dm};
  const unsigned bB[2] = {64, 64};
  const unsigned long long dO[2] = {(unsigned long long)H * d, (unsigned long long)B * N};
  const unsigned bO[2] = {64, 32};
  if (!encode_map(&tm.Xq, CU_TENSOR_MAP_DATA_TYPE_BFLOAT16, 2, 3, Xq, dA, bA) ||
      !encode_map(&tm.Wq, CU_TENSOR_MAP_DATA_TYPE_BFLOAT16, 2, 2, Wq, dB, bB) ||
      !encode_map(&tm.Qp, CU_TENSOR_MAP_DATA_TYPE_BFLOAT16, 2, 2, Qp, dO, bO)) {
    *cuda_err = (int)cudaErrorInvalidValue;
    return -6;
  }
  K0Params p;
  p.mode = 1; p.M = B * N; p.chunks = dm / 64; p.b_chunks = dm / 64; p.ncols = H * d; p.d = d; p.H = H;
  p.Z = 1; p.zb_shift = 1; p.nsplit = 1;
  p.row_blocks = (p.M + 255) / 256;
  p.col_groups = (H * d + 255) / 256;
  p.status = status;
  if (stage1_pairs() && (H * d) % 256 == 0) {
    // as pairs of CTAs: 256 rows x 512 columns per pair
    p.col_groups = (H * d + 511) / 512;
    if (!tc.k0p_attr) {
      cudaError_t e = cudaFuncSetAttribute(k0_query_map_pair, cudaFuncAttributeMaxDynamicSharedMemorySize, kK0PSmemBytes);
      if (e != cudaSuccess) { *cuda_err = (int)e; (void)cudaGetLastError(); return -6; }
      tc.k0p_attr = true;
    }
    k0_query_map_pair<<<2 * p.row_blocks * p.col_groups, kK0Threads, kK0PSmemBytes, st>>>(tm.Xq.map, tm.Wq.map, tm.Qp.map, p);
    cudaError_t e = cudaGetLastError();
    if (e != cudaSuccess) { *cuda_err = (int)e; return -6; }
    return 0;
  }
  int rc = k0_set_attr(tc, cuda_err);
  if (rc) return rc;
  k0_linear_map<<<p.row_blocks * p.col_groups, kK0Threads, kK0SmemBytes, st>>>(tm.Xq.map, tm.Wq.map, tm.Wq.map,
                                                                               tm.Qp.map, p);
  cudaError_t e = cudaGetLastError();
  if (e != cudaSuccess) { *cuda_err = (int)e; return -6; }
  return 0;
}

// Launch with programmatic stream serialisation: the kernel may be scheduled while the previous
// kernel in the stream is finishing (its CTAs call griddepcontrol.launch_dependents late in their
// life) and waits in griddepcontrol.wait before it touches that kernel's results.
template <typename... KArgs, typename... Args>
inline cudaError_t launch_after_predecessor(void (*fn)(KArgs...), int grid, int block, size_t smem, cudaStream_t st,
                                            Args... args) {
  cudaLaunchConfig_t cfg = {};
  cfg.gridDim = dim3((unsigned)grid, 1, 1);
  cfg.blockDim = dim3((unsigned)block, 1, 1);
  cfg.dynamicSmemBytes = smem;
  cfg.stream = st;
  cudaLaunchAttribute attr[1];
  attr[0].id = cudaLaunchAttributeProgrammaticStreamSerialization;
  attr[0].val.programmaticStreamSerializationAllowed = 1;
  cfg.attrs = attr;
  cfg.numAttrs = 1;
  return cudaLaunchKernelEx(&cfg, fn, KArgs(args)...);
}

// Key splits of stage 2: with few (head, feature tile) pairs the keys are divided over up to four
// CTAs per pair, as long as all of them fit on the machine at once.
inline int k2_nsplit(int sms, bool performer, int BH, int k, int p) {
  if (!performer) return 1;
  const int units = BH * ((p + 127) / 128);
  const int chunks = (k + kK2Chunk - 1) / kK2Chunk;
  int ns = sms / units;
  if (ns > chunks) ns = chunks;
  if (ns > 4) ns = 4;
  return ns < 1 ? 1 : ns;
}

// scratch floats for the partial results of a split stage 2, sized for the largest split the
// problem could get on any device (so the workspace size does not depend on the device)
inline size_t k2_part_floats(bool performer, int BH, int d, int k, int p) {
  if (!performer) return 0;
  int chunks = (k + kK2Chunk - 1) / kK2Chunk;
  if (chunks > 4) chunks = 4;
  if (chunks < 2) return 0;
  return (size_t)BH * ((p + 127) / 128) * chunks * (size_t)(d + 2) * 128;
}

// ---- stage 2: per-feature summaries a (fp16, transposed) and weights b / z from K', V' --------
inline int launch_k2(TensorContext& tc, bool performer, const float* kpvp, const void* W, float* weight,
                     __half* aT16, float* part, int* counters, int BH, int d, int k, int p, int* status,
                     cudaStream_t st, int* cuda_err, float* a32 = nullptr) {
  TensorMaps& tm = tc.maps;
  if (performer) {
    const unsigned long long dW[2] = {(unsigned long long)d, (unsigned long long)p};
    const unsigned bW[2] = {64, 128};
    if (!encode_map(&tm.W2, CU_TENSOR_MAP_DATA_TYPE_BFLOAT16, 2, 2, W, dW, bW)) {
      *cuda_err = (int)cudaErrorInvalidValue;
      return -6;
    }
  }
  K2Params prm;
  prm.d = d; prm.k = k; prm.p = p; prm.BH = BH;
  prm.ftiles = (p + 127) / 128;
  prm.kpvp = kpvp;
  prm.weight = weight;
  prm.aT16 = aT16;
  prm.a32 = a32;
  prm.status = status;
  prm.nsplit = (part && counters) ? k2_nsplit(tc.sm_total(), performer, BH, k, p) : 1;
  prm.part = part;
  prm.counters = counters;
  auto fn = performer ? k2_key_side<true> : k2_key_side<false>;
  cudaError_t e = cudaFuncSetAttribute(fn, cudaFuncAttributeMaxDynamicSharedMemorySize, kK2SmemBytes);
  if (e != cudaSuccess) { *cuda_err = (int)e; (void)cudaGetLastError(); return -6; }
  // the RNN kernel ignores tmW; pass any valid map
  e = launch_after_predecessor(fn, BH * prm.ftiles * prm.nsplit, kK2Threads, kK2SmemBytes, st,
                               performer ? tm.W2.map : tm.kpvp.map, prm);
  if (e != cudaSuccess) { *cuda_err = (int)e; (void)cudaGetLastError(); return -6; }
  e = cudaGetLastError();
  if (e != cudaSuccess) { *cuda_err = (int)e; return -6; }
  return 0;
}

// ---- stage 3: O from Q, W and the key-side summaries ------------------------------------------
inline int launch_k3(TensorContext& tc, bool performer, const void* Q, const void* W, const __half* aT16,
                     const float* weight, void* out, int BH, int H, int N, int d, int p, int* status, cudaStream_t st,
                     int* cuda_err) {
  TensorMaps& tm = tc.maps;
  const unsigned long long dQ[3] = {(unsigned long long)(H > 0 ? H * d : d), (unsigned long long)N,
                                    (unsigned long long)(H > 0 ? BH / H : BH)};
  const unsigned bQ[3] = {64, 128, 1};
  const unsigned long long dA[3] = {(unsigned long long)p, (unsigned long long)d, (unsigned long long)BH};
  const unsigned bA[3] = {64, (unsigned)d, 1};
  const unsigned bO[3] = {64, 32, 1};                 // d = 64: one row-owner warp's slab of the output
  if (d == 64 && !encode_map(&tm.O, CU_TENSOR_MAP_DATA_TYPE_BFLOAT16, 2, 3, out, dQ, bO)) {
    *cuda_err = (int)cudaErrorInvalidValue;
    return -6;
  }
  if (!encode_map(&tm.Q, CU_TENSOR_MAP_DATA_TYPE_BFLOAT16, 2, 3, Q, dQ, bQ) ||
      !encode_map(&tm.aT, CU_TENSOR_MAP_DATA_TYPE_FLOAT16, 2, 3, aT16, dA, bA)) {
    *cuda_err = (int)cudaErrorInvalidValue;
    return -6;
  }
  if (performer) {
    const unsigned long long dW[2] = {(unsigned long long)d, (unsigned long long)p};
    const unsigned bW[2] = {64, (unsigned)p};
    if (!encode_map(&tm.W, CU_TENSOR_MAP_DATA_TYPE_BFLOAT16, 2, 2, W, dW, bW)) {
      *cuda_err = (int)cudaErrorInvalidValue;
      return -6;
    }
  }
  K3Params prm;
  prm.N = N; prm.d = d; prm.p = p; prm.BH = BH; prm.H = H;
  prm.tiles_per_head = (N + 127) / 128;
  prm.total_tiles = prm.tiles_per_head * BH;
  prm.weight = weight;
  prm.out = reinterpret_cast<__nv_bfloat16*>(out);
  prm.status = status;
  const K3Smem L = k3_smem_plan(d, p, performer);
  auto fn = performer ? k3_query_side<true> : k3_query_side<false>;
  cudaError_t e = cudaFuncSetAttribute(fn, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)L.total);
  if (e != cudaSuccess) { *cuda_err = (int)e; (void)cudaGetLastError(); return -6; }
  int grid = tc.sm_count();
  if (grid > prm.total_tiles) grid = prm.total_tiles;
  // the RNN kernel ignores tmW and only d = 64 stores through tmO; pass any valid map otherwise
  e = launch_after_predecessor(fn, grid, kK3Threads, L.total, st, tm.Q.map, performer ? tm.W.map : tm.Q.map,
                               tm.aT.map, d == 64 ? tm.O.map : tm.Q.map, prm);
  if (e != cudaSuccess) { *cuda_err = (int)e; (void)cudaGetLastError(); return -6; }
  e = cudaGetLastError();
  if (e != cudaSuccess) { *cuda_err = (int)e; return -6; }
  return 0;
}

// ---- backward of the query side (PERFORMER, d = 64, p = 64, 128, 192 or 256): dQ, and da, db added to --
// abf: scratch for the two bf16 terms of a, [BH][2][p][64]
inline int launch_k4(TensorContext& tc, bool performer, const void* Q, const void* dO, const void* W, const float* a32,
                     const float* weight, __nv_bfloat16* abf, void* dQ, float* da, float* db, int BH, int H, int N,
                     int d, int p, int* status, cudaStream_t st, int* cuda_err, void* rowstat = nullptr) {
  // rowstat: d = 128 only, 8 bytes per query row of every 128-row tile (BH * ceil(N / 128) * 128 rows)
  TensorMaps& tm = tc.maps;
  const bool stream = d == 128;      // W and a come in per step of 128 features (boxes of 128 rows)
  const unsigned long long dQd[3] = {(unsigned long long)(H > 0 ? H * d : d), (unsigned long long)N,
                                     (unsigned long long)(H > 0 ? BH / H : BH)};
  const unsigned bQ[3] = {64, 128, 1};
  const unsigned long long dW[2] = {(unsigned long long)d, (unsigned long long)p};
  const unsigned prows = stream ? 128u : (unsigned)((p + 127) / 128) * 128;   // whole 128-feature tiles; rows past p read as zero
  const unsigned bW[2] = {64, prows};
  const unsigned long long dA[3] = {(unsigned long long)d, (unsigned long long)p, (unsigned long long)BH * 2};
  const unsigned bA[3] = {64, prows, 1};
  if (!encode_map(&tm.Q, CU_TENSOR_MAP_DATA_TYPE_BFLOAT16, 2, 3, Q, dQd, bQ) ||
      !encode_map(&tm.dO, CU_TENSOR_MAP_DATA_TYPE_BFLOAT16, 2, 3, dO, dQd, bQ) ||
      (performer && !encode_map(&tm.W, CU_TENSOR_MAP_DATA_TYPE_BFLOAT16, 2, 2, W, dW, bW)) ||
      !encode_map(&tm.abf, CU_TENSOR_MAP_DATA_TYPE_BFLOAT16, 2, 3, abf, dA, bA)) {
    *cuda_err = (int)cudaErrorInvalidValue;
    return -6;
  }
  {
    const long long total = (long long)BH * p * d;
    int grid = (int)((total + 255) / 256);
    if (grid > 148 * 8) grid = 148 * 8;
    k4_split_a<<<grid, 256, 0, st>>>(a32, abf, BH, p, d);
  }
  K4Params prm;
  prm.N = N; prm.p = p; prm.BH = BH; prm.H = H; prm.d = d;
  prm.tiles_per_head = (N + 127) / 128;
  prm.total_tiles = prm.tiles_per_head * BH;
  prm.weight = weight; prm.a32 = a32;
  prm.dQ = reinterpret_cast<__nv_bfloat16*>(dQ);
  prm.da = da; prm.db = db; prm.status = status;
  prm.rowstat = reinterpret_cast<float2*>(rowstat);
  auto fn = stream ? k4_bwd_query_side<true, true> : (performer ? k4_bwd_query_side<true, false> : k4_bwd_query_side<false, false>);
  cudaError_t e = cudaFuncSetAttribute(fn, cudaFuncAttributeMaxDynamicSharedMemorySize, kK4SmemBytes);
  if (e != cudaSuccess) { *cuda_err = (int)e; (void)cudaGetLastError(); return -6; }
  int grid = tc.sm_count();
  if (grid > prm.total_tiles) grid = prm.total_tiles;
  // the RNN kernel ignores tmW; pass any valid map
  fn<<<grid, kK4Threads, kK4SmemBytes, st>>>(tm.Q.map, tm.dO.map, performer ? tm.W.map : tm.Q.map, tm.abf.map, prm);
  e = cudaGetLastError();
  if (e != cudaSuccess) { *cuda_err = (int)e; return -6; }
  return 0;
}

// ---- backward of the down-projection: dK, dV, dE, dF from the fp32 dK', dV' (shared E, F) -------------
// split: scratch for the two bf16 terms of dK', dV', [2][k][2][BH][d]
inline int launch_k5(TensorContext& tc, const void* E, const void* F, const void* K, const void* V, const float* dkpvp,
                     __nv_bfloat16* split, void* dK, void* dV, void* dE, void* dF, int BH, int H, int N, int d, int k,
                     int* status, cudaStream_t st, int* cuda_err) {
  TensorMaps& tm = tc.maps;
  const unsigned long long hd = (unsigned long long)BH * d;
  const unsigned long long dEF[2] = {(unsigned long long)N, (unsigned long long)k};
  const unsigned bEF[2] = {64, 64}, bGE[2] = {64, 32};
  const unsigned long long dKV[3] = {(unsigned long long)(H > 0 ? H * d : d), (unsigned long long)N,
                                     (unsigned long long)(H > 0 ? BH / H : BH)};
  const unsigned bKV[3] = {64, 256, 1}, bGK[3] = {64, 32, 1};
  const unsigned long long dS[3] = {2 * hd, (unsigned long long)k, 2};
  const unsigned bS64[3] = {64, 64, 1}, bS128[3] = {64, 128, 1};
  const CUtensorMapDataType bf = CU_TENSOR_MAP_DATA_TYPE_BFLOAT16;
  if (!encode_map(&tm.bE, bf, 2, 2, E, dEF, bEF) || !encode_map(&tm.bF, bf, 2, 2, F, dEF, bEF) ||
      !encode_map(&tm.bK, bf, 2, 3, K, dKV, bKV) || !encode_map(&tm.bV, bf, 2, 3, V, dKV, bKV) ||
      !encode_map(&tm.split64, bf, 2, 3, split, dS, bS64) || !encode_map(&tm.split128, bf, 2, 3, split, dS, bS128) ||
      !encode_map(&tm.gK, bf, 2, 3, dK, dKV, bGK) || !encode_map(&tm.gV, bf, 2, 3, dV, dKV, bGK) ||
      !encode_map(&tm.gE, bf, 2, 2, dE, dEF, bGE) || !encode_map(&tm.gF, bf, 2, 2, dF, dEF, bGE)) {
    *cuda_err = (int)cudaErrorInvalidValue;
    return -6;
  }
  if (!tc.k5_attr) {
    cudaError_t e = cudaFuncSetAttribute(k5_bwd_projections<0>, cudaFuncAttributeMaxDynamicSharedMemorySize,
                                         K5Shape<0>::kSmemBytes);
    if (e == cudaSuccess)
      e = cudaFuncSetAttribute(k5_bwd_projections<1>, cudaFuncAttributeMaxDynamicSharedMemorySize, K5Shape<1>::kSmemBytes);
    if (e == cudaSuccess)
      e = cudaFuncSetAttribute(k5_bwd_projections<2>, cudaFuncAttributeMaxDynamicSharedMemorySize, K5Shape<2>::kSmemBytes);
    if (e != cudaSuccess) { *cuda_err = (int)e; (void)cudaGetLastError(); return -6; }
    tc.k5_attr = true;
  }
  {
    const long long total = (long long)2 * BH * k * (d / 4);
    int grid = (int)((total + 255) / 256);
    if (grid > 148 * 8) grid = 148 * 8;
    k5_split_rows<<<grid, 256, 0, st>>>(dkpvp, split, BH, k, d);
  }
  K5Params p;
  p.N = N; p.k = k; p.d = d; p.BH = BH; p.H = H; p.status = status;
  p.row_blocks = (N + K5Shape<0>::kRows - 1) / K5Shape<0>::kRows;
  p.col_groups = (int)((hd + 255) / 256);
  k5_bwd_projections<0><<<2 * p.row_blocks * p.col_groups, kK5Threads, K5Shape<0>::kSmemBytes, st>>>(
      tm.bE.map, tm.bF.map, tm.split64.map, tm.gK.map, tm.gV.map, p);
  p.row_blocks = (k + 255) / 256;
  p.col_groups = (N + 255) / 256;
  if (2 * p.row_blocks * p.col_groups >= 100) {
    k5_bwd_projections<1><<<2 * p.row_blocks * p.col_groups, kK5Threads, K5Shape<1>::kSmemBytes, st>>>(
        tm.bK.map, tm.bV.map, tm.split128.map, tm.gE.map, tm.gF.map, p);
  } else {
    // few tiles: 128-row tiles put twice as many CTAs to work, each with four smaller stages in flight
    p.row_blocks = (k + 127) / 128;
    k5_bwd_projections<2><<<2 * p.row_blocks * p.col_groups, kK5Threads, K5Shape<2>::kSmemBytes, st>>>(
        tm.bK.map, tm.bV.map, tm.split128.map, tm.gE.map, tm.gF.map, p);
  }
  cudaError_t e = cudaGetLastError();
  if (e != cudaSuccess) { *cuda_err = (int)e; return -6; }
  return 0;
}

// ---- backward of the key side (PERFORMER, d = 64): dK', dV' from da, db ---------------------------------
inline int launch_k6(TensorContext& tc, const void* W, const float* kpvp, const float* weight, const float* a32,
                     const float* da, const float* db, float* dkpvp, int BH, int k, int p, int* status, cudaStream_t st,
                     int* cuda_err) {
  TensorMaps& tm = tc.maps;
  const unsigned long long dW[2] = {64ull, (unsigned long long)p};
  const unsigned bW[2] = {64, 128};
  if (!encode_map(&tm.W2, CU_TENSOR_MAP_DATA_TYPE_BFLOAT16, 2, 2, W, dW, bW)) {
    *cuda_err = (int)cudaErrorInvalidValue;
    return -6;
  }
  K6Params prm;
  prm.k = k; prm.p = p; prm.BH = BH;
  prm.kpvp = kpvp; prm.weight = weight; prm.a32 = a32; prm.da = da; prm.db = db; prm.dkpvp = dkpvp; prm.status = status;
  cudaError_t e = cudaFuncSetAttribute(k6_bwd_key_side, cudaFuncAttributeMaxDynamicSharedMemorySize, kK6SmemBytes);
  if (e != cudaSuccess) { *cuda_err = (int)e; (void)cudaGetLastError(); return -6; }
  k6_bwd_key_side<<<BH * ((k + 127) / 128), kK6Threads, kK6SmemBytes, st>>>(tm.W2.map, prm);
  e = cudaGetLastError();
  if (e != cudaSuccess) { *cuda_err = (int)e; return -6; }
  return 0;
}

}  // namespace flurka

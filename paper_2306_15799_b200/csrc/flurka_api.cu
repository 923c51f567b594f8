// Host side of the FLuRKA forward library: argument checks, workspace, path selection, launches.
// The C ABI is declared and documented in include/flurka.h.
#include "flurka.h"

#include <cuda_runtime.h>

#include <algorithm>
#include <stdint.h>

#include "simt_backward.cuh"
#include "simt_kernels.cuh"
#include "tensor_path.cuh"

namespace {

using namespace flurka;

struct Problem {
  int kernel;      // FLURKA_PERFORMER / FLURKA_RNN
  bool fp32;       // element type of the I/O tensors
  bool bnhd;       // Q, K, V, out are [B,N,H,d] (heads merged into the row) instead of [B,H,N,d]
  bool ef_per_head;  // E, F are [H,k,N]: one pair per head, shared over the batch
  int B, H, N, d, k, m;
  int seq_major_heads() const { return bnhd ? H : 0; }   // what head_view() takes
  int ef_heads() const { return ef_per_head ? H : 0; }
  int BH() const { return B * H; }
  int p() const { return kernel == FLURKA_PERFORMER ? m : d; }   // feature dimension
  size_t esize() const { return fp32 ? 4 : 2; }
  size_t qkv_elems() const { return (size_t)B * H * N * d; }
  size_t ef_elems() const { return (size_t)k * N * (ef_per_head ? H : 1); }
  size_t w_elems() const { return kernel == FLURKA_PERFORMER ? (size_t)m * d : 0; }
};

// Workspace layout (all offsets 256-byte aligned):
//   status  int32[4] at offset 0 whatever the problem, then one arrival counter per
//           (head, 128-feature tile) of stage 2
//   kpvp    fp32 [2][BH][k][d]     K' then V'
//           (status and kpvp are adjacent: one memset per forward clears both)
//   weight  fp32 [BH][p]           b_i (PERFORMER) or z_i (RNN)
//   a32     fp32 [BH][p][d]        key-side summary, feature-major
//   aT16    fp16 [BH][d][p]        the same, transposed, as the tensor-core B operand
//   part    fp32 partial results of a key-split stage 2 (tensor-core path only)
struct Layout {
  size_t status, status_bytes, kpvp, kpvp_end, weight, a32, aT16, part, total;
};

size_t align256(size_t x) { return (x + 255) & ~(size_t)255; }

// `with_split_scratch`: reserve room for the partial results of a key-split tensor-core stage 2
// (the SIMT path never needs it)
Layout make_layout(const Problem& pr, bool with_split_scratch = true) {
  Layout L;
  size_t off = 0;
  L.status_bytes = 16 + (with_split_scratch ? (size_t)pr.BH() * ((pr.p() + 127) / 128) * 4 : 0);
  L.status = off; off = align256(off + L.status_bytes);
  L.kpvp = off;   L.kpvp_end = off + (size_t)2 * pr.BH() * pr.k * pr.d * 4; off = align256(L.kpvp_end);
  L.weight = off; off = align256(off + (size_t)pr.BH() * pr.p() * 4);
  L.a32 = off;    off = align256(off + (size_t)pr.BH() * pr.p() * pr.d * 4);
  L.aT16 = off;   off = align256(off + (size_t)pr.BH() * pr.p() * pr.d * 2);
  const size_t part_floats = (with_split_scratch && !pr.fp32)
                                 ? k2_part_floats(pr.kernel == FLURKA_PERFORMER, pr.BH(), pr.d, pr.k, pr.p())
                                 : 0;
  L.part = off;   off = align256(off + part_floats * 4);
  L.total = off;
  return L;
}

// Everything that belongs to one GPU: scratch, staging, streams, events, tensor maps and the record
// of the last forward.  Slot = CUDA device ordinal of the device that is current at the call.
struct DeviceState {
  void* user_ws = nullptr;
  size_t user_ws_bytes = 0;
  void* own_ws = nullptr;
  size_t own_ws_bytes = 0;
  int last_path = 0;
  int last_launches = 0;
  // most recent forward (for flurka_debug_copy / flurka_last_status)
  bool have_last = false;
  bool partial_pending = false;        // the last call was the first half of a sequence-sharded forward
  Problem last_problem{};
  char* last_ws = nullptr;
  // host-buffer entry point: device staging
  void* stage = nullptr;
  size_t stage_bytes = 0;
  cudaStream_t out_stream = nullptr;   // device-to-host copies of finished head groups
  cudaEvent_t group_done[8] = {};      // one per head group of a host-buffer call
  cudaEvent_t out_done = nullptr;
  StageTimer timer;
  TensorContext tc;
};

constexpr int kMaxDevices = 64;
DeviceState g_dev[kMaxDevices];

// Process-wide settings
int g_path = FLURKA_PATH_AUTO;
bool g_stage_timing = false;
int g_last_cuda_error = 0;

// The slot of the current device (slot 0 when there is no usable device: the calls that reach
// this without one only touch host-side fields).
DeviceState& dev_state() {
  int dev = 0;
  if (cudaGetDevice(&dev) != cudaSuccess) { (void)cudaGetLastError(); dev = 0; }
  if (dev < 0 || dev >= kMaxDevices) dev = 0;
  return g_dev[dev];
}

int cuda_fail(cudaError_t e) {
  g_last_cuda_error = (int)e;
  (void)cudaGetLastError();
  return FLURKA_ERR_CUDA;
}

int parse_problem(int variant, int B, int H, int N, int d, int k, int m, Problem* pr) {
  const int kernel = variant & 0xff;
  const int io = variant & 0x100;
  const int layout = variant & 0x200;
  if (kernel != FLURKA_PERFORMER && kernel != FLURKA_RNN) return FLURKA_ERR_VARIANT;
  if (variant & ~0x7ff) return FLURKA_ERR_VARIANT;
  if (B <= 0 || H <= 0 || N <= 0 || d <= 0 || k <= 0) return FLURKA_ERR_SHAPE;
  if (d > 128 || k > 4096) return FLURKA_ERR_SHAPE;
  if (kernel == FLURKA_PERFORMER && m <= 0) return FLURKA_ERR_SHAPE;
  if ((long long)B * H > 65535) return FLURKA_ERR_SHAPE;
  pr->kernel = kernel;
  pr->fp32 = io == FLURKA_IO_FP32;
  pr->bnhd = layout == FLURKA_LAYOUT_BNHD;
  pr->ef_per_head = (variant & FLURKA_EF_PER_HEAD) != 0;
  pr->B = B; pr->H = H; pr->N = N; pr->d = d; pr->k = k;
  pr->m = kernel == FLURKA_PERFORMER ? m : 0;
  return FLURKA_OK;
}

bool overlaps(const void* a, size_t na, const void* b, size_t nb) {
  const uintptr_t x = (uintptr_t)a, y = (uintptr_t)b;
  return x < y + nb && y < x + na;
}

bool tensor_path_ok(const Problem& pr) {
  if (pr.fp32) return false;
  if (pr.d != 64 && pr.d != 128) return false;
  if (pr.N % 8) return false;       // row pitch of E, F (N elements) must be a multiple of 16 bytes for TMA
  if (pr.k % 64 || pr.k > 512) return false;
  if (pr.kernel == FLURKA_PERFORMER && (pr.m % 64 || pr.m > 256)) return false;
  return true;
}

// The library-owned workspace grows in stream order: the old block is released and the new one
// obtained on the call's stream, so nothing waits on the host and earlier work queued on that
// stream still finds its block.
int get_workspace(DeviceState& ds, size_t need, cudaStream_t st, char** ws) {
  if (ds.user_ws) {
    if (ds.user_ws_bytes < need) return FLURKA_ERR_WORKSPACE;
    *ws = (char*)ds.user_ws;
    return FLURKA_OK;
  }
  if (ds.own_ws_bytes < need) {
    if (ds.own_ws) {
      cudaError_t e = cudaFreeAsync(ds.own_ws, st);
      if (e != cudaSuccess) return cuda_fail(e);
      ds.own_ws = nullptr;
      ds.own_ws_bytes = 0;
      ds.have_last = false;
    }
    cudaError_t e = cudaMallocAsync(&ds.own_ws, need, st);
    if (e != cudaSuccess) { cuda_fail(e); ds.own_ws = nullptr; return FLURKA_ERR_WORKSPACE; }
    ds.own_ws_bytes = need;
  }
  *ws = (char*)ds.own_ws;
  return FLURKA_OK;
}

int check_device() {
  int dev = 0;
  if (cudaGetDevice(&dev) != cudaSuccess) { (void)cudaGetLastError(); return FLURKA_ERR_DEVICE; }
  if (dev < 0 || dev >= kMaxDevices) return FLURKA_ERR_DEVICE;
  int major = 0;
  if (cudaDeviceGetAttribute(&major, cudaDevAttrComputeCapabilityMajor, dev) != cudaSuccess) {
    (void)cudaGetLastError();
    return FLURKA_ERR_DEVICE;
  }
  return major == 10 ? FLURKA_OK : FLURKA_ERR_DEVICE;
}

template <typename T>
int launch_simt_down_project(const Problem& pr, const void* K, const void* V, const void* E,
                             const void* F, float* kpvp, cudaStream_t st, int* launches) {
  // enough sequence splits to fill the machine; each split is a multiple of the 32-wide tile
  const int jt = (pr.k + 31) / 32;
  int nsplit = (4 * 148 + jt * pr.BH() * 2 - 1) / (jt * pr.BH() * 2);
  const int max_split = (pr.N + 255) / 256;
  if (nsplit > max_split) nsplit = max_split;
  if (nsplit < 1) nsplit = 1;
  if (nsplit > 16384) nsplit = 16384;
  int chunk = (pr.N + nsplit - 1) / nsplit;
  chunk = (chunk + 31) / 32 * 32;
  nsplit = (pr.N + chunk - 1) / chunk;
  dim3 grid(jt, pr.BH(), 2 * nsplit);
  simt_down_project<T><<<grid, 256, 0, st>>>((const T*)K, (const T*)V, (const T*)E, (const T*)F, kpvp,
                                            pr.BH(), pr.N, pr.d, pr.k, nsplit, chunk, pr.seq_major_heads(),
                                            pr.ef_heads());
  ++*launches;
  return FLURKA_OK;
}

template <typename T, bool P>
int launch_simt_key_side(const Problem& pr, const float* kpvp, const void* W, float* weight, float* a32,
                         __half* aT16, cudaStream_t st, int* launches) {
  const size_t smem = ((size_t)8 * pr.k + 32 * (pr.d + 1)) * 4;
  auto fn = simt_key_side<T, P>;
  if (smem > 24 * 1024) {
    cudaError_t e = cudaFuncSetAttribute(fn, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)smem);
    if (e != cudaSuccess) return cuda_fail(e);
  }
  dim3 grid((pr.p() + 7) / 8, pr.BH());
  fn<<<grid, 256, smem, st>>>(kpvp, (const T*)W, weight, a32, aT16, pr.BH(), pr.d, pr.k, pr.p());
  ++*launches;
  return FLURKA_OK;
}

template <typename T, bool P>
int launch_simt_query_side(const Problem& pr, const void* Q, const void* W, const float* weight,
                           const float* a32, void* out, cudaStream_t st, int* launches) {
  const size_t smem = ((size_t)32 * (pr.d + 1) + 32 * pr.d) * 4;
  dim3 grid((pr.N + 31) / 32, pr.BH());
  if (smem > 24 * 1024) {   // static (16.6 KB) + dynamic may pass the 48 KB default limit
    cudaError_t e = cudaFuncSetAttribute(simt_query_side<T, P>, cudaFuncAttributeMaxDynamicSharedMemorySize,
                                         (int)smem);
    if (e != cudaSuccess) return cuda_fail(e);
  }
  simt_query_side<T, P><<<grid, 256, smem, st>>>((const T*)Q, (const T*)W, weight, a32, (T*)out, pr.N,
                                                 pr.d, pr.p(), pr.seq_major_heads());
  ++*launches;
  return FLURKA_OK;
}

template <typename T>
int key_side_dispatch(const Problem& pr, const float* kpvp, const void* W, float* weight, float* a32,
                      __half* aT16, cudaStream_t st, int* launches) {
  return pr.kernel == FLURKA_PERFORMER
             ? launch_simt_key_side<T, true>(pr, kpvp, W, weight, a32, aT16, st, launches)
             : launch_simt_key_side<T, false>(pr, kpvp, W, weight, a32, aT16, st, launches);
}

// The three stages in order.  tc1 / tc3 choose the tensor-core kernel for stage 1 / stage 3
// (bf16 only); tc2 (which needs tc3) does the same for stage 2.  `timer` (may be NULL) gets an
// event before and after each stage.  `keep_status`: the status words are left as they are (a
// later head group of one host-buffer call; they only ever gain bits).
// `stage1(kpvp, status, launches)` fills the (zeroed) K', V' accumulators: the down-projection of
// already projected heads, or the contraction and the linear maps of un-projected inputs.
template <typename T, typename Stage1>
int run_pipeline_with(const Problem& pr, const Layout& L, char* ws, const void* Q, const void* W, void* out,
                      cudaStream_t st, bool tc2, bool tc3, TensorContext* tc, StageTimer* timer, bool keep_status,
                      int* launches, Stage1&& stage1, int phases = 3) {
  // phases: bit 0 = clear the accumulators and run stage 1, bit 1 = run stages 2 and 3 (a sequence-sharded
  // forward does the two halves in separate calls, with the sum over the shards in between)
  float* kpvp = (float*)(ws + L.kpvp);
  float* weight = (float*)(ws + L.weight);
  float* a32 = (float*)(ws + L.a32);
  __half* aT16 = (__half*)(ws + L.aT16);
  int* status = (int*)(ws + L.status);
  const bool performer = pr.kernel == FLURKA_PERFORMER;
  int cuda_err = 0;
  // one memset: the status words, the arrival counters and the K', V' accumulators the kernels add into
  const size_t clear_from = L.status + (keep_status ? 16 : 0);
  cudaError_t e = cudaSuccess;
  int rc = FLURKA_OK;
  if (phases & 1) {
    e = cudaMemsetAsync(ws + clear_from, 0, L.kpvp_end - clear_from, st);
    if (e != cudaSuccess) return cuda_fail(e);
    if (timer) timer->mark(0, st);
    rc = stage1(kpvp, status, launches);
    if (rc) return rc;
    if (timer) timer->mark(1, st);
  }
  if (!(phases & 2)) {
    e = cudaGetLastError();
    return e == cudaSuccess ? FLURKA_OK : cuda_fail(e);
  }
  if (tc2) {
    float* part = L.total > L.part ? (float*)(ws + L.part) : nullptr;
    rc = launch_k2(*tc, performer, kpvp, W, weight, aT16, part, status + 4, pr.BH(), pr.d, pr.k, pr.p(), status, st,
                   &cuda_err);
    if (rc) { g_last_cuda_error = cuda_err; return rc; }
    ++*launches;
  } else {
    rc = key_side_dispatch<T>(pr, kpvp, W, weight, tc3 ? nullptr : a32, tc3 ? aT16 : nullptr, st, launches);
    if (rc) return rc;
  }
  if (timer) timer->mark(2, st);
  if (tc3) {
    rc = launch_k3(*tc, performer, Q, W, aT16, weight, out, pr.BH(), pr.seq_major_heads(), pr.N, pr.d, pr.p(),
                   status, st, &cuda_err);
    if (rc) { g_last_cuda_error = cuda_err; return rc; }
    ++*launches;
  } else {
    rc = performer ? launch_simt_query_side<T, true>(pr, Q, W, weight, a32, out, st, launches)
                   : launch_simt_query_side<T, false>(pr, Q, W, weight, a32, out, st, launches);
    if (rc) return rc;
  }
  if (timer) timer->mark(3, st);
  e = cudaGetLastError();
  if (e != cudaSuccess) return cuda_fail(e);
  return FLURKA_OK;
}

template <typename T>
int run_pipeline(const Problem& pr, const Layout& L, char* ws, const void* Q, const void* K, const void* V,
                 const void* E, const void* F, const void* W, void* out, cudaStream_t st, bool tc1, bool tc2,
                 bool tc3, TensorContext* tc, StageTimer* timer, bool keep_status, int* launches, int phases = 3) {
  auto stage1 = [&](float* kpvp, int* status, int* n) -> int {
    if (tc1) {
      int cuda_err = 0;
      int rc = launch_k1(*tc, K, V, E, F, kpvp, pr.BH(), pr.seq_major_heads(), pr.N, pr.d, pr.k, status, st, &cuda_err,
                         pr.ef_heads());
      if (rc) { g_last_cuda_error = cuda_err; return rc; }
      ++*n;
      return FLURKA_OK;
    }
    return launch_simt_down_project<T>(pr, K, V, E, F, kpvp, st, n);
  };
  return run_pipeline_with<T>(pr, L, ws, Q, W, out, st, tc2, tc3, tc, timer, keep_status, launches, stage1, phases);
}

int validate_pointers(const Problem& pr, const void* Q, const void* K, const void* V, const void* E,
                      const void* F, const void* W, const void* out) {
  if (!Q || !K || !V || !E || !F || !out) return FLURKA_ERR_NULL;
  if (pr.kernel == FLURKA_PERFORMER && !W) return FLURKA_ERR_NULL;
  const void* ptrs[7] = {Q, K, V, E, F, W, out};
  for (const void* ptr : ptrs)
    if (ptr && ((uintptr_t)ptr & 15)) return FLURKA_ERR_ALIGN;
  const size_t qb = pr.qkv_elems() * pr.esize(), eb = pr.ef_elems() * pr.esize(),
               wb = pr.w_elems() * pr.esize();
  if (overlaps(out, qb, Q, qb) || overlaps(out, qb, K, qb) || overlaps(out, qb, V, qb) ||
      overlaps(out, qb, E, eb) || overlaps(out, qb, F, eb) || (W && wb && overlaps(out, qb, W, wb)))
    return FLURKA_ERR_OVERLAP;
  return FLURKA_OK;
}

// flurka_forward proper.  `reserve` (>= the problem's own need, or 0) is the workspace size to ask
// for, so that a caller that runs several problems in a row gets one block that fits them all.
int forward_device(const void* Q, const void* K, const void* V, const void* E, const void* F, const void* W,
                   int variant, int B, int H, int N, int d, int k, int m, void* out, void* stream,
                   bool keep_status, size_t reserve, int phases = 3) {
  Problem pr;
  int rc = parse_problem(variant, B, H, N, d, k, m, &pr);
  if (rc) return rc;
  if (phases == 3) {
    rc = validate_pointers(pr, Q, K, V, E, F, W, out);
  } else if (phases == 1) {
    // first half of a sequence-sharded forward: keys, values and projections only
    if (!K || !V || !E || !F) return FLURKA_ERR_NULL;
    for (const void* ptr : {K, V, E, F})
      if ((uintptr_t)ptr & 15) return FLURKA_ERR_ALIGN;
  } else {
    // second half: queries, the random features, the output
    if (!Q || !out || (pr.kernel == FLURKA_PERFORMER && !W)) return FLURKA_ERR_NULL;
    for (const void* ptr : {Q, W, (const void*)out})
      if (ptr && ((uintptr_t)ptr & 15)) return FLURKA_ERR_ALIGN;
    if (overlaps(out, pr.qkv_elems() * pr.esize(), Q, pr.qkv_elems() * pr.esize())) return FLURKA_ERR_OVERLAP;
  }
  if (rc) return rc;
  int path = g_path;
  const bool tensor_ok = tensor_path_ok(pr);
  if (path >= FLURKA_PATH_TENSOR && !tensor_ok) return FLURKA_ERR_SHAPE;
  if (path == FLURKA_PATH_AUTO) path = tensor_ok ? FLURKA_PATH_TENSOR : FLURKA_PATH_SIMT;
  rc = check_device();
  if (rc) return rc;
  DeviceState& ds = dev_state();
  const Layout L = make_layout(pr);
  cudaStream_t st = (cudaStream_t)stream;
  char* ws = nullptr;
  if (phases == 2) {
    // the second half works on what the first half (and the caller's sum over the shards) left in the
    // workspace: same device, same head count and sizes (the slice length may differ)
    const Problem& lp = ds.last_problem;
    if (!ds.have_last || !ds.partial_pending || lp.BH() != pr.BH() || lp.d != pr.d || lp.k != pr.k || lp.m != pr.m ||
        lp.kernel != pr.kernel || lp.fp32 != pr.fp32)
      return FLURKA_ERR_WORKSPACE;
    ws = ds.last_ws;
  } else {
    rc = get_workspace(ds, std::max(L.total, reserve), st, &ws);
    if (rc) return rc;
  }
  int launches = 0;
  ds.timer.on = g_stage_timing && phases == 3;
  StageTimer* timer = ds.timer.on ? &ds.timer : nullptr;
  if (timer) {
    rc = timer->create();
    if (rc != cudaSuccess) return cuda_fail((cudaError_t)rc);
  }
  if (pr.fp32) {
    rc = run_pipeline<float>(pr, L, ws, Q, K, V, E, F, W, out, st, false, false, false, &ds.tc, timer, keep_status,
                             &launches, phases);
  } else {
    const bool tc1 = path == FLURKA_PATH_TENSOR || path == FLURKA_PATH_TENSOR_STAGE1;
    const bool tc2 = path == FLURKA_PATH_TENSOR || path == FLURKA_PATH_TENSOR_STAGE23;
    const bool tc3 = path == FLURKA_PATH_TENSOR || path == FLURKA_PATH_TENSOR_STAGE3 || tc2;
    rc = run_pipeline<__nv_bfloat16>(pr, L, ws, Q, K, V, E, F, W, out, st, tc1, tc2, tc3, &ds.tc, timer,
                                     keep_status, &launches, phases);
  }
  if (rc) return rc;
  ds.partial_pending = phases != 3;       // K', V' of a sharded forward stay in the workspace
  ds.timer.have = ds.timer.on;
  ds.last_path = path;
  ds.last_launches = launches;
  ds.have_last = true;
  ds.last_problem = pr;
  ds.last_ws = ws;
  return FLURKA_OK;
}

}  // namespace

extern "C" {

int flurka_forward(const void* Q, const void* K, const void* V, const void* E, const void* F,
                   const void* W, int variant, int B, int H, int N, int d, int k, int m, void* out,
                   void* stream) {
  return forward_device(Q, K, V, E, F, W, variant, B, H, N, d, k, m, out, stream, /*keep_status=*/false, 0);
}

int flurka_forward_partial(const void* K, const void* V, const void* E, const void* F, int variant, int B, int H,
                           int N, int d, int k, int m, void* stream) {
  return forward_device(nullptr, K, V, E, F, nullptr, variant, B, H, N, d, k, m, nullptr, stream, false, 0, /*phases=*/1);
}

int flurka_forward_finish(const void* Q, const void* W, int variant, int B, int H, int N, int d, int k, int m,
                          void* out, void* stream) {
  return forward_device(Q, nullptr, nullptr, nullptr, nullptr, W, variant, B, H, N, d, k, m, out, stream, false, 0,
                        /*phases=*/2);
}

int flurka_partial_sums(void** dev_ptr, size_t* bytes) {
  if (!dev_ptr || !bytes) return FLURKA_ERR_NULL;
  DeviceState& ds = dev_state();
  if (!ds.have_last || !ds.partial_pending) return FLURKA_ERR_WORKSPACE;
  const Layout L = make_layout(ds.last_problem);
  *dev_ptr = ds.last_ws + L.kpvp;
  *bytes = L.kpvp_end - L.kpvp;
  return FLURKA_OK;
}

int flurka_forward_host(const void* Q, const void* K, const void* V, const void* E, const void* F,
                        const void* W, int variant, int B, int H, int N, int d, int k, int m, void* out,
                        void* stream) {
  Problem pr;
  int rc = parse_problem(variant, B, H, N, d, k, m, &pr);
  if (rc) return rc;
  if (!Q || !K || !V || !E || !F || !out) return FLURKA_ERR_NULL;
  if (pr.kernel == FLURKA_PERFORMER && !W) return FLURKA_ERR_NULL;
  rc = check_device();
  if (rc) return rc;
  DeviceState& ds = dev_state();
  const size_t qb = align256(pr.qkv_elems() * pr.esize());
  const size_t eb = align256(pr.ef_elems() * pr.esize());
  const size_t wb = align256(pr.w_elems() * pr.esize());
  const size_t need = 4 * qb + 2 * eb + wb;
  if (ds.stage_bytes < need) {
    if (ds.stage) {
      cudaError_t e = cudaDeviceSynchronize();
      if (e != cudaSuccess) return cuda_fail(e);
      cudaFree(ds.stage);
      ds.stage = nullptr;
      ds.stage_bytes = 0;
    }
    cudaError_t e = cudaMalloc(&ds.stage, need);
    if (e != cudaSuccess) { cuda_fail(e); return FLURKA_ERR_WORKSPACE; }
    ds.stage_bytes = need;
  }
  char* base = (char*)ds.stage;
  char* dQ = base;
  char* dK = dQ + qb;
  char* dV = dK + qb;
  char* dO = dV + qb;
  char* dE = dO + qb;
  char* dF = dE + eb;
  char* dW = dF + eb;
  cudaStream_t st = (cudaStream_t)stream;
  const size_t qn = pr.qkv_elems() * pr.esize(), en = pr.ef_elems() * pr.esize(),
               wn = pr.w_elems() * pr.esize();
  cudaError_t e;
  if ((e = cudaMemcpyAsync(dE, E, en, cudaMemcpyHostToDevice, st)) != cudaSuccess) return cuda_fail(e);
  if ((e = cudaMemcpyAsync(dF, F, en, cudaMemcpyHostToDevice, st)) != cudaSuccess) return cuda_fail(e);
  if (wn && (e = cudaMemcpyAsync(dW, W, wn, cudaMemcpyHostToDevice, st)) != cudaSuccess)
    return cuda_fail(e);

  // The heads are independent, so the call works through them in up to eight groups: while the
  // inputs of one group travel to the device, the output of the group before travels back on a second
  // stream (the link is full duplex), and the compute of a group hides under the copies.
  // (units that are contiguous in memory: heads for [B,H,N,d], batches for [B,N,H,d]; whole batches
  // also when every head has its own E, F, so that a group's heads keep their numbers)
  const bool by_batch = pr.bnhd || pr.ef_per_head;
  const int heads = by_batch ? pr.B : pr.BH();
  int groups = (int)std::min<size_t>(8, qn >> 20);           // at least 1 MiB of Q per group
  groups = std::max(1, std::min(groups, heads));
  if (groups > 1 && !ds.out_stream) {
    if ((e = cudaStreamCreateWithFlags(&ds.out_stream, cudaStreamNonBlocking)) != cudaSuccess) return cuda_fail(e);
    for (int i = 0; i < 8; ++i)
      if ((e = cudaEventCreateWithFlags(&ds.group_done[i], cudaEventDisableTiming)) != cudaSuccess) return cuda_fail(e);
    if ((e = cudaEventCreateWithFlags(&ds.out_done, cudaEventDisableTiming)) != cudaSuccess) return cuda_fail(e);
  }
  // The groups need not be equal (12 heads in 8 groups: 1, 2, 1, 2, ...).  One workspace that fits the
  // largest group is obtained before the first group runs, so it never moves between groups; the
  // status words sit at its start for every group size.
  size_t reserve = 0;
  for (int gi = 0; gi < groups; ++gi) {
    const int cnt = (int)((long long)heads * (gi + 1) / groups) - (int)((long long)heads * gi / groups);
    Problem sub = pr;
    if (by_batch) sub.B = cnt; else { sub.B = 1; sub.H = cnt; }
    reserve = std::max(reserve, make_layout(sub).total);
  }
  const size_t head_bytes = (size_t)N * d * pr.esize() * (by_batch ? H : 1);
  rc = FLURKA_OK;
  for (int gi = 0; gi < groups && rc == FLURKA_OK; ++gi) {
    const int h0 = (int)((long long)heads * gi / groups), h1 = (int)((long long)heads * (gi + 1) / groups);
    const size_t off = (size_t)h0 * head_bytes, len = (size_t)(h1 - h0) * head_bytes;
    if ((e = cudaMemcpyAsync(dQ + off, (const char*)Q + off, len, cudaMemcpyHostToDevice, st)) != cudaSuccess ||
        (e = cudaMemcpyAsync(dK + off, (const char*)K + off, len, cudaMemcpyHostToDevice, st)) != cudaSuccess ||
        (e = cudaMemcpyAsync(dV + off, (const char*)V + off, len, cudaMemcpyHostToDevice, st)) != cudaSuccess) {
      rc = cuda_fail(e);
      break;
    }
    rc = forward_device(dQ + off, dK + off, dV + off, dE, dF, wn ? dW : nullptr, variant, by_batch ? h1 - h0 : 1,
                        by_batch ? H : h1 - h0, N, d, k, m, dO + off, stream, /*keep_status=*/gi > 0, reserve);
    if (rc) break;
    if (groups == 1) {
      if ((e = cudaMemcpyAsync(out, dO, qn, cudaMemcpyDeviceToHost, st)) != cudaSuccess) rc = cuda_fail(e);
    } else {
      if ((e = cudaEventRecord(ds.group_done[gi], st)) != cudaSuccess ||
          (e = cudaStreamWaitEvent(ds.out_stream, ds.group_done[gi], 0)) != cudaSuccess ||
          (e = cudaMemcpyAsync((char*)out + off, dO + off, len, cudaMemcpyDeviceToHost, ds.out_stream)) != cudaSuccess)
        rc = cuda_fail(e);
    }
  }
  if (groups > 1) {
    // the caller's stream also waits for the copies on the second stream
    if (cudaEventRecord(ds.out_done, ds.out_stream) == cudaSuccess) cudaStreamWaitEvent(st, ds.out_done, 0);
  }
  e = cudaStreamSynchronize(st);
  if (rc) return rc;
  if (e != cudaSuccess) return cuda_fail(e);
  return FLURKA_OK;
}

size_t flurka_workspace_bytes(int variant, int B, int H, int N, int d, int k, int m) {
  Problem pr;
  if (parse_problem(variant, B, H, N, d, k, m, &pr)) return 0;
  return make_layout(pr).total;
}

int flurka_set_workspace(void* dev_ptr, size_t bytes) {
  if (dev_ptr && ((uintptr_t)dev_ptr & 255)) return FLURKA_ERR_ALIGN;
  if (dev_ptr && bytes == 0) return FLURKA_ERR_WORKSPACE;
  DeviceState& ds = dev_state();
  ds.user_ws = dev_ptr;
  ds.user_ws_bytes = dev_ptr ? bytes : 0;
  ds.have_last = false;
  return FLURKA_OK;
}

int flurka_set_path(int path) {
  const int prev = g_path;
  if (path >= FLURKA_PATH_AUTO && path <= FLURKA_PATH_TENSOR_STAGE23) g_path = path;
  return prev;
}

int flurka_set_cta_limit(int max_ctas) {
  const int prev = cta_limit();
  cta_limit() = max_ctas > 0 ? max_ctas : 0;
  return prev;
}

int flurka_set_stage1_pairs(int on) {
  const int prev = stage1_pairs();
  stage1_pairs() = on != 0;
  return prev;
}

int flurka_last_path(void) { return dev_state().last_path; }
int flurka_last_launches(void) { return dev_state().last_launches; }

int flurka_debug_copy(int which, void* dev_dst, size_t bytes, void* stream) {
  if (!dev_dst) return FLURKA_ERR_NULL;
  DeviceState& ds = dev_state();
  if (!ds.have_last) return FLURKA_ERR_WORKSPACE;
  const Problem& pr = ds.last_problem;
  const Layout L = make_layout(pr);
  const size_t kd = (size_t)pr.BH() * pr.k * pr.d * 4;
  size_t off = 0, size = 0;
  switch (which) {
    case 0: off = L.kpvp; size = kd; break;
    case 1: off = L.kpvp + kd; size = kd; break;
    case 2: off = L.a32; size = (size_t)pr.BH() * pr.p() * pr.d * 4; break;
    case 3: off = L.weight; size = (size_t)pr.BH() * pr.p() * 4; break;
    case 4: off = L.status; size = 16; break;
    default: return FLURKA_ERR_VARIANT;
  }
  if (bytes != size) return FLURKA_ERR_SHAPE;
  cudaError_t e = cudaMemcpyAsync(dev_dst, ds.last_ws + off, size, cudaMemcpyDeviceToDevice,
                                  (cudaStream_t)stream);
  if (e != cudaSuccess) return cuda_fail(e);
  return FLURKA_OK;
}

int flurka_last_status(void) {
  DeviceState& ds = dev_state();
  if (!ds.have_last) return 0;
  const Layout L = make_layout(ds.last_problem);
  int words[4] = {0, 0, 0, 0};
  cudaError_t e = cudaDeviceSynchronize();
  if (e != cudaSuccess) return cuda_fail(e);
  e = cudaMemcpy(words, ds.last_ws + L.status, 16, cudaMemcpyDeviceToHost);
  if (e != cudaSuccess) return cuda_fail(e);
  return words[0];
}

int flurka_last_cuda_error(void) { return g_last_cuda_error; }

int flurka_set_stage_timing(int on) {
  g_stage_timing = on != 0;
  for (int i = 0; i < kMaxDevices; ++i) g_dev[i].timer.have = false;
  return FLURKA_OK;
}

int flurka_last_stage_ms(float* ms3) {
  if (!ms3) return FLURKA_ERR_NULL;
  DeviceState& ds = dev_state();
  if (!ds.timer.have) return FLURKA_ERR_WORKSPACE;
  cudaError_t e = cudaEventSynchronize(ds.timer.ev[3]);
  if (e != cudaSuccess) return cuda_fail(e);
  for (int i = 0; i < 3; ++i) {
    e = cudaEventElapsedTime(&ms3[i], ds.timer.ev[i], ds.timer.ev[i + 1]);
    if (e != cudaSuccess) return cuda_fail(e);
  }
  return FLURKA_OK;
}

const char* flurka_strerror(int code) {
  switch (code) {
    case FLURKA_OK: return "ok";
    case FLURKA_ERR_NULL: return "a required pointer is NULL";
    case FLURKA_ERR_VARIANT: return "unknown kernel variant, element type or selector";
    case FLURKA_ERR_SHAPE: return "unsupported shape";
    case FLURKA_ERR_ALIGN: return "pointer not sufficiently aligned";
    case FLURKA_ERR_WORKSPACE: return "workspace missing, too small or not allocatable";
    case FLURKA_ERR_CUDA: return "a CUDA call failed (see flurka_last_cuda_error)";
    case FLURKA_ERR_DEVICE: return "no sm_100 device is current";
    case FLURKA_ERR_OVERLAP: return "out overlaps an input";
    case FLURKA_ERR_TOO_LARGE: return "problem needs more scratch than the built-in array holds";
    default: return "unknown flurka status";
  }
}

int flurka_version(void) { return FLURKA_VERSION; }

}  // extern "C"

namespace {

// Scratch of the entry point with un-projected inputs, after the inner problem's own layout:
//   kt    fp32 E Xk[b], F Xv[b]: tensor path [2][B][dm/64][k][64] (64-wide column blocks), else [2][B][k][dm]
//   a3    bf16 [2B][k][3 dm]: three-term split of kt (tensor path only)
//   qp    Xq W^Q as [B,N,H,d] in the I/O type
struct FusedLayout {
  Layout L;
  size_t kt, kt_bytes, a3, qp, total;
};

FusedLayout make_fused_layout(const Problem& pr, int dm) {
  FusedLayout f;
  f.L = make_layout(pr);
  size_t off = f.L.total;
  f.kt_bytes = (size_t)2 * pr.B * pr.k * dm * 4;
  f.kt = off; off = align256(off + f.kt_bytes);
  f.a3 = off; off = align256(off + (pr.fp32 ? 0 : (size_t)2 * pr.B * pr.k * 3 * dm * 2));
  f.qp = off; off = align256(off + pr.qkv_elems() * pr.esize());
  f.total = off;
  return f;
}

bool fused_tensor_ok(const Problem& pr, int dm) { return tensor_path_ok(pr) && dm % 64 == 0 && dm >= 64; }

template <typename T>
int simt_map(const void* A, const void* Bm, void* C, bool a_f32, bool c_f32, int M, int K, int ncols, int Z,
             size_t a_stride, size_t b_stride, int head_d, int z0, cudaStream_t st, int* launches) {
  dim3 grid((ncols + 31) / 32, (M + 31) / 32, Z);
  if (a_f32)
    simt_linear_map<float, T, float><<<grid, 256, 0, st>>>((const float*)A, (const T*)Bm, (float*)C, M, K, ncols,
                                                           a_stride, b_stride, head_d, z0);
  else if (c_f32)
    simt_linear_map<T, T, float><<<grid, 256, 0, st>>>((const T*)A, (const T*)Bm, (float*)C, M, K, ncols, a_stride,
                                                       b_stride, head_d, z0);
  else
    simt_linear_map<T, T, T><<<grid, 256, 0, st>>>((const T*)A, (const T*)Bm, (T*)C, M, K, ncols, a_stride, b_stride,
                                                   head_d, z0);
  ++*launches;
  cudaError_t e = cudaGetLastError();
  return e == cudaSuccess ? FLURKA_OK : cuda_fail(e);
}

template <typename T>
int fused_pipeline(const Problem& pr, int dm, const FusedLayout& FL, char* ws, const void* Xq, const void* Xk,
                   const void* Xv, const void* E, const void* F, const void* Wq, const void* Wk, const void* Wv,
                   const void* W, void* out, cudaStream_t st, bool tensor, TensorContext* tc, StageTimer* timer,
                   int* launches) {
  float* kt = (float*)(ws + FL.kt);
  void* qp = ws + FL.qp;
  auto stage1 = [&](float* kpvp, int* status, int* n) -> int {
    int cuda_err = 0, rc;
    cudaError_t e = cudaMemsetAsync(kt, 0, FL.kt_bytes, st);
    if (e != cudaSuccess) return cuda_fail(e);
    if (tensor) {
      // Q = Xq W^Q first (the long one), then the contraction of the un-projected keys and values as
      // dm/64 pseudo-heads of width 64, then W^K, W^V on the k contracted rows
      rc = launch_k0_query_map(*tc, Xq, Wq, qp, pr.B, pr.N, pr.H, dm, pr.d, status, st, &cuda_err);
      if (rc) { g_last_cuda_error = cuda_err; return rc; }
      rc = launch_k1(*tc, Xk, Xv, E, F, kt, pr.B * (dm / 64), dm / 64, pr.N, 64, pr.k, status, st, &cuda_err);
      if (rc) { g_last_cuda_error = cuda_err; return rc; }
      rc = launch_k0_key_value_maps(*tc, kt, (__nv_bfloat16*)(ws + FL.a3), Wk, Wv, kpvp, pr.B, pr.H, dm, pr.d, pr.k,
                                    status, st, &cuda_err);
      if (rc) { g_last_cuda_error = cuda_err; return rc; }
      *n += 4;
      return FLURKA_OK;
    }
    const size_t xb = (size_t)pr.N * dm, ktb = (size_t)pr.k * dm;
    // kt[t][b] = (E | F) X[b];  K', V' = kt W^K, kt W^V (head-split);  Q = Xq W^Q
    if ((rc = simt_map<T>(E, Xk, kt, false, true, pr.k, pr.N, dm, pr.B, 0, xb, 0, 0, st, n))) return rc;
    if ((rc = simt_map<T>(F, Xv, kt + (size_t)pr.B * ktb, false, true, pr.k, pr.N, dm, pr.B, 0, xb, 0, 0, st, n))) return rc;
    if ((rc = simt_map<T>(kt, Wk, kpvp, true, true, pr.k, dm, pr.H * pr.d, pr.B, ktb, 0, pr.d, 0, st, n))) return rc;
    if ((rc = simt_map<T>(kt + (size_t)pr.B * ktb, Wv, kpvp, true, true, pr.k, dm, pr.H * pr.d, pr.B, ktb, 0, pr.d, pr.B,
                          st, n))) return rc;
    return simt_map<T>(Xq, Wq, qp, false, sizeof(T) == 4, pr.B * pr.N, dm, pr.H * pr.d, 1, 0, 0, 0, 0, st, n);
  };
  return run_pipeline_with<T>(pr, FL.L, ws, qp, W, out, st, tensor, tensor, tc, timer, /*keep_status=*/false, launches,
                              stage1);
}

}  // namespace

extern "C" {

size_t flurka_fused_workspace_bytes(int variant, int B, int H, int N, int dm, int d, int k, int m) {
  Problem pr;
  if (parse_problem(variant | FLURKA_LAYOUT_BNHD, B, H, N, d, k, m, &pr) || dm <= 0) return 0;
  return make_fused_layout(pr, dm).total;
}

int flurka_forward_fused(const void* Xq, const void* Xk, const void* Xv, const void* E, const void* F,
                         const void* Wq, const void* Wk, const void* Wv, const void* W, int variant, int B, int H,
                         int N, int dm, int d, int k, int m, void* out, void* stream) {
  Problem pr;
  // the layout is fixed (out is [B,N,H,d]); the contraction is shared by all heads, so E, F cannot be per head
  if (variant & (FLURKA_LAYOUT_BNHD | FLURKA_EF_PER_HEAD)) return FLURKA_ERR_VARIANT;
  int rc = parse_problem(variant | FLURKA_LAYOUT_BNHD, B, H, N, d, k, m, &pr);
  if (rc) return rc;
  if (dm <= 0 || dm > 16384) return FLURKA_ERR_SHAPE;
  if (!Xq || !Xk || !Xv || !E || !F || !Wq || !Wk || !Wv || !out) return FLURKA_ERR_NULL;
  if (pr.kernel == FLURKA_PERFORMER && !W) return FLURKA_ERR_NULL;
  const void* ptrs[10] = {Xq, Xk, Xv, E, F, Wq, Wk, Wv, W, out};
  for (const void* ptr : ptrs)
    if (ptr && ((uintptr_t)ptr & 15)) return FLURKA_ERR_ALIGN;
  const size_t xb = (size_t)B * N * dm * pr.esize(), ob = pr.qkv_elems() * pr.esize(),
               eb = pr.ef_elems() * pr.esize(), mb = (size_t)dm * H * d * pr.esize(), wb = pr.w_elems() * pr.esize();
  if (overlaps(out, ob, Xq, xb) || overlaps(out, ob, Xk, xb) || overlaps(out, ob, Xv, xb) || overlaps(out, ob, E, eb) ||
      overlaps(out, ob, F, eb) || overlaps(out, ob, Wq, mb) || overlaps(out, ob, Wk, mb) || overlaps(out, ob, Wv, mb) ||
      (W && wb && overlaps(out, ob, W, wb)))
    return FLURKA_ERR_OVERLAP;
  int path = g_path;
  const bool tensor_ok = fused_tensor_ok(pr, dm);
  if (path >= FLURKA_PATH_TENSOR && !tensor_ok) return FLURKA_ERR_SHAPE;
  if (path == FLURKA_PATH_AUTO) path = tensor_ok ? FLURKA_PATH_TENSOR : FLURKA_PATH_SIMT;
  if (path != FLURKA_PATH_TENSOR && path != FLURKA_PATH_SIMT) return FLURKA_ERR_VARIANT;   // no bisecting paths here
  rc = check_device();
  if (rc) return rc;
  DeviceState& ds = dev_state();
  const FusedLayout FL = make_fused_layout(pr, dm);
  cudaStream_t st = (cudaStream_t)stream;
  char* ws = nullptr;
  rc = get_workspace(ds, FL.total, st, &ws);
  if (rc) return rc;
  int launches = 0;
  ds.timer.on = g_stage_timing;
  StageTimer* timer = g_stage_timing ? &ds.timer : nullptr;
  if (timer) {
    rc = timer->create();
    if (rc != cudaSuccess) return cuda_fail((cudaError_t)rc);
  }
  if (pr.fp32)
    rc = fused_pipeline<float>(pr, dm, FL, ws, Xq, Xk, Xv, E, F, Wq, Wk, Wv, W, out, st, false, &ds.tc, timer, &launches);
  else
    rc = fused_pipeline<__nv_bfloat16>(pr, dm, FL, ws, Xq, Xk, Xv, E, F, Wq, Wk, Wv, W, out, st,
                                       path == FLURKA_PATH_TENSOR, &ds.tc, timer, &launches);
  if (rc) return rc;
  ds.timer.have = g_stage_timing;
  ds.partial_pending = false;
  ds.last_path = path;
  ds.last_launches = launches;
  ds.have_last = true;
  ds.last_problem = pr;
  ds.last_ws = ws;
  return FLURKA_OK;
}

}  // extern "C"

namespace {

// Scratch of the backward pass, after the forward layout: da [BH][p][d], db [BH][p] (adjacent: one
// memset), then dK', dV' [2][BH][k][d]; all fp32.
struct BackwardLayout {
  Layout L;
  size_t da, dab_bytes, db, dkpvp, abf, split, rowstat, total;
};

// the query side of the backward has a tensor-core kernel for d = 64 (PERFORMER: any feature count the
// forward's tensor path takes, 64 to 256; RNN: its 64 features are the head dimension) and for PERFORMER
// with d = 128
bool backward_tensor_ok(const Problem& pr) {
  return tensor_path_ok(pr) && (pr.d == 64 || pr.kernel == FLURKA_PERFORMER);
}

BackwardLayout make_backward_layout(const Problem& pr) {
  BackwardLayout b;
  b.L = make_layout(pr, /*with_split_scratch=*/false);
  size_t off = b.L.total;
  const size_t da_bytes = (size_t)pr.BH() * pr.p() * pr.d * 4;
  b.da = off;
  b.db = off + da_bytes;
  b.dab_bytes = da_bytes + (size_t)pr.BH() * pr.p() * 4;
  off = align256(off + b.dab_bytes);
  b.dkpvp = off; off = align256(off + (size_t)2 * pr.BH() * pr.k * pr.d * 4);
  b.abf = off;
  if (backward_tensor_ok(pr)) off = align256(off + (size_t)2 * pr.BH() * pr.p() * pr.d * 2);   // a as two bf16 terms
  b.rowstat = off;
  if (backward_tensor_ok(pr) && pr.d == 128)             // (log-sum-exp, delta) of every row of every 128-row tile
    off = align256(off + (size_t)pr.BH() * ((pr.N + 127) / 128) * 128 * 8);
  b.split = off;
  if (tensor_path_ok(pr)) off = align256(off + (size_t)2 * pr.k * 2 * pr.BH() * pr.d * 2);      // dK', dV' as two bf16 terms
  b.total = off;
  return b;
}

template <typename T, bool P>
int backward_pipeline(const Problem& pr, const BackwardLayout& BL, char* ws, const void* Q, const void* K,
                      const void* V, const void* E, const void* F, const void* W, const void* dO, void* dQ, void* dK,
                      void* dV, void* dE, void* dF, cudaStream_t st, int* launches, TensorContext* tc, bool tcq) {
  // tc != NULL: stage 1 and (with shared E, F) the projection gradients run on the tensor-core kernels;
  // tcq: so does the query side (bf16 PERFORMER, d = 64, 128 or 256 features)
  const Layout& L = BL.L;
  float* kpvp = (float*)(ws + L.kpvp);
  float* weight = (float*)(ws + L.weight);
  float* a32 = (float*)(ws + L.a32);
  float* da = (float*)(ws + BL.da);
  float* db = (float*)(ws + BL.db);
  float* dkpvp = (float*)(ws + BL.dkpvp);
  const int smh = pr.seq_major_heads(), efh = pr.ef_heads();
  cudaError_t e = cudaMemsetAsync(ws + L.status, 0, L.kpvp_end - L.status, st);
  if (e != cudaSuccess) return cuda_fail(e);
  if ((e = cudaMemsetAsync(da, 0, BL.dab_bytes, st)) != cudaSuccess) return cuda_fail(e);
  // the forward's stages 1 and 2 again: K', V', a_i, b_i (or z_i)
  int rc = FLURKA_OK;
  int cuda_err = 0;
  if (tc) {
    rc = launch_k1(*tc, K, V, E, F, kpvp, pr.BH(), smh, pr.N, pr.d, pr.k, (int*)(ws + L.status), st, &cuda_err, efh);
    if (rc) { g_last_cuda_error = cuda_err; return rc; }
    ++*launches;
  } else {
    rc = launch_simt_down_project<T>(pr, K, V, E, F, kpvp, st, launches);
    if (rc) return rc;
  }
  if (tc) {
    // the key side on its tensor-core kernel, one CTA per (head, feature tile), with a in fp32 as well
    rc = launch_k2(*tc, P, kpvp, W, weight, (__half*)(ws + L.aT16), nullptr, nullptr, pr.BH(), pr.d, pr.k, pr.p(),
                   (int*)(ws + L.status), st, &cuda_err, a32);
    if (rc) { g_last_cuda_error = cuda_err; return rc; }
    ++*launches;
  } else {
    rc = launch_simt_key_side<T, P>(pr, kpvp, W, weight, a32, nullptr, st, launches);
    if (rc) return rc;
  }
  if (tc && tcq) {
    rc = launch_k4(*tc, P, Q, dO, W, a32, weight, (__nv_bfloat16*)(ws + BL.abf), dQ, da, db, pr.BH(), smh, pr.N, pr.d, pr.p(),
                   (int*)(ws + L.status), st, &cuda_err, ws + BL.rowstat);
    if (rc) { g_last_cuda_error = cuda_err; return rc; }
    *launches += 2;
  } else {
    auto fn = simt_bwd_query_side<T, P>;
    const size_t smem = ((size_t)2 * 32 * (pr.d + 1) + 32 * 33 + 32 * pr.d) * 4;
    if ((e = cudaFuncSetAttribute(fn, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)smem)) != cudaSuccess)
      return cuda_fail(e);
    dim3 grid((pr.N + 31) / 32, pr.BH());
    fn<<<grid, 256, smem, st>>>((const T*)Q, (const T*)W, (const T*)dO, weight, a32, (T*)dQ, da, db, pr.N, pr.d,
                                pr.p(), smh);
    ++*launches;
  }
  if (tc && P && pr.d == 64) {
    rc = launch_k6(*tc, W, kpvp, weight, a32, da, db, dkpvp, pr.BH(), pr.k, pr.p(), (int*)(ws + L.status), st, &cuda_err);
    if (rc) { g_last_cuda_error = cuda_err; return rc; }
    ++*launches;
  } else {
    auto fn = simt_bwd_key_side<T, P>;
    const size_t smem = ((size_t)3 * 32 * (pr.d + 1) + (size_t)2 * 8 * kBwdKeysPerWarp * pr.d) * 4;
    if ((e = cudaFuncSetAttribute(fn, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)smem)) != cudaSuccess)
      return cuda_fail(e);
    dim3 grid((pr.k + 8 * kBwdKeysPerWarp - 1) / (8 * kBwdKeysPerWarp), pr.BH());
    fn<<<grid, 256, smem, st>>>(kpvp, (const T*)W, weight, a32, da, db, dkpvp, pr.BH(), pr.d, pr.k, pr.p());
    ++*launches;
  }
  if (tc && efh == 0) {
    rc = launch_k5(*tc, E, F, K, V, dkpvp, (__nv_bfloat16*)(ws + BL.split), dK, dV, dE, dF, pr.BH(), smh, pr.N, pr.d, pr.k,
                   (int*)(ws + L.status), st, &cuda_err);
    if (rc) { g_last_cuda_error = cuda_err; return rc; }
    *launches += 3;
  } else {
    dim3 grid((pr.N + 31) / 32, pr.BH(), 2);
    simt_bwd_inputs<T><<<grid, 256, 0, st>>>((const T*)E, (const T*)F, dkpvp, (T*)dK, (T*)dV, pr.BH(), pr.N, pr.d,
                                             pr.k, smh, efh);
    ++*launches;
    dim3 grid2((pr.N + 31) / 32, (pr.k + 31) / 32, 2 * (efh > 0 ? efh : 1));
    simt_bwd_projections<T><<<grid2, 256, 0, st>>>((const T*)K, (const T*)V, dkpvp, (T*)dE, (T*)dF, pr.BH(), pr.N,
                                                   pr.d, pr.k, smh, efh);
    ++*launches;
  }
  e = cudaGetLastError();
  return e == cudaSuccess ? FLURKA_OK : cuda_fail(e);
}

}  // namespace

extern "C" {

size_t flurka_backward_workspace_bytes(int variant, int B, int H, int N, int d, int k, int m) {
  Problem pr;
  if (parse_problem(variant, B, H, N, d, k, m, &pr)) return 0;
  return make_backward_layout(pr).total;
}

int flurka_backward(const void* Q, const void* K, const void* V, const void* E, const void* F, const void* W,
                    const void* dO, int variant, int B, int H, int N, int d, int k, int m, void* dQ, void* dK,
                    void* dV, void* dE, void* dF, void* stream) {
  Problem pr;
  int rc = parse_problem(variant, B, H, N, d, k, m, &pr);
  if (rc) return rc;
  if (!Q || !K || !V || !E || !F || !dO || !dQ || !dK || !dV || !dE || !dF) return FLURKA_ERR_NULL;
  if (pr.kernel == FLURKA_PERFORMER && !W) return FLURKA_ERR_NULL;
  const void* ins[7] = {Q, K, V, E, F, W, dO};
  void* outs[5] = {dQ, dK, dV, dE, dF};
  const size_t qb = pr.qkv_elems() * pr.esize(), eb = pr.ef_elems() * pr.esize(), wb = pr.w_elems() * pr.esize();
  const size_t in_bytes[7] = {qb, qb, qb, eb, eb, wb, qb}, out_bytes[5] = {qb, qb, qb, eb, eb};
  for (const void* ptr : ins)
    if (ptr && ((uintptr_t)ptr & 15)) return FLURKA_ERR_ALIGN;
  for (int o = 0; o < 5; ++o) {
    if ((uintptr_t)outs[o] & 15) return FLURKA_ERR_ALIGN;
    for (int i = 0; i < 7; ++i)
      if (ins[i] && in_bytes[i] && overlaps(outs[o], out_bytes[o], ins[i], in_bytes[i])) return FLURKA_ERR_OVERLAP;
    for (int o2 = 0; o2 < o; ++o2)
      if (overlaps(outs[o], out_bytes[o], outs[o2], out_bytes[o2])) return FLURKA_ERR_OVERLAP;
  }
  rc = check_device();
  if (rc) return rc;
  DeviceState& ds = dev_state();
  const BackwardLayout BL = make_backward_layout(pr);
  cudaStream_t st = (cudaStream_t)stream;
  char* ws = nullptr;
  rc = get_workspace(ds, BL.total, st, &ws);
  if (rc) return rc;
  int launches = 0;
  const bool perf = pr.kernel == FLURKA_PERFORMER;
  // tensor-core kernels for stage 1 and the query side where the shape allows (and the path knob does not
  // force the CUDA-core kernels); a forced tensor path with another shape is refused
  const bool tensor_ok = backward_tensor_ok(pr);
  if (g_path >= FLURKA_PATH_TENSOR && !tensor_ok) return FLURKA_ERR_SHAPE;
  TensorContext* tc = (tensor_path_ok(pr) && g_path != FLURKA_PATH_SIMT) ? &ds.tc : nullptr;
  const bool tcq = tc && tensor_ok;
  if (pr.fp32)
    rc = perf ? backward_pipeline<float, true>(pr, BL, ws, Q, K, V, E, F, W, dO, dQ, dK, dV, dE, dF, st, &launches, nullptr, false)
              : backward_pipeline<float, false>(pr, BL, ws, Q, K, V, E, F, W, dO, dQ, dK, dV, dE, dF, st, &launches,
                                                nullptr, false);
  else
    rc = perf ? backward_pipeline<__nv_bfloat16, true>(pr, BL, ws, Q, K, V, E, F, W, dO, dQ, dK, dV, dE, dF, st, &launches, tc, tcq)
              : backward_pipeline<__nv_bfloat16, false>(pr, BL, ws, Q, K, V, E, F, W, dO, dQ, dK, dV, dE, dF, st,
                                                        &launches, tc, tcq);
  if (rc) return rc;
  ds.partial_pending = false;
  ds.timer.have = false;
  ds.last_path = tcq ? FLURKA_PATH_TENSOR : (tc ? FLURKA_PATH_TENSOR_STAGE1 : FLURKA_PATH_SIMT);
  ds.last_launches = launches;
  ds.have_last = true;
  ds.last_problem = pr;
  ds.last_ws = ws;
  return FLURKA_OK;
}

// A loop of nothing but exponentials: eight independent ex2.approx chains per thread, every SM full.
namespace {
__global__ void ex2_rate_kernel(int iters, float* sink) {
  float x[8];
#pragma unroll
  for (int c = 0; c < 8; ++c) x[c] = -0.001f * (float)(threadIdx.x + c + 1);
  for (int i = 0; i < iters; ++i) {
#pragma unroll
    for (int c = 0; c < 8; ++c) asm volatile("ex2.approx.ftz.f32 %0, %0;" : "+f"(x[c]));
  }
  float acc = 0.f;
#pragma unroll
  for (int c = 0; c < 8; ++c) acc += x[c];
  if (acc == -1.f) sink[0] = acc;       // never true (2^x > 0): keeps the chains alive
}
}  // namespace

int flurka_measure_ex2_rate(double* gexp_per_s) {
  if (!gexp_per_s) return FLURKA_ERR_NULL;
  int rc = check_device();
  if (rc) return rc;
  DeviceState& ds = dev_state();
  const int blocks = ds.tc.sm_total() * 8, threads = 256, iters = 4096;
  float* sink = nullptr;
  cudaEvent_t e0 = nullptr, e1 = nullptr;
  cudaError_t e = cudaMalloc(&sink, sizeof(float));
  if (e != cudaSuccess) return cuda_fail(e);
  if ((e = cudaEventCreate(&e0)) != cudaSuccess || (e = cudaEventCreate(&e1)) != cudaSuccess) {
    cudaFree(sink);
    if (e0) cudaEventDestroy(e0);
    return cuda_fail(e);
  }
  float best_ms = 0.f;
  for (int rep = 0; rep < 4; ++rep) {               // the first launch warms up
    cudaEventRecord(e0, 0);
    ex2_rate_kernel<<<blocks, threads>>>(iters, sink);
    cudaEventRecord(e1, 0);
    e = cudaEventSynchronize(e1);
    if (e != cudaSuccess) break;
    float ms = 0.f;
    cudaEventElapsedTime(&ms, e0, e1);
    if (rep > 0 && (best_ms == 0.f || ms < best_ms)) best_ms = ms;
  }
  cudaEventDestroy(e0);
  cudaEventDestroy(e1);
  cudaFree(sink);
  if (e != cudaSuccess) return cuda_fail(e);
  if (best_ms <= 0.f) return FLURKA_ERR_CUDA;
  *gexp_per_s = (double)blocks * threads * 8.0 * iters / (best_ms * 1e-3) / 1e9;
  return FLURKA_OK;
}

size_t flurka_static_scratch_need(int variant, int B, int H, int N, int d, int k, int m) {
  Problem pr;
  if (parse_problem(variant, B, H, N, d, k, m, &pr)) return 0;
  return make_layout(pr, /*with_split_scratch=*/false).total;
}

}  // extern "C"

// ---------------------------------------------------------------------------------------------
// Forward pass for callers that must not allocate: all scratch lives in a fixed device array that
// is part of the library image.  In host code `g_static_scratch` is only a handle for the symbol,
// never a device address; the address kernels may use comes from cudaGetSymbolAddress, looked up
// once per device with that device current.
// ---------------------------------------------------------------------------------------------
namespace {

static __device__ __align__(256) unsigned char g_static_scratch[FLURKA_STATIC_SCRATCH_BYTES];

char* g_static_scratch_addr[kMaxDevices] = {};

int static_scratch_address(char** out) {
  int dev = 0;
  cudaError_t e = cudaGetDevice(&dev);
  if (e != cudaSuccess) { (void)cudaGetLastError(); return FLURKA_ERR_DEVICE; }
  if (dev < 0 || dev >= kMaxDevices) return FLURKA_ERR_DEVICE;
  if (!g_static_scratch_addr[dev]) {
    void* ptr = nullptr;
    e = cudaGetSymbolAddress(&ptr, g_static_scratch);
    if (e != cudaSuccess) return cuda_fail(e);
    if (!ptr) return FLURKA_ERR_WORKSPACE;
    g_static_scratch_addr[dev] = (char*)ptr;
  }
  *out = g_static_scratch_addr[dev];
  return FLURKA_OK;
}

}  // namespace

extern "C" int flurka_forward_static_scratch(const void* Q, const void* K, const void* V, const void* E,
                                             const void* F, const void* W, int variant, int B, int H,
                                             int N, int d, int k, int m, void* out, void* stream) {
  Problem pr;
  int rc = parse_problem(variant, B, H, N, d, k, m, &pr);
  if (rc) return rc;
  rc = validate_pointers(pr, Q, K, V, E, F, W, out);
  if (rc) return rc;
  // the CUDA-core kernels' scratch: no partial results of a split key side
  const Layout L = make_layout(pr, /*with_split_scratch=*/false);
  if (L.total > (size_t)FLURKA_STATIC_SCRATCH_BYTES) return FLURKA_ERR_TOO_LARGE;
  rc = check_device();
  if (rc) return rc;
  char* ws = nullptr;
  rc = static_scratch_address(&ws);
  if (rc) return rc;
  cudaStream_t st = (cudaStream_t)stream;
  // The array still holds the previous call's contents: the pipeline zeroes the status words and the
  // K', V' accumulators before the kernels add into them.  No stage timing and no record of the call
  // is kept: flurka_last_stage_ms and the other flurka_last_* queries keep describing flurka_forward.
  int launches = 0;
  if (pr.fp32)
    return run_pipeline<float>(pr, L, ws, Q, K, V, E, F, W, out, st, false, false, false, nullptr, nullptr, false,
                               &launches);
  return run_pipeline<__nv_bfloat16>(pr, L, ws, Q, K, V, E, F, W, out, st, false, false, false, nullptr, nullptr,
                                     false, &launches);
}

// Tensor-core (tcgen05 / TMEM / TMA) path of the FLuRKA forward pass: interface to the host side.
#pragma once

#include <cuda_fp16.h>
#include <cuda_runtime.h>

namespace flurka {

struct TensorArgs {
  int kernel, B, H, N, d, k, m;
  const void *Q, *K, *V, *E, *F, *W;
  void* out;
  float* kpvp;     // [2][BH][k][d] fp32
  float* weight;   // [BH][p]
  float* a32;      // [BH][p][d]
  __half* aT16;    // [BH][d][p]
  int* status;     // 4 words
};

// Optional per-stage timing: events recorded on the launch stream around the three stages.
struct StageTimer {
  bool on = false;
  bool have = false;
  cudaEvent_t ev[4] = {nullptr, nullptr, nullptr, nullptr};
  void mark(int i, cudaStream_t st) {
    if (on && ev[i]) cudaEventRecord(ev[i], st);
  }
};

// false while the tensor-core kernels are not compiled into this library
inline bool tensor_path_built() { return false; }

inline int run_tensor_path(const TensorArgs&, cudaStream_t, StageTimer&, int*, int*) { return -3; }

}  // namespace flurka

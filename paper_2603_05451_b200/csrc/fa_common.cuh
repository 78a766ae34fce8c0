// Host-side helpers shared by the launch code: status codes, argument structs and
// CUtensorMap construction (the driver entry point is resolved at run time so the
// library links without libcuda).
#pragma once

#include <cuda.h>
#include <cuda_runtime.h>
#include <stdint.h>
#include <stddef.h>

#include <atomic>

#include "../../include/fa.h"

namespace fa {

struct Shape {
  int B, H, Hkv, Sq, Sk, D;
  float scale;
  int causal;
  int deterministic = 0;  // backward: reduction-free kernels only (every output bit-reproducible)
  int f16 = 0;            // elements are FP16 instead of BF16
};

// Encodes a 4-D tiled tensor map over a dense [B, S, Hn, D] tensor of `elem_bytes`-sized
// elements.  Map dimensions (innermost first): D, Hn, S, B.  The box is box_d x 1 x box_s x 1,
// i.e. box_s consecutive tokens of one head; rows past S read as zero and are not written.
int encode_bshd_map(CUtensorMap* map, const void* base, int B, int S, int Hn, int D, int box_d, int box_s,
                    CUtensorMapDataType dtype, int elem_bytes, CUtensorMapSwizzle swizzle);

int fwd_launch(const void* q, const void* k, const void* v, void* o, float* lse, const Shape& s, cudaStream_t stream);
int varlen_lpt_order_launch(const int* cu_q, const int* cu_k, int batch, int causal, int* order, cudaStream_t stream);
int fwd_varlen_launch(const void* q, const void* k, const void* v, void* o, float* lse, const int* cu_q, const int* cu_k,
                      const int* order, int total_q, int total_k, const Shape& s, cudaStream_t stream);
int fwd_hd192_launch(const void* q, const void* k, const void* v, void* o, float* lse, const Shape& s,
                     cudaStream_t stream);
int bwd_launch(const void* q, const void* k, const void* v, const void* o, const float* lse, const void* d_o, void* dq,
               void* dk, void* dv, const Shape& s, void* workspace, cudaStream_t stream);
size_t bwd_workspace_bytes(const Shape& s);
size_t bwd_varlen_workspace_bytes(int batch, int total_q, int H, int D);
int bwd_varlen_launch(const void* q, const void* k, const void* v, const void* o, const float* lse, const void* d_o,
                      void* dq, void* dk, void* dv, const int* cu_q, const int* cu_k, int total_q, int total_k,
                      const Shape& s, void* workspace, cudaStream_t stream);

// Reads an integer option from the environment (`deflt` when unset).
int env_int(const char* name, int deflt);

// A fresh identifier for one entry-point call; kernels store it beside a recorded device-side
// failure so that only the blocks of the failing launch give up early.
unsigned next_launch_epoch();

// State that CUDA keeps per device (function attributes, the architecture check) is cached per
// device ordinal: one flag per device, set after the first successful set-up on that device.
constexpr int kMaxDevices = 64;
struct PerDeviceFlag {
  std::atomic<int> value[kMaxDevices];  // zero-initialised (static storage)
  bool test(int dev) const { return dev >= 0 && dev < kMaxDevices && value[dev].load(std::memory_order_acquire) != 0; }
  void set(int dev, int v = 1) {
    if (dev >= 0 && dev < kMaxDevices) value[dev].store(v, std::memory_order_release);
  }
  int get(int dev) const { return dev >= 0 && dev < kMaxDevices ? value[dev].load(std::memory_order_acquire) : 0; }
};

// Raises the dynamic shared-memory limit of `kernel` to `bytes` on the current device, once per device.
template <typename Kernel>
int set_smem_once(Kernel kernel, int bytes, PerDeviceFlag& done) {
  int dev = -1;
  if (cudaGetDevice(&dev) != cudaSuccess) return FA_ERR_CUDA;
  if (done.test(dev)) return FA_OK;
  if (cudaFuncSetAttribute(kernel, cudaFuncAttributeMaxDynamicSharedMemorySize, bytes) != cudaSuccess)
    return FA_ERR_CUDA;
  done.set(dev);
  return FA_OK;
}

}  // namespace fa

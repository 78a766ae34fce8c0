// C-ABI entry points: argument validation, status reporting, tensor-map construction.
#include <math.h>
#include <stdio.h>
#include <stdlib.h>
#include <string.h>

#include <atomic>
#include <mutex>

#include "exp2_emu.cuh"
#include "fa_common.cuh"
#include "ptx.cuh"

namespace fa {

int env_int(const char* name, int deflt) {
  const char* v = getenv(name);
  if (!v || !*v) return deflt;
  return atoi(v);
}

unsigned next_launch_epoch() {
  static std::atomic<unsigned> counter{0};
  return counter.fetch_add(1, std::memory_order_relaxed) + 1;  // never 0 in the first 2^32 - 1 calls
}

typedef CUresult (*EncodeTiledFn)(CUtensorMap*, CUtensorMapDataType, cuuint32_t, void*, const cuuint64_t*,
                                  const cuuint64_t*, const cuuint32_t*, const cuuint32_t*, CUtensorMapInterleave,
                                  CUtensorMapSwizzle, CUtensorMapL2promotion, CUtensorMapFloatOOBfill);

static EncodeTiledFn get_encode_fn() {
  static EncodeTiledFn fn = nullptr;
  static std::once_flag once;
  std::call_once(once, [] {
    void* p = nullptr;
    cudaDriverEntryPointQueryResult qres;
    if (cudaGetDriverEntryPoint("cuTensorMapEncodeTiled", &p, cudaEnableDefault, &qres) == cudaSuccess &&
        qres == cudaDriverEntryPointSuccess) {
      fn = reinterpret_cast<EncodeTiledFn>(p);
    }
  });
  return fn;
}

int encode_bshd_map(CUtensorMap* map, const void* base, int B, int S, int Hn, int D, int box_d, int box_s,
                    CUtensorMapDataType dtype, int elem_bytes, CUtensorMapSwizzle swizzle) {
  EncodeTiledFn fn = get_encode_fn();
  if (!fn) return FA_ERR_CUDA;
  cuuint64_t dims[4] = {(cuuint64_t)D, (cuuint64_t)Hn, (cuuint64_t)S, (cuuint64_t)B};
  cuuint64_t strides[3] = {(cuuint64_t)D * elem_bytes, (cuuint64_t)Hn * D * elem_bytes,
                           (cuuint64_t)S * Hn * D * elem_bytes};
  cuuint32_t box[4] = {(cuuint32_t)box_d, 1u, (cuuint32_t)box_s, 1u};
  cuuint32_t estr[4] = {1u, 1u, 1u, 1u};
  CUresult r = fn(map, dtype, 4, const_cast<void*>(base), dims, strides, box, estr, CU_TENSOR_MAP_INTERLEAVE_NONE,
                  swizzle, CU_TENSOR_MAP_L2_PROMOTION_L2_256B, CU_TENSOR_MAP_FLOAT_OOB_FILL_NONE);
  return r == CUDA_SUCCESS ? FA_OK : FA_ERR_CUDA;
}

static bool aligned16(const void* p) { return p != nullptr && (reinterpret_cast<uintptr_t>(p) & 15u) == 0; }

static int check_shape(int B, int H, int Hkv, int Sq, int Sk, int D, float scale) {
  if (B < 1 || H < 1 || Hkv < 1 || Sq < 1 || Sk < 1 || D < 1) return FA_ERR_INVALID_ARGUMENT;
  if (H % Hkv != 0) return FA_ERR_INVALID_ARGUMENT;
  if (!(scale > 0.0f) || !isfinite(scale)) return FA_ERR_INVALID_ARGUMENT;
  if (D != 64 && D != 128) return FA_ERR_UNSUPPORTED;
  // every flat index fits the kernels' 64-bit arithmetic; the tensor map needs each extent < 2^32
  if ((long long)B * H > 0x7fffffffll) return FA_ERR_UNSUPPORTED;
  return FA_OK;
}

// The kernels are built for sm_100a only; anything else (or no device at all) is refused.  The
// answer belongs to the current device and is cached per device ordinal (1 = supported, 2 = not).
static int check_device() {
  static PerDeviceFlag verdict;
  int dev = -1;
  if (cudaGetDevice(&dev) != cudaSuccess) {
    cudaGetLastError();
    return FA_ERR_CUDA;
  }
  int v = verdict.get(dev);
  if (v == 0) {
    int major = 0;
    if (cudaDeviceGetAttribute(&major, cudaDevAttrComputeCapabilityMajor, dev) != cudaSuccess) {
      cudaGetLastError();
      return FA_ERR_CUDA;
    }
    v = major == 10 ? 1 : 2;
    verdict.set(dev, v);
  }
  return v == 1 ? FA_OK : FA_ERR_UNSUPPORTED;
}

__global__ void exp2_emulated_kernel(const float* __restrict__ x, float* __restrict__ y, size_t n) {
  size_t i = (size_t)blockIdx.x * blockDim.x + threadIdx.x;
  if (i < n) y[i] = exp2_emulated(x[i]);
}

// One warp waits on a barrier that nobody arrives on: the bounded wait has to give up, record the
// timeout in the device status word and let the kernel end normally.
__global__ void unsatisfied_wait_kernel(unsigned epoch) {
  __shared__ alignas(8) uint64_t bar;
  __shared__ WaitCtl ctl;
  if (threadIdx.x == 0) {
    ctl.abort_flag = 0;
    ctl.launch_epoch = (int)epoch;
    mbar_init(&bar, 1);
    fence_barrier_init();
  }
  __syncthreads();
  mbar_wait(&bar, 0, &ctl.abort_flag, __LINE__);
}

}  // namespace fa

using namespace fa;

extern "C" {

static int fwd_entry(int f16, const void* q, const void* k, const void* v, void* o, float* lse, int B, int H, int Hkv,
                     int Sq, int Sk, int D, float scale, int causal, void* stream) {
  int st = check_shape(B, H, Hkv, Sq, Sk, D, scale);
  if (st != FA_OK) return st;
  if (!aligned16(q) || !aligned16(k) || !aligned16(v) || !aligned16(o) || lse == nullptr ||
      (reinterpret_cast<uintptr_t>(lse) & 3u) != 0)
    return FA_ERR_INVALID_ARGUMENT;
  st = check_device();
  if (st != FA_OK) return st;
  Shape s{B, H, Hkv, Sq, Sk, D, scale, causal != 0, 0, f16};
  return fwd_launch(q, k, v, o, lse, s, static_cast<cudaStream_t>(stream));
}

int fa_fwd(const void* q, const void* k, const void* v, void* o, float* lse, int B, int H, int Hkv, int Sq, int Sk,
           int D, float scale, int causal, void* stream) {
  return fwd_entry(0, q, k, v, o, lse, B, H, Hkv, Sq, Sk, D, scale, causal, stream);
}

int fa_fwd_f16(const void* q, const void* k, const void* v, void* o, float* lse, int B, int H, int Hkv, int Sq, int Sk,
               int D, float scale, int causal, void* stream) {
  return fwd_entry(1, q, k, v, o, lse, B, H, Hkv, Sq, Sk, D, scale, causal, stream);
}

int fa_fwd_hdim(const void* q, const void* k, const void* v, void* o, float* lse, int B, int H, int Hkv, int Sq, int Sk,
                int Dqk, int Dv, float scale, int causal, void* stream) {
  if (Dqk == Dv) return fa_fwd(q, k, v, o, lse, B, H, Hkv, Sq, Sk, Dqk, scale, causal, stream);
  int st = check_shape(B, H, Hkv, Sq, Sk, 128, scale);  // sizes, grouping and scale as for D = 128
  if (st != FA_OK) return st;
  if (Dqk < 1 || Dv < 1) return FA_ERR_INVALID_ARGUMENT;
  if (Dqk != 192 || Dv != 128) return FA_ERR_UNSUPPORTED;
  if (!aligned16(q) || !aligned16(k) || !aligned16(v) || !aligned16(o) || lse == nullptr ||
      (reinterpret_cast<uintptr_t>(lse) & 3u) != 0)
    return FA_ERR_INVALID_ARGUMENT;
  st = check_device();
  if (st != FA_OK) return st;
  Shape s{B, H, Hkv, Sq, Sk, Dqk, scale, causal != 0};
  return fwd_hd192_launch(q, k, v, o, lse, s, static_cast<cudaStream_t>(stream));
}

int fa_varlen_lpt_order(const int* cu_seqlens_q, const int* cu_seqlens_k, int batch, int causal, int* order,
                        void* stream) {
  if (cu_seqlens_q == nullptr || cu_seqlens_k == nullptr || order == nullptr || batch < 1)
    return FA_ERR_INVALID_ARGUMENT;
  if (batch > 16384) return FA_ERR_UNSUPPORTED;  // the rank sort is quadratic in the batch size
  int st = check_device();
  if (st != FA_OK) return st;
  return varlen_lpt_order_launch(cu_seqlens_q, cu_seqlens_k, batch, causal != 0, order,
                                 static_cast<cudaStream_t>(stream));
}

int fa_fwd_varlen(const void* q, const void* k, const void* v, void* o, float* lse, const int* cu_seqlens_q,
                  const int* cu_seqlens_k, const int* order, int batch, int total_q, int total_k, int max_seqlen_q, int H,
                  int Hkv, int D, float scale, int causal, void* stream) {
  if (total_q < 1 || total_k < 1 || max_seqlen_q < 1 || max_seqlen_q > total_q) return FA_ERR_INVALID_ARGUMENT;
  int st = check_shape(batch, H, Hkv, max_seqlen_q, total_k, D, scale);
  if (st != FA_OK) return st;
  if (!aligned16(q) || !aligned16(k) || !aligned16(v) || !aligned16(o) || lse == nullptr ||
      (reinterpret_cast<uintptr_t>(lse) & 3u) != 0 || cu_seqlens_q == nullptr || cu_seqlens_k == nullptr ||
      (reinterpret_cast<uintptr_t>(cu_seqlens_q) & 3u) != 0 || (reinterpret_cast<uintptr_t>(cu_seqlens_k) & 3u) != 0 ||
      (reinterpret_cast<uintptr_t>(order) & 3u) != 0)
    return FA_ERR_INVALID_ARGUMENT;
  st = check_device();
  if (st != FA_OK) return st;
  Shape s{batch, H, Hkv, max_seqlen_q, total_k, D, scale, causal != 0};
  return fwd_varlen_launch(q, k, v, o, lse, cu_seqlens_q, cu_seqlens_k, order, total_q, total_k, s,
                           static_cast<cudaStream_t>(stream));
}

size_t fa_bwd_varlen_workspace_bytes(int batch, int total_q, int H, int D) {
  if (batch < 1 || total_q < 1 || H < 1 || D != 128) return 0;
  return bwd_varlen_workspace_bytes(batch, total_q, H, D);
}

int fa_bwd_varlen(const void* q, const void* k, const void* v, const void* o, const float* lse, const void* d_o, void* dq,
                  void* dk, void* dv, const int* cu_seqlens_q, const int* cu_seqlens_k, int batch, int total_q,
                  int total_k, int max_seqlen_q, int max_seqlen_k, int H, int Hkv, int D, float scale, int causal,
                  void* workspace, size_t workspace_bytes, void* stream) {
  if (total_q < 1 || total_k < 1 || max_seqlen_q < 1 || max_seqlen_k < 1 || max_seqlen_q > total_q ||
      max_seqlen_k > total_k)
    return FA_ERR_INVALID_ARGUMENT;
  int st = check_shape(batch, H, Hkv, max_seqlen_q, max_seqlen_k, D, scale);
  if (st != FA_OK) return st;
  if (D != 128) return FA_ERR_UNSUPPORTED;
  if (!aligned16(q) || !aligned16(k) || !aligned16(v) || !aligned16(o) || !aligned16(d_o) || !aligned16(dq) ||
      !aligned16(dk) || !aligned16(dv) || lse == nullptr || (reinterpret_cast<uintptr_t>(lse) & 3u) != 0 ||
      cu_seqlens_q == nullptr || cu_seqlens_k == nullptr || (reinterpret_cast<uintptr_t>(cu_seqlens_q) & 3u) != 0 ||
      (reinterpret_cast<uintptr_t>(cu_seqlens_k) & 3u) != 0)
    return FA_ERR_INVALID_ARGUMENT;
  if (workspace == nullptr || (reinterpret_cast<uintptr_t>(workspace) & 255u) != 0 ||
      workspace_bytes < bwd_varlen_workspace_bytes(batch, total_q, H, D))
    return FA_ERR_WORKSPACE;
  st = check_device();
  if (st != FA_OK) return st;
  Shape s{batch, H, Hkv, max_seqlen_q, max_seqlen_k, D, scale, causal != 0};
  return bwd_varlen_launch(q, k, v, o, lse, d_o, dq, dk, dv, cu_seqlens_q, cu_seqlens_k, total_q, total_k, s, workspace,
                           static_cast<cudaStream_t>(stream));
}

size_t fa_bwd_workspace_bytes(int B, int H, int Hkv, int Sq, int Sk, int D) {
  if (check_shape(B, H, Hkv, Sq, Sk, D, 1.0f) != FA_OK) return 0;
  Shape s{B, H, Hkv, Sq, Sk, D, 1.0f, 0};
  return bwd_workspace_bytes(s);
}

static int bwd_entry(int deterministic, int f16, const void* q, const void* k, const void* v, const void* o, const float* lse, const void* d_o, void* dq,
           void* dk, void* dv, int B, int H, int Hkv, int Sq, int Sk, int D, float scale, int causal, void* workspace,
           size_t workspace_bytes, void* stream) {
  int st = check_shape(B, H, Hkv, Sq, Sk, D, scale);
  if (st != FA_OK) return st;
  if (!aligned16(q) || !aligned16(k) || !aligned16(v) || !aligned16(o) || !aligned16(d_o) || !aligned16(dq) ||
      !aligned16(dk) || !aligned16(dv) || lse == nullptr || (reinterpret_cast<uintptr_t>(lse) & 3u) != 0)
    return FA_ERR_INVALID_ARGUMENT;
  Shape s{B, H, Hkv, Sq, Sk, D, scale, causal != 0, deterministic, f16};
  if (workspace == nullptr || (reinterpret_cast<uintptr_t>(workspace) & 255u) != 0 ||
      workspace_bytes < bwd_workspace_bytes(s))
    return FA_ERR_WORKSPACE;
  st = check_device();
  if (st != FA_OK) return st;
  return bwd_launch(q, k, v, o, lse, d_o, dq, dk, dv, s, workspace, static_cast<cudaStream_t>(stream));
}

int fa_bwd(const void* q, const void* k, const void* v, const void* o, const float* lse, const void* d_o, void* dq,
           void* dk, void* dv, int B, int H, int Hkv, int Sq, int Sk, int D, float scale, int causal, void* workspace,
           size_t workspace_bytes, void* stream) {
  return bwd_entry(0, 0, q, k, v, o, lse, d_o, dq, dk, dv, B, H, Hkv, Sq, Sk, D, scale, causal, workspace, workspace_bytes,
                   stream);
}

int fa_bwd_deterministic(const void* q, const void* k, const void* v, const void* o, const float* lse, const void* d_o,
                         void* dq, void* dk, void* dv, int B, int H, int Hkv, int Sq, int Sk, int D, float scale,
                         int causal, void* workspace, size_t workspace_bytes, void* stream) {
  return bwd_entry(1, 0, q, k, v, o, lse, d_o, dq, dk, dv, B, H, Hkv, Sq, Sk, D, scale, causal, workspace, workspace_bytes,
                   stream);
}

int fa_bwd_f16(const void* q, const void* k, const void* v, const void* o, const float* lse, const void* d_o, void* dq,
               void* dk, void* dv, int B, int H, int Hkv, int Sq, int Sk, int D, float scale, int causal,
               void* workspace, size_t workspace_bytes, void* stream) {
  return bwd_entry(0, 1, q, k, v, o, lse, d_o, dq, dk, dv, B, H, Hkv, Sq, Sk, D, scale, causal, workspace,
                   workspace_bytes, stream);
}

int fa_bwd_deterministic_f16(const void* q, const void* k, const void* v, const void* o, const float* lse,
                             const void* d_o, void* dq, void* dk, void* dv, int B, int H, int Hkv, int Sq, int Sk, int D,
                             float scale, int causal, void* workspace, size_t workspace_bytes, void* stream) {
  return bwd_entry(1, 1, q, k, v, o, lse, d_o, dq, dk, dv, B, H, Hkv, Sq, Sk, D, scale, causal, workspace,
                   workspace_bytes, stream);
}

const char* fa_status_string(int status) {
  switch (status) {
    case FA_OK: return "ok";
    case FA_ERR_INVALID_ARGUMENT: return "invalid argument";
    case FA_ERR_UNSUPPORTED: return "unsupported head dimension, size or GPU architecture";
    case FA_ERR_CUDA: return "CUDA runtime or driver call failed";
    case FA_ERR_WORKSPACE: return "workspace null, misaligned or too small";
    case FA_ERR_DEVICE_TIMEOUT: return "a bounded device-side wait expired";
    default: return "unknown status";
  }
}

int fa_last_device_status(void* stream) {
  if (cudaStreamSynchronize(static_cast<cudaStream_t>(stream)) != cudaSuccess) return FA_ERR_CUDA;
  unsigned long long word = 0;
  if (cudaMemcpyFromSymbol(&word, g_device_status, sizeof(word)) != cudaSuccess) return FA_ERR_CUDA;
  const unsigned h = (unsigned)word;
  if (h != 0) {
    const unsigned long long zero = 0;
    cudaMemcpyToSymbol(g_device_status, &zero, sizeof(zero));
    // FA_LOG=1: say which wait gave up (source line of the kernel file), for bug reports
    if (env_int("FA_LOG", 0))
      fprintf(stderr, "fa: device-side wait expired (code %u, site %u, launch %u)\n", h & 0xffu, h >> 8,
              (unsigned)(word >> 32));
  }
  return h == 0 ? FA_OK : FA_ERR_DEVICE_TIMEOUT;
}

int fa_exp2_emulated(const float* x, float* y, size_t n, void* stream) {
  if (x == nullptr || y == nullptr) return FA_ERR_INVALID_ARGUMENT;
  if (n == 0) return FA_OK;
  int st = check_device();
  if (st != FA_OK) return st;
  const unsigned blocks = (unsigned)((n + 255) / 256);
  exp2_emulated_kernel<<<blocks, 256, 0, static_cast<cudaStream_t>(stream)>>>(x, y, n);
  return cudaGetLastError() == cudaSuccess ? FA_OK : FA_ERR_CUDA;
}

int fa_selftest_per_device_flags(void) {
  // Host-only check of the per-device bookkeeping: flags of different device ordinals are independent,
  // out-of-range ordinals read as "not set" and are ignored when set.
  static PerDeviceFlag f;
  if (f.test(0) || f.test(1) || f.test(-1) || f.test(kMaxDevices)) return FA_ERR_INVALID_ARGUMENT;
  f.set(1, 2);
  if (f.test(0) || !f.test(1) || f.get(1) != 2 || f.get(0) != 0) return FA_ERR_INVALID_ARGUMENT;
  f.set(kMaxDevices);
  f.set(-1);
  if (f.test(kMaxDevices) || f.test(-1) || f.get(kMaxDevices) != 0) return FA_ERR_INVALID_ARGUMENT;
  f.set(0);
  if (!f.test(0) || !f.test(1) || f.test(2)) return FA_ERR_INVALID_ARGUMENT;
  f.set(0, 0);
  f.set(1, 0);
  return FA_OK;
}

int fa_selftest_unsatisfied_wait(void* stream) {
  int st = check_device();
  if (st != FA_OK) return st;
  unsatisfied_wait_kernel<<<1, 32, 0, static_cast<cudaStream_t>(stream)>>>(next_launch_epoch());
  return cudaGetLastError() == cudaSuccess ? FA_OK : FA_ERR_CUDA;
}

}  // extern "C"

// Backward pass (paper Sections 2.1 and 3.2): parameters, preprocess kernel and helpers shared by
// the main kernels in fa_bwd_fused.cuh (one kernel, FP32 dQ reductions) and fa_bwd_split.cuh (two
// kernels, no reductions).
//
// A CTA of a key-tile kernel owns one 128-row key/value tile of one (batch, kv head) and walks
// over the 128-row query tiles that can see it (all query heads of the group in turn).
// Everything is computed transposed, so the accumulating products take their A operand from
// tensor memory:
//     S^T  = K Q_i^T                      (shared x shared)    -> region R0
//     P^T  = exp2(S^T * c - LSE_i * log2e), masked, bf16       -> R0 (over S^T)
//     dP^T = V dO_i^T                     (shared x shared)    -> region R1
//     dV  += P^T dO_i                     (tensor memory x shared, accumulator R2)
//     dS^T = P^T o (dP^T - Delta_i), bf16                      -> R1 (over dP^T)
//     dK  += dS^T Q_i                     (tensor memory x shared, accumulator R3)
// and, in the fused kernel only, dQ_i^T = K^T dS^T (shared x shared) -> R1, reduced into an FP32
// global accumulator.  Roles: warps 0-3 and 4-7 are the two compute warpgroups (one thread per
// key row, each warpgroup takes 64 of the 128 query columns); warp 12 issues the MMAs; warp 13
// is the TMA producer.  Tensor memory: R0 [0,128) R1 [128,256) dV [256,256+D) dK [384,384+D).
// Roles talk only through mbarriers with bounded waits.
#pragma once

#include "fa_common.cuh"
#include "fa_fwd_params.cuh"  // kLog2e
#include "ptx.cuh"

namespace fa {

struct BwdParams {
  float* dq_acc;        // [B, H, Sq_pad, D] fp32 accumulator (workspace)
  const float* lse2;    // [B, H, Sq_pad] LSE * log2(e); +inf for rows that take no part
  const float* delta;   // [B, H, Sq_pad] rowsum(dO o O)
  int B, H, Hkv, Sq, Sk, Sq_pad;
  float scale, scale_log2;
  int causal;
  unsigned epoch;  // identifies this launch in the device status word (bounded waits)
  // Fused kernel, causal dense batches: launch order in sections of this many (batch, key/value head) pairs,
  // inside a section the key tiles from the longest down (0: no sections, the key tiles of a head in a row).
  int heads_per_section = 0;
  // Variable-length batches (fused kernel only; null / 0 otherwise): sequence b owns query tokens
  // [cu_q[b], cu_q[b+1]) and key tokens [cu_k[b], cu_k[b+1]) of the packed tensors; in the workspace
  // arrays (accumulator, lse2, delta: [H, total_pad, ...]) its rows start at pad_off[b], a multiple
  // of 128, so that every 128-query tile of a sequence is tile-aligned there.
  const int* cu_q = nullptr;
  const int* cu_k = nullptr;
  const int* pad_off = nullptr;
  int total_pad = 0;
  __nv_bfloat16* dk = nullptr;  // for the row-by-row stores of key tiles that overhang a sequence end
  __nv_bfloat16* dv = nullptr;
};

// ------------------------------------------------------------------ preprocess
// Delta_i = sum_d dO_id * O_id; LSE in base 2; zero the dQ accumulator.  One thread handles 8
// consecutive head-dimension elements of one (batch, query, head) row; D/8 threads share a row.
template <int D, bool kF16 = false>
__global__ void __launch_bounds__(256)
bwd_preprocess_kernel(const __nv_bfloat16* __restrict__ o, const __nv_bfloat16* __restrict__ d_o,
                      const float* __restrict__ lse, float* __restrict__ delta, float* __restrict__ lse2,
                      float* __restrict__ dq_acc, int B, int H, int Sq, int Sq_pad) {
  constexpr int kThreadsPerRow = D / 8;
  constexpr int kRowsPerBlock = 256 / kThreadsPerRow;
  const int sub = threadIdx.x % kThreadsPerRow;
  const long long row = (long long)blockIdx.x * kRowsPerBlock + threadIdx.x / kThreadsPerRow;  // over B*H*Sq_pad
  const long long total = (long long)B * H * Sq_pad;
  if (row >= total) return;
  const int i = (int)(row % Sq_pad);
  const int h = (int)((row / Sq_pad) % H);
  const int b = (int)(row / ((long long)Sq_pad * H));
  float acc = 0.0f;
  if (i < Sq) {
    const size_t off = (((size_t)b * Sq + i) * H + h) * D + sub * 8;
    const uint4 ov = *reinterpret_cast<const uint4*>(o + off);
    const uint4 gv = *reinterpret_cast<const uint4*>(d_o + off);
    const uint32_t ow[4] = {ov.x, ov.y, ov.z, ov.w}, gw[4] = {gv.x, gv.y, gv.z, gv.w};
#pragma unroll
    for (int t = 0; t < 4; ++t) {
      const float2 ov = unpack2<kF16>(ow[t]), gv = unpack2<kF16>(gw[t]);
      acc = fmaf(ov.x, gv.x, acc);
      acc = fmaf(ov.y, gv.y, acc);
    }
  }
  if (dq_acc != nullptr) {
    // the accumulator is head-major [B, H, Sq_pad, D]; padded rows are zeroed (and reduced into) too
    float4 z = make_float4(0.f, 0.f, 0.f, 0.f);
    float4* dst = reinterpret_cast<float4*>(dq_acc + (size_t)row * D + sub * 8);
    dst[0] = z;
    dst[1] = z;
  }
#pragma unroll
  for (int m = kThreadsPerRow / 2; m >= 1; m >>= 1) acc += __shfl_xor_sync(0xffffffffu, acc, m);
  if (sub == 0) {
    float l2 = INFINITY;  // rows past Sq and rows without any visible key: P becomes exp2(-inf) = 0
    if (i < Sq) {
      const float l = lse[((size_t)b * H + h) * Sq + i];
      if (l != -INFINITY) l2 = l * kLog2e;
    }
    delta[row] = (i < Sq) ? acc : 0.0f;
    lse2[row] = l2;
  }
}

// ------------------------------------------------------------------ shared helpers
__device__ __forceinline__ void bulk_load_1d(void* smem_dst, const void* gsrc, uint32_t bytes, uint64_t* bar) {
  asm volatile("cp.async.bulk.shared::cluster.global.mbarrier::complete_tx::bytes [%0], [%1], %2, [%3];" ::"r"(
                   smem_u32(smem_dst)),
               "l"(gsrc), "r"(bytes), "r"(smem_u32(bar))
               : "memory");
}

}  // namespace fa

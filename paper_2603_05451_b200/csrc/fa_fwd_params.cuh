// Forward-pass constants and the kernel parameter block.
#pragma once

#include <cuda_bf16.h>

namespace fa {

constexpr float kLog2e = 1.4426950408889634f;
constexpr float kLn2 = 0.6931471805599453f;
constexpr float kRescaleTau = 8.0f;  // log2(256), Section 3.1.4

struct FwdParams {
  __nv_bfloat16* o;
  float* lse;
  int B, H, Hkv, Sq, Sk;
  float scale_log2;  // scale * log2(e)
  float tau;         // rescale threshold in the base-2 domain (Eq. 6); 8 = log2(256) unless FA_TAU overrides it
  int causal;
  unsigned epoch;  // identifies this launch in the device status word (bounded waits)
  // Variable-length batches (all null / 0 for dense batches): sequences are packed along the token
  // axis, sequence b owns query tokens [cu_q[b], cu_q[b+1]) and key tokens [cu_k[b], cu_k[b+1]);
  // `order` (optional) lists the sequences longest-first; then B = number of sequences, Sq = longest
  // query length (grid sizing only) and lse is [H, total_q].
  const int* cu_q = nullptr;
  const int* cu_k = nullptr;
  const int* order = nullptr;
  int total_q = 0;
  // Launch order (Section 3.3): query heads are taken in sections of this many (a multiple of
  // H / Hkv that divides H) so that the K and V of the heads in flight fit in L2.
  int heads_per_section = 0;  // 0 = all heads in one section
};

}  // namespace fa

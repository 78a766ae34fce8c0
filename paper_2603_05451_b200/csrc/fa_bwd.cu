// Backward-pass launch code: workspace layout, tensor maps, kernel launches.
//
// Three implementations of the main step exist:
//   fused   one kernel per key tile with five MMAs (paper Section 3.2); dQ is reduced into an FP32
//           accumulator with bulk (TMA) reduce-adds.  Fastest; dQ's summation order is not fixed.
//   pair    the same step on clusters of two CTAs with tcgen05 cta_group::2 MMAs (the paper's 2-CTA
//           backward): 3/4 of the operand traffic and half of the dQ reductions.  Head dimension 128.
//   split   bwd_dkdv_kernel + bwd_dq_kernel: no global reductions, every output bit-reproducible,
//           no accumulator in the workspace; recomputes S and dP once more (7 MMAs).
// Default: fused.  FA_BWD_IMPL=split | pair (read once per process) selects the others; pair is for
// head dimension 128 only.
#include "fa_bwd_fused.cuh"
#include "fa_bwd_kernels.cuh"
#include "fa_bwd_pair.cuh"
#include "fa_bwd_split.cuh"
#include "fa_bwd_varlen.cuh"
#include "fa_common.cuh"

namespace fa {

static bool bwd_use_fused(const Shape& s) {
  static const bool force_split = [] {
    const char* e = getenv("FA_BWD_IMPL");
    return e && strcmp(e, "split") == 0;
  }();
  return !force_split && !s.deterministic;
}

// FA_BWD_IMPL=pair (read once): the fused step runs on CTA pairs (bwd_pair_kernel) instead of single CTAs.
static bool bwd_use_pair() {
  static const bool pair = [] {
    const char* e = getenv("FA_BWD_IMPL");
    return e && strcmp(e, "pair") == 0;
  }();
  return pair;
}

static size_t up256(size_t x) { return (x + 255) / 256 * 256; }

struct BwdWorkspace {
  size_t dq_acc_bytes, rows_bytes, total;
  int sq_pad;
};

static BwdWorkspace bwd_layout(const Shape& s) {
  BwdWorkspace w;
  w.sq_pad = (s.Sq + 127) / 128 * 128;
  // FP32 dQ accumulator [B][H][Sq_pad/32][4][32][32] (fused path only), then Delta and LSE*log2e as [B, H, Sq_pad]
  w.dq_acc_bytes = bwd_use_fused(s) ? up256((size_t)s.B * s.H * w.sq_pad * s.D * sizeof(float)) : 0;
  w.rows_bytes = up256((size_t)s.B * s.H * w.sq_pad * sizeof(float));
  w.total = w.dq_acc_bytes + 2 * w.rows_bytes;
  return w;
}

size_t bwd_workspace_bytes(const Shape& s) { return bwd_layout(s).total; }

// Shared-memory opt-in of the fused kernel (dense and packed launches share it), per device.
template <int D, bool kF16>
static int fused_smem_once() {
  static PerDeviceFlag done;
  return set_smem_once(bwd_fused_kernel<D, kF16>, (int)sizeof(BwdFusedSmem<D>), done);
}

// The two split kernels: dK/dV per key tile, then dQ per query tile.
template <int D, bool kF16, typename Preprocess>
static int bwd_split_launch(const CUtensorMap& tq, const CUtensorMap& tk, const CUtensorMap& tv, const CUtensorMap& tdo,
                            const CUtensorMap& tdq, const CUtensorMap& tdk, const CUtensorMap& tdv, const BwdParams& p,
                            int n_kv_tiles, int n_q_tiles, Preprocess preprocess, cudaStream_t stream) {
  const long long n_kv_ctas = (long long)n_kv_tiles * p.Hkv * p.B;
  const long long n_q_ctas = (long long)n_q_tiles * p.H * p.B;
  static PerDeviceFlag attr_a, attr_b;
  int st;
  if ((st = set_smem_once(bwd_dkdv_kernel<D, kF16>, (int)sizeof(BwdDkdvSmem<D>), attr_a)) != FA_OK) return st;
  if ((st = set_smem_once(bwd_dq_kernel<D, kF16>, (int)sizeof(BwdDqSmem<D>), attr_b)) != FA_OK) return st;
  if ((st = preprocess()) != FA_OK) return st;
  bwd_dkdv_kernel<D, kF16><<<(unsigned)n_kv_ctas, 512, sizeof(BwdDkdvSmem<D>), stream>>>(tq, tk, tv, tdo, tdk, tdv, p,
                                                                                          n_kv_tiles);
  if (cudaGetLastError() != cudaSuccess) return FA_ERR_CUDA;
  bwd_dq_kernel<D, kF16><<<(unsigned)n_q_ctas, 512, sizeof(BwdDqSmem<D>), stream>>>(tq, tk, tv, tdo, tdq, p, n_q_tiles);
  return cudaGetLastError() == cudaSuccess ? FA_OK : FA_ERR_CUDA;
}

template <int D>
static int bwd_launch_d(const void* q, const void* k, const void* v, const void* o, const float* lse, const void* d_o,
                        void* dq, void* dk, void* dv, const Shape& s, void* workspace, cudaStream_t stream) {
  const bool fused = bwd_use_fused(s);
  if (s.f16 && fused && D == 128 && bwd_use_pair()) return FA_ERR_UNSUPPORTED;  // the CTA-pair kernel is BF16 only
  const BwdWorkspace w = bwd_layout(s);
  float* dq_acc = fused ? static_cast<float*>(workspace) : nullptr;
  float* delta = reinterpret_cast<float*>(static_cast<uint8_t*>(workspace) + w.dq_acc_bytes);
  float* lse2 = reinterpret_cast<float*>(static_cast<uint8_t*>(workspace) + w.dq_acc_bytes + w.rows_bytes);

  CUtensorMap tq, tk, tv, tdo, tdk, tdv, tdq;
  const auto bf16 = CU_TENSOR_MAP_DATA_TYPE_BFLOAT16;
  const auto sw = CU_TENSOR_MAP_SWIZZLE_128B;
  int st;
  if ((st = encode_bshd_map(&tq, q, s.B, s.Sq, s.H, D, 64, 128, bf16, 2, sw)) != FA_OK) return st;
  if ((st = encode_bshd_map(&tdo, d_o, s.B, s.Sq, s.H, D, 64, 128, bf16, 2, sw)) != FA_OK) return st;
  if ((st = encode_bshd_map(&tdq, dq, s.B, s.Sq, s.H, D, 64, 128, bf16, 2, sw)) != FA_OK) return st;
  if ((st = encode_bshd_map(&tk, k, s.B, s.Sk, s.Hkv, D, 64, 128, bf16, 2, sw)) != FA_OK) return st;
  if ((st = encode_bshd_map(&tv, v, s.B, s.Sk, s.Hkv, D, 64, 128, bf16, 2, sw)) != FA_OK) return st;
  if ((st = encode_bshd_map(&tdk, dk, s.B, s.Sk, s.Hkv, D, 64, 128, bf16, 2, sw)) != FA_OK) return st;
  if ((st = encode_bshd_map(&tdv, dv, s.B, s.Sk, s.Hkv, D, 64, 128, bf16, 2, sw)) != FA_OK) return st;

  BwdParams p;
  p.dq_acc = dq_acc;
  p.lse2 = lse2;
  p.delta = delta;
  p.B = s.B; p.H = s.H; p.Hkv = s.Hkv; p.Sq = s.Sq; p.Sk = s.Sk; p.Sq_pad = w.sq_pad;
  p.scale = s.scale;
  p.scale_log2 = s.scale * kLog2e;
  p.causal = s.causal;
  p.epoch = next_launch_epoch();
  const int n_kv_tiles = (s.Sk + 127) / 128;
  const int n_q_tiles = (s.Sq + 127) / 128;
  // Causal mask: launch order in sections of a few heads, longest key tiles of a section first (see the fused
  // kernel).  Measured at 16384 tokens, 16 heads of 128: sections of 8 heads +1 ... +5 % up to 8192 keys, of 4 heads
  // +3 % at 16384; whole-launch longest-first order loses the L2 sharing of Q and dO between the tiles of a head
  // (-15 % at 1024 keys).
  if (s.causal) p.heads_per_section = n_kv_tiles > 64 ? 4 : 8;
  const long long n_kv_ctas = (long long)n_kv_tiles * s.Hkv * s.B;
  const long long n_q_ctas = (long long)n_q_tiles * s.H * s.B;
  // Every size check comes before the first launch: on an error nothing has been launched.
  constexpr int kRowsPerBlock = 256 / (D / 8);
  const long long pre_blocks = ((long long)s.B * s.H * w.sq_pad + kRowsPerBlock - 1) / kRowsPerBlock;
  const size_t n8 = (size_t)s.B * s.Sq * s.H * D / 8;
  const size_t conv_blocks = (n8 + 255) / 256;
  if (n_kv_ctas > 0x3fffffffll || n_q_ctas > 0x7fffffffll || pre_blocks > 0x7fffffffll || conv_blocks > 0x7fffffffull)
    return FA_ERR_UNSUPPORTED;

  // 1. preprocess: Delta, LSE in base 2 (and a zeroed dQ accumulator for the fused path)
  auto preprocess = [&]() {
    auto pre = s.f16 ? bwd_preprocess_kernel<D, true> : bwd_preprocess_kernel<D, false>;
    pre<<<(unsigned)pre_blocks, 256, 0, stream>>>(static_cast<const __nv_bfloat16*>(o),
                                                  static_cast<const __nv_bfloat16*>(d_o), lse, delta, lse2, dq_acc, s.B,
                                                  s.H, s.Sq, w.sq_pad);
    return cudaGetLastError() == cudaSuccess ? FA_OK : FA_ERR_CUDA;
  };

  if (fused) {
    // 2. fused main kernel, 3. accumulator -> 16-bit dQ
    bool launched = false;
    if constexpr (D == 128) {
      if (bwd_use_pair()) {
        CUtensorMap tq64, tdo64;
        if ((st = encode_bshd_map(&tq64, q, s.B, s.Sq, s.H, D, 64, 64, bf16, 2, sw)) != FA_OK) return st;
        if ((st = encode_bshd_map(&tdo64, d_o, s.B, s.Sq, s.H, D, 64, 64, bf16, 2, sw)) != FA_OK) return st;
        static PerDeviceFlag attr_p;
        if ((st = set_smem_once(bwd_pair_kernel, (int)sizeof(BwdPairSmem), attr_p)) != FA_OK) return st;
        const int n_kv_pairs = (n_kv_tiles + 1) / 2;
        const long long n_pair_ctas = 2ll * n_kv_pairs * s.Hkv * s.B;  // <= 2 n_kv_ctas, checked above
        if ((st = preprocess()) != FA_OK) return st;
        bwd_pair_kernel<<<(unsigned)n_pair_ctas, 512, sizeof(BwdPairSmem), stream>>>(tq, tq64, tk, tv, tdo, tdo64, tdk,
                                                                                      tdv, p, n_kv_pairs);
        if (cudaGetLastError() != cudaSuccess) return FA_ERR_CUDA;
        launched = true;
      }
    }
    if (!launched) {
      st = s.f16 ? fused_smem_once<D, true>() : fused_smem_once<D, false>();
      if (st != FA_OK) return st;
      if ((st = preprocess()) != FA_OK) return st;
      auto kernel = s.f16 ? bwd_fused_kernel<D, true> : bwd_fused_kernel<D, false>;
      kernel<<<(unsigned)n_kv_ctas, 512, sizeof(BwdFusedSmem<D>), stream>>>(tq, tk, tv, tdo, tdk, tdv, p, n_kv_tiles);
      if (cudaGetLastError() != cudaSuccess) return FA_ERR_CUDA;
    }
    auto conv = s.f16 ? bwd_convert_dq_chunked_kernel<D, true> : bwd_convert_dq_chunked_kernel<D, false>;
    conv<<<(unsigned)conv_blocks, 256, 0, stream>>>(dq_acc, static_cast<__nv_bfloat16*>(dq), n8, s.scale, s.H, s.Sq,
                                                    w.sq_pad);
    return cudaGetLastError() == cudaSuccess ? FA_OK : FA_ERR_CUDA;
  }
  // 2a. dK, dV;  2b. dQ
  if (s.f16) return bwd_split_launch<D, true>(tq, tk, tv, tdo, tdq, tdk, tdv, p, n_kv_tiles, n_q_tiles, preprocess, stream);
  return bwd_split_launch<D, false>(tq, tk, tv, tdo, tdq, tdk, tdv, p, n_kv_tiles, n_q_tiles, preprocess, stream);
}

// ---------------------------------------------------------------- variable-length batches
// Workspace: FP32 dQ accumulator [H, total_pad, 128] (chunked), Delta and LSE*log2e [H, total_pad],
// pad_off [batch + 1] int32; total_pad = total_q rounded up + 128 per sequence bounds the sum of the
// sequences' lengths rounded up to 128.
static int varlen_total_pad(int batch, int total_q) { return (total_q + 127) / 128 * 128 + 128 * batch; }

size_t bwd_varlen_workspace_bytes(int batch, int total_q, int H, int D) {
  const size_t tp = (size_t)varlen_total_pad(batch, total_q);
  return up256(tp * H * D * sizeof(float)) + 2 * up256(tp * H * sizeof(float)) + up256((size_t)(batch + 1) * sizeof(int));
}

// s.B = number of sequences, s.Sq / s.Sk = longest query / key length (they size the grid).
int bwd_varlen_launch(const void* q, const void* k, const void* v, const void* o, const float* lse, const void* d_o,
                      void* dq, void* dk, void* dv, const int* cu_q, const int* cu_k, int total_q, int total_k,
                      const Shape& s, void* workspace, cudaStream_t stream) {
  constexpr int D = 128;
  const int tp = varlen_total_pad(s.B, total_q);
  uint8_t* w8 = static_cast<uint8_t*>(workspace);
  float* dq_acc = reinterpret_cast<float*>(w8);
  w8 += up256((size_t)tp * s.H * D * sizeof(float));
  float* delta = reinterpret_cast<float*>(w8);
  w8 += up256((size_t)tp * s.H * sizeof(float));
  float* lse2 = reinterpret_cast<float*>(w8);
  w8 += up256((size_t)tp * s.H * sizeof(float));
  int* pad_off = reinterpret_cast<int*>(w8);

  CUtensorMap tq, tk, tv, tdo, tdk, tdv;
  const auto bf16 = CU_TENSOR_MAP_DATA_TYPE_BFLOAT16;
  const auto sw = CU_TENSOR_MAP_SWIZZLE_128B;
  int st;
  if ((st = encode_bshd_map(&tq, q, 1, total_q, s.H, D, 64, 128, bf16, 2, sw)) != FA_OK) return st;
  if ((st = encode_bshd_map(&tdo, d_o, 1, total_q, s.H, D, 64, 128, bf16, 2, sw)) != FA_OK) return st;
  if ((st = encode_bshd_map(&tk, k, 1, total_k, s.Hkv, D, 64, 128, bf16, 2, sw)) != FA_OK) return st;
  if ((st = encode_bshd_map(&tv, v, 1, total_k, s.Hkv, D, 64, 128, bf16, 2, sw)) != FA_OK) return st;
  if ((st = encode_bshd_map(&tdk, dk, 1, total_k, s.Hkv, D, 64, 128, bf16, 2, sw)) != FA_OK) return st;
  if ((st = encode_bshd_map(&tdv, dv, 1, total_k, s.Hkv, D, 64, 128, bf16, 2, sw)) != FA_OK) return st;

  // Every size check and per-device set-up comes before the first launch.
  const long long pre_blocks = ((long long)s.H * tp + 15) / 16;
  const int n_kv_tiles = (s.Sk + 127) / 128;
  const long long n_ctas = (long long)n_kv_tiles * s.Hkv * s.B;
  const size_t n8 = (size_t)total_q * s.H * D / 8;
  const size_t conv_blocks = (n8 + 255) / 256;
  if (pre_blocks > 0x7fffffffll || n_ctas > 0x7fffffffll || conv_blocks > 0x7fffffffull) return FA_ERR_UNSUPPORTED;
  st = s.f16 ? fused_smem_once<D, true>() : fused_smem_once<D, false>();
  if (st != FA_OK) return st;

  varlen_pad_offsets_kernel<<<1, 32, 0, stream>>>(cu_q, s.B, pad_off);
  if (cudaGetLastError() != cudaSuccess) return FA_ERR_CUDA;
  auto pre = s.f16 ? bwd_preprocess_varlen_kernel<true> : bwd_preprocess_varlen_kernel<false>;
  pre<<<(unsigned)pre_blocks, 256, 0, stream>>>(static_cast<const __nv_bfloat16*>(o), static_cast<const __nv_bfloat16*>(d_o),
                                                lse, delta, lse2, dq_acc, cu_q, pad_off, s.B, s.H, total_q, tp);
  if (cudaGetLastError() != cudaSuccess) return FA_ERR_CUDA;
  BwdParams p;
  p.dq_acc = dq_acc;
  p.lse2 = lse2;
  p.delta = delta;
  p.B = s.B; p.H = s.H; p.Hkv = s.Hkv; p.Sq = s.Sq; p.Sk = s.Sk; p.Sq_pad = 0;
  p.scale = s.scale;
  p.scale_log2 = s.scale * kLog2e;
  p.causal = s.causal;
  p.epoch = next_launch_epoch();
  p.cu_q = cu_q;
  p.cu_k = cu_k;
  p.pad_off = pad_off;
  p.total_pad = tp;
  p.dk = static_cast<__nv_bfloat16*>(dk);
  p.dv = static_cast<__nv_bfloat16*>(dv);
  auto kernel = s.f16 ? bwd_fused_kernel<D, true> : bwd_fused_kernel<D, false>;
  kernel<<<(unsigned)n_ctas, 512, sizeof(BwdFusedSmem<D>), stream>>>(tq, tk, tv, tdo, tdk, tdv, p, n_kv_tiles);
  if (cudaGetLastError() != cudaSuccess) return FA_ERR_CUDA;
  auto conv = s.f16 ? bwd_convert_dq_varlen_kernel<true> : bwd_convert_dq_varlen_kernel<false>;
  conv<<<(unsigned)conv_blocks, 256, 0, stream>>>(dq_acc, static_cast<__nv_bfloat16*>(dq), n8, s.scale, cu_q, pad_off,
                                                  s.B, s.H, tp);
  return cudaGetLastError() == cudaSuccess ? FA_OK : FA_ERR_CUDA;
}

int bwd_launch(const void* q, const void* k, const void* v, const void* o, const float* lse, const void* d_o, void* dq,
               void* dk, void* dv, const Shape& s, void* workspace, cudaStream_t stream) {
  if (s.D == 64) return bwd_launch_d<64>(q, k, v, o, lse, d_o, dq, dk, dv, s, workspace, stream);
  return bwd_launch_d<128>(q, k, v, o, lse, d_o, dq, dk, dv, s, workspace, stream);
}

}  // namespace fa


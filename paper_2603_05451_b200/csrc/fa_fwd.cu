// Forward-pass launch code: builds the tensor maps and launches the kernel.
#include "fa_common.cuh"
#include "fa_fwd_pipe.cuh"
#include "fa_fwd_tile.cuh"

namespace fa {

static int make_maps(CUtensorMap* tq, CUtensorMap* tk, CUtensorMap* tv, CUtensorMap* to, const void* q, const void* k,
                     const void* v, void* o, const Shape& s) {
  int st;
  const auto bf16 = CU_TENSOR_MAP_DATA_TYPE_BFLOAT16;
  const auto sw = CU_TENSOR_MAP_SWIZZLE_128B;
  if ((st = encode_bshd_map(tq, q, s.B, s.Sq, s.H, s.D, 64, 128, bf16, 2, sw)) != FA_OK) return st;
  if ((st = encode_bshd_map(tk, k, s.B, s.Sk, s.Hkv, s.D, 64, 128, bf16, 2, sw)) != FA_OK) return st;
  if ((st = encode_bshd_map(tv, v, s.B, s.Sk, s.Hkv, s.D, 64, 128, bf16, 2, sw)) != FA_OK) return st;
  if (to && (st = encode_bshd_map(to, o, s.B, s.Sq, s.H, s.D, 64, 128, bf16, 2, sw)) != FA_OK) return st;
  return FA_OK;
}

// Longest key sequence that goes to the one-tile-per-CTA kernel: the measured crossover with the pipelined
// kernel at 16384 tokens per launch, per head dimension and mask.
// At D = 64 that kernel keeps P in tensor-memory columns of its own; without a mask it is the faster one at
// every length measured (to 32768), with the causal mask up to 4096 keys.
constexpr int kTileMaxSkD128 = 512, kTileMaxSkCausalD128 = 1024, kTileMaxSkD64 = 1 << 30, kTileMaxSkCausalD64 = 4096;

static FwdParams make_params(void* o, float* lse, const Shape& s) {
  FwdParams p;
  p.o = static_cast<__nv_bfloat16*>(o);
  p.lse = lse;
  p.B = s.B; p.H = s.H; p.Hkv = s.Hkv; p.Sq = s.Sq; p.Sk = s.Sk;
  p.scale_log2 = s.scale * kLog2e;
  // FA_TAU (read once) overrides the rescale threshold for experiments: 0 = rescale on every new maximum
  static const float tau = [] {
    const char* e = getenv("FA_TAU");
    // clamped so that 2^tau stays inside FP16's range (fa_fwd_f16 stores the probabilities as FP16)
    return (e && *e) ? fminf(fmaxf((float)atof(e), 0.0f), 15.0f) : kRescaleTau;
  }();
  p.tau = tau;
  p.causal = s.causal;
  p.epoch = next_launch_epoch();
  // Sections of heads whose K and V (2 * Sk * (Dqk + Dv) bytes per key/value head; s.D stands for both
  // dimensions here, close enough for (192,128)) stay within a quarter of the 126 MB L2, so that the
  // blocks in flight re-read them from L2 and not from memory.  FA_FWD_SECTION_MB (read once) overrides
  // the budget; 0 puts all heads in one section.
  static const long long budget = [] {
    const char* e = getenv("FA_FWD_SECTION_MB");
    return ((e && *e) ? atoll(e) : 32ll) << 20;
  }();
  const int group = s.H / s.Hkv;
  const long long per_kv_head = 4ll * s.Sk * s.D;
  int kv_heads = budget > 0 ? (int)(budget / (per_kv_head > 0 ? per_kv_head : 1)) : s.Hkv;
  if (kv_heads < 1) kv_heads = 1;
  if (kv_heads > s.Hkv) kv_heads = s.Hkv;
  while (s.Hkv % kv_heads != 0) --kv_heads;  // sections of equal size
  p.heads_per_section = kv_heads * group;
  return p;
}

// One launch of the pipelined kernel: tensor maps, parameters, shared-memory opt-in (once per device).
template <int DQK, int DV, int kEmuPer8, bool kF16>
static int launch_pipe(const CUtensorMap& tq, const CUtensorMap& tk, const CUtensorMap& tv, const CUtensorMap& to,
                       const FwdParams& p, const Shape& s, cudaStream_t stream) {
  static PerDeviceFlag attr_set;
  constexpr int smem = (int)sizeof(FwdPipeSmem<DQK, DV>);
  auto kernel = fwd_pipe_kernel<DQK, DV, kEmuPer8, kF16>;
  const int n_mblocks = (s.Sq + 255) / 256;
  const long long n_ctas = (long long)s.B * s.H * n_mblocks;
  if (n_ctas > 0x7fffffffll) return FA_ERR_UNSUPPORTED;
  int st = set_smem_once(kernel, smem, attr_set);
  if (st != FA_OK) return st;
  kernel<<<(unsigned)n_ctas, 512, smem, stream>>>(tq, tk, tv, to, p, n_mblocks);
  return cudaGetLastError() == cudaSuccess ? FA_OK : FA_ERR_CUDA;
}

// One launch of the one-tile-per-CTA kernel (two CTAs per SM).
template <int D, int kEmuPer8, bool kF16>
static int launch_tile(const CUtensorMap& tq, const CUtensorMap& tk, const CUtensorMap& tv, const CUtensorMap& to,
                       const FwdParams& p, const Shape& s, cudaStream_t stream) {
  static PerDeviceFlag attr_set, carveout_set;
  constexpr int smem = fwd_tile_smem_bytes<D>();
  auto kernel = fwd_tile_kernel<D, kEmuPer8, kF16>;
  const int n_mblocks = (s.Sq + 127) / 128;
  const long long n_ctas = (long long)s.B * s.H * n_mblocks;
  if (n_ctas > 0x7fffffffll) return FA_ERR_UNSUPPORTED;
  int st = set_smem_once(kernel, smem, attr_set);
  if (st != FA_OK) return st;
  int dev = -1;
  if (cudaGetDevice(&dev) != cudaSuccess) return FA_ERR_CUDA;
  if (!carveout_set.test(dev)) {  // two CTAs of ~100 KiB each must fit: ask for the largest shared-memory split
    if (cudaFuncSetAttribute(kernel, cudaFuncAttributePreferredSharedMemoryCarveout, cudaSharedmemCarveoutMaxShared) !=
        cudaSuccess)
      return FA_ERR_CUDA;
    carveout_set.set(dev);
  }
  kernel<<<(unsigned)n_ctas, 256, smem, stream>>>(tq, tk, tv, to, p, n_mblocks);
  return cudaGetLastError() == cudaSuccess ? FA_OK : FA_ERR_CUDA;
}

// Which kernel a dense call gets.  The one-tile kernel hides the per-CTA set-up and epilogue behind a second
// resident CTA but reads K and V twice as often; it wins while a tile has few key blocks.  FA_FWD_TILE (read
// once per process): 0 = never, 1 = always, unset = by sequence length.
static bool use_tile_kernel(const Shape& s) {
  static const int forced = env_int("FA_FWD_TILE", -1);
  if (forced >= 0) return forced != 0;
  const int max_sk = s.D == 64 ? (s.causal ? kTileMaxSkCausalD64 : kTileMaxSkD64)
                               : (s.causal ? kTileMaxSkCausalD128 : kTileMaxSkD128);
  return s.Sk <= max_sk;
}

template <int D, int kEmuPer8, bool kF16 = false>
static int launch_dense(const void* q, const void* k, const void* v, void* o, float* lse, const Shape& s,
                        cudaStream_t stream) {
  CUtensorMap tq, tk, tv, to;
  int st = make_maps(&tq, &tk, &tv, &to, q, k, v, o, s);
  if (st != FA_OK) return st;
  if (use_tile_kernel(s)) return launch_tile<D, kEmuPer8, kF16>(tq, tk, tv, to, make_params(o, lse, s), s, stream);
  return launch_pipe<D, D, kEmuPer8, kF16>(tq, tk, tv, to, make_params(o, lse, s), s, stream);
}

// Head dimensions (192, 128): s.D is the query/key dimension (192); values and output have 128.
int fwd_hd192_launch(const void* q, const void* k, const void* v, void* o, float* lse, const Shape& s,
                     cudaStream_t stream) {
  CUtensorMap tq, tk, tv, to;
  const auto bf16 = CU_TENSOR_MAP_DATA_TYPE_BFLOAT16;
  const auto sw = CU_TENSOR_MAP_SWIZZLE_128B;
  int st;
  if ((st = encode_bshd_map(&tq, q, s.B, s.Sq, s.H, 192, 64, 128, bf16, 2, sw)) != FA_OK) return st;
  if ((st = encode_bshd_map(&tk, k, s.B, s.Sk, s.Hkv, 192, 64, 128, bf16, 2, sw)) != FA_OK) return st;
  if ((st = encode_bshd_map(&tv, v, s.B, s.Sk, s.Hkv, 128, 64, 128, bf16, 2, sw)) != FA_OK) return st;
  if ((st = encode_bshd_map(&to, o, s.B, s.Sq, s.H, 128, 64, 128, bf16, 2, sw)) != FA_OK) return st;
  return launch_pipe<192, 128, 0, false>(tq, tk, tv, to, make_params(o, lse, s), s, stream);
}

// How many of every 8 exponentials use the software 2^x (Section 3.1.3).  The default is the measured best per
// kernel, head dimension and mask: 1 of 8 where the exponential unit is the limit and nothing else is in the
// way (D = 64 in the one-tile kernel, no mask: +2 ... +6 %), none elsewhere.  FA_EMU_PER8 = 0..3 (read once per
// process) overrides it for every call.
static int emu_per8(const Shape& s) {
  static const int forced = env_int("FA_EMU_PER8", -1);
  if (forced >= 0) return forced > 3 ? 3 : forced;
  return (s.D == 64 && !s.causal && use_tile_kernel(s)) ? 1 : 0;
}

int fwd_launch(const void* q, const void* k, const void* v, void* o, float* lse, const Shape& s, cudaStream_t stream) {
  if (s.f16) {  // FP16 elements: MUFU exponentials only
    return s.D == 64 ? launch_dense<64, 0, true>(q, k, v, o, lse, s, stream)
                     : launch_dense<128, 0, true>(q, k, v, o, lse, s, stream);
  }
  const int emu = emu_per8(s);
  if (s.D == 64) {
    switch (emu) {
      case 1: return launch_dense<64, 1>(q, k, v, o, lse, s, stream);
      case 2: return launch_dense<64, 2>(q, k, v, o, lse, s, stream);
      case 3: return launch_dense<64, 3>(q, k, v, o, lse, s, stream);
      default: return launch_dense<64, 0>(q, k, v, o, lse, s, stream);
    }
  }
  switch (emu) {
    case 1: return launch_dense<128, 1>(q, k, v, o, lse, s, stream);
    case 2: return launch_dense<128, 2>(q, k, v, o, lse, s, stream);
    case 3: return launch_dense<128, 3>(q, k, v, o, lse, s, stream);
    default: return launch_dense<128, 0>(q, k, v, o, lse, s, stream);
  }
}

// ---------------------------------------------------------------- variable-length batches (Section 3.3)
// Longest-processing-time-first order of the sequences of a packed batch: order[r] = index of the
// sequence with the r-th largest amount of work (visible score area), ties by index.  A rank sort:
// every thread ranks one sequence against all others; meant for batches of up to a few thousand.
__global__ void __launch_bounds__(256)
varlen_lpt_order_kernel(const int* __restrict__ cu_q, const int* __restrict__ cu_k, int batch, int causal,
                        int* __restrict__ order) {
  auto work = [&](int b) {
    const double sq = cu_q[b + 1] - cu_q[b], sk = cu_k[b + 1] - cu_k[b];
    if (!causal) return sq * sk;
    // bottom-right aligned mask: row i of sq sees min(sk, max(0, i + sk - sq + 1)) keys
    return sk >= sq ? sq * sk - sq * (sq - 1.0) * 0.5 : sk * (sk + 1.0) * 0.5;
  };
  const int i = blockIdx.x * blockDim.x + threadIdx.x;
  if (i >= batch) return;
  const double wi = work(i);
  int rank = 0;
  for (int j = 0; j < batch; ++j) {
    const double wj = work(j);
    rank += (wj > wi || (wj == wi && j < i)) ? 1 : 0;
  }
  order[rank] = i;
}

int varlen_lpt_order_launch(const int* cu_q, const int* cu_k, int batch, int causal, int* order, cudaStream_t stream) {
  varlen_lpt_order_kernel<<<(batch + 255) / 256, 256, 0, stream>>>(cu_q, cu_k, batch, causal, order);
  return cudaGetLastError() == cudaSuccess ? FA_OK : FA_ERR_CUDA;
}

// s.B = number of sequences, s.Sq = longest query length (sizes the grid), s.Sk = total_k.
int fwd_varlen_launch(const void* q, const void* k, const void* v, void* o, float* lse, const int* cu_q, const int* cu_k,
                      const int* order, int total_q, int total_k, const Shape& s, cudaStream_t stream) {
  Shape packed = s;
  packed.B = 1;
  packed.Sq = total_q;
  packed.Sk = total_k;
  FwdParams p = make_params(o, lse, s);
  p.cu_q = cu_q;
  p.cu_k = cu_k;
  p.order = order;
  p.total_q = total_q;
  CUtensorMap tq, tk, tv, to;
  int st = make_maps(&tq, &tk, &tv, &to, q, k, v, o, packed);
  if (st != FA_OK) return st;
  // Choice of the kernel: half the longest query length stands for the typical key length (the call has no bound
  // on the key lengths, and in a batch of mixed lengths most sequences are well below the longest), so batches of
  // short sequences go to the one-tile kernel like short dense calls.  Measured at 16 heads of 128: 32 lengths of
  // 64...2048 causal +12 %, 64 of 64...1024 +2...6 % / +20 % (causal), 128 of 32...512 +10 % / +25 %.
  Shape longest = s;
  longest.Sk = (s.Sq + 1) / 2;
  if (use_tile_kernel(longest)) {
    if (s.D == 64) return launch_tile<64, 0, false>(tq, tk, tv, to, p, s, stream);
    return launch_tile<128, 0, false>(tq, tk, tv, to, p, s, stream);
  }
  if (s.D == 64) return launch_pipe<64, 64, 0, false>(tq, tk, tv, to, p, s, stream);
  return launch_pipe<128, 128, 0, false>(tq, tk, tv, to, p, s, stream);
}

}  // namespace fa


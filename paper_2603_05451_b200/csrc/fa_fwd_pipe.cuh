// Warp-specialised forward kernel (paper Section 3.1).
//
// One CTA owns 256 query rows of one (batch, head): two 128-row tiles ("tile 0" / "tile 1",
// the paper's high/low tiles) that ping-pong on the tensor cores.  Roles:
//   warps 0-3   softmax warpgroup of tile 0   (one thread per row, Section 3.1.2)
//   warps 4-7   softmax warpgroup of tile 1
//   warps 8-11  correction warpgroup: rescales O in tensor memory when asked (Section 3.1.4),
//               and runs the epilogue (O / l -> bf16 -> shared memory -> TMA store)
//   warp 12     issues every tcgen05.mma:  S_t = Q_t K_j^T  (both operands in shared memory) and
//               O_t += P_t V_j  (P read from tensor memory, V from shared memory)
//   warp 13     TMA producer: Q tiles once, then K_j, V_j through an mbarrier ring
//   warps 14-15 idle (they only donate registers)
// Tensor memory (512 columns): one score buffer S [0,128) shared by both tiles, the 16-bit
// probabilities P_0 [128,192) and P_1 [192,256), the accumulators O_0 [256,256+D) and O_1 [384,384+D).
// Roles talk only through mbarriers with bounded waits; there is no CTA-wide barrier between
// set-up and tear-down, so a role that gives up cannot strand another one.
#pragma once

#include "exp2_emu.cuh"
#include "fa_common.cuh"
#include "fa_fwd_params.cuh"
#include "ptx.cuh"

namespace fa {

// DQK = head dimension of queries and keys, DV = of values and the output (Section 5 benchmarks
// 64, 128 and the pair (192, 128)).  K blocks and V blocks travel through rings of their own:
//   (128,128): 3 + 2 stages of 32 KiB   (64,64): 6 + 6 of 16 KiB   (192,128): 2 of 48 KiB + 1 of 32 KiB
// which with the two Q tiles fills 224 KiB in every case.
template <int DQK, int DV>
struct FwdPipeSmem {
  static constexpr int kQkTileBytes = 128 * DQK * 2;
  static constexpr int kVTileBytes = 128 * DV * 2;
  static constexpr int kKStages = DQK == 192 ? 2 : (DQK == 128 ? 3 : 6);
  static constexpr int kVStages = DQK == 192 ? 1 : (DQK == 128 ? 2 : 6);
  alignas(1024) uint8_t q[2][kQkTileBytes];  // reused as the O staging buffer in the epilogue
  alignas(1024) uint8_t k[kKStages][kQkTileBytes];
  alignas(1024) uint8_t v[kVStages][kVTileBytes];
  float scale[2][128];  // per-row O rescale factor of the current block
  float inv_l[2][128];  // per-row 1/l after the last block
  alignas(8) uint64_t q_full[2];
  uint64_t k_full[kKStages], k_empty[kKStages];
  uint64_t v_full[kVStages], v_empty[kVStages];
  uint64_t s_full[2];      // MMA -> softmax: S_t(j) is in tensor memory
  uint64_t s_free;         // softmax -> MMA: the score buffer has been read into registers
  uint64_t p_full[2];      // softmax + correction -> MMA: first 3/4 of P_t(j) stored and O_t rescaled
  uint64_t p_last[2];      // softmax -> MMA: last quarter of P_t(j) stored (Section 3.1.2, staged store)
  uint64_t o_full[2];      // MMA -> correction: O_t += P_t(j) V_j finished
  uint64_t stat_full[2][4];  // softmax warp w of tile t -> correction warp w: scale[t][32w..] written
  uint64_t fin_full[2][4];   // softmax warp w of tile t -> correction warp w: inv_l[t][32w..] written (once)
  uint64_t o_staged[2];    // correction warps -> storing thread: O_t tile is in shared memory
  uint32_t tmem_base;
  WaitCtl ctl;  // abort flag and launch epoch, read by every bounded wait
};

struct FwdTile {
  int b, h, hk, m0;  // batch, query head, kv head, first query row of the CTA
};

// Number of key blocks tile rows [m_first, m_first + 128) need.
__device__ __forceinline__ int fwd_num_blocks(int Sq, int Sk, int causal, int m_first) {
  if (m_first >= Sq) return 0;
  const int kv_end = causal ? min(Sk, m_first + 128 + (Sk - Sq)) : Sk;
  return kv_end > 0 ? (kv_end + 127) / 128 : 0;
}

template <int D, int kEmuPer8, bool kF16>
__device__ __forceinline__ void softmax_exp_chunk(const uint32_t (&s)[32], uint32_t (&out)[16], float c, float neg_mc,
                                                  float2& sum2, float x_top, bool& top_emulated) {
  // 32 scores -> 16 packed pairs of 16-bit probabilities (bf16, or fp16 when kF16).  Of every 8 elements, kEmuPer8 use the
  // software 2^x on the FMA pipe (Section 3.1.3, partial emulation), the rest MUFU.EX2.  `top_emulated` is raised when an
  // emulated element has the exponent `x_top` of the block's largest score: the row-sum compensation of the caller has to
  // round the very value that was stored for that element.
  const float2 c2 = make_float2(c, c), m2 = make_float2(neg_mc, neg_mc);
#pragma unroll
  for (int i = 0; i < 16; ++i) {
    const float2 x = __ffma2_rn(make_float2(__uint_as_float(s[2 * i]), __uint_as_float(s[2 * i + 1])), c2, m2);
    float2 e;
    const bool emu0 = ((2 * i) & 7) < kEmuPer8, emu1 = ((2 * i + 1) & 7) < kEmuPer8;
    e.x = emu0 ? exp2_emulated(x.x) : ex2_approx(x.x);
    e.y = emu1 ? exp2_emulated(x.y) : ex2_approx(x.y);
    if (emu0) top_emulated |= x.x == x_top;
    if (emu1) top_emulated |= x.y == x_top;
    sum2 = __fadd2_rn(sum2, e);
    out[i] = pack2<kF16>(e.x, e.y);
  }
}
// What rounding to 16 bits added to the block's largest probability (exponent x_top), computed the way the element
// itself was (see softmax_exp_chunk).
template <int kEmuPer8, bool kF16>
__device__ __forceinline__ float top_rounding_excess(float x_top, bool top_emulated) {
  float p_top = ex2_approx(x_top);
  if (kEmuPer8 > 0 && top_emulated) p_top = exp2_emulated(x_top);
  return unpack2<kF16>(pack2<kF16>(p_top, 0.0f)).x - p_top;
}

// D: value / output head dimension; kF16: inputs and output are FP16 instead of BF16
template <int DQK, int D, int kEmuPer8, bool kF16 = false>
__global__ void __launch_bounds__(512, 1)
fwd_pipe_kernel(const __grid_constant__ CUtensorMap tm_q, const __grid_constant__ CUtensorMap tm_k,
                const __grid_constant__ CUtensorMap tm_v, const __grid_constant__ CUtensorMap tm_o,
                const FwdParams p, const int n_mblocks) {
  extern __shared__ __align__(1024) uint8_t smem_raw[];
  using Smem = FwdPipeSmem<DQK, D>;
  Smem& sm = *reinterpret_cast<Smem*>(smem_raw);
  if ((smem_u32(smem_raw) & 1023u) != 0) {  // swizzled tiles need 1024-byte alignment; never seen, but checked
    if (threadIdx.x == 0) record_device_status(5, __LINE__, p.epoch);
    return;
  }
  constexpr int kKStages = Smem::kKStages, kVStages = Smem::kVStages;
  constexpr int kRegions = D / 64, kQkRegions = DQK / 64;
  constexpr int kRegionBytes = 128 * 128;
  constexpr uint32_t kIdescS = make_idesc(128, 128, false, false, kF16);
  constexpr uint32_t kIdescO = make_idesc(128, D, false, true, kF16);

  const int tid = threadIdx.x, warp = tid >> 5, lane = tid & 31;
  volatile int* abort_flag = &sm.ctl.abort_flag;

  // Work decode: batches outermost, then sections of heads whose K and V fit in L2 together, then
  // 256-row blocks from the LAST one down (longest causal tiles first, Section 3.3), the heads of the
  // section fastest so the heads sharing K/V run together.
  FwdTile tile;
  int Sq = p.Sq, Sk = p.Sk;  // for a variable-length batch: this sequence's lengths (set below)
  int q_row0, k_row0, tma_b;  // token-axis origin of this sequence in the tensor maps, and their batch coordinate
  float* lse_rows;            // LSE of (this sequence, this head), indexed by the row inside the sequence
  {
    // batch, then head section, then 256-row block (last first), then the heads of the section
    const int idx = blockIdx.x;
    const int hs = p.heads_per_section > 0 ? p.heads_per_section : p.H;
    const int per_batch = p.H * n_mblocks, per_section = hs * n_mblocks;
    tile.b = idx / per_batch;
    const int r = idx % per_batch;
    const int r2 = r % per_section;
    tile.h = (r / per_section) * hs + r2 % hs;
    tile.m0 = (n_mblocks - 1 - r2 / hs) * 256;
    tile.hk = tile.h / (p.H / p.Hkv);
    if (p.cu_q != nullptr) {
      // Packed sequences (Section 3.3, variable sequence length): virtual batch index -> sequence in
      // longest-first order; 256-row blocks past the end of a short sequence leave at once.
      const int seq = p.order != nullptr ? p.order[tile.b] : tile.b;
      q_row0 = p.cu_q[seq];
      k_row0 = p.cu_k[seq];
      Sq = p.cu_q[seq + 1] - q_row0;
      Sk = p.cu_k[seq + 1] - k_row0;
      if (tile.m0 >= Sq) return;
      tma_b = 0;
      lse_rows = p.lse + (size_t)tile.h * p.total_q + q_row0;
    } else {
      q_row0 = 0;
      k_row0 = 0;
      tma_b = tile.b;
      lse_rows = p.lse + ((size_t)tile.b * p.H + tile.h) * Sq;
    }
  }
  const int n_blk[2] = {fwd_num_blocks(Sq, Sk, p.causal, tile.m0), fwd_num_blocks(Sq, Sk, p.causal, tile.m0 + 128)};
  const bool valid[2] = {tile.m0 < Sq, tile.m0 + 128 < Sq};
  const int n_max = max(n_blk[0], n_blk[1]);
  const int n_blk_mine = (warp >> 2) == 1 ? n_blk[1] : n_blk[0];  // softmax warps: blocks of their tile

  auto load_q = [&](int t) {
    if (n_blk[t] > 0) {
      mbar_expect_tx(&sm.q_full[t], Smem::kQkTileBytes);
      for (int r = 0; r < kQkRegions; ++r)
        tma_load_4d(sm.q[t] + r * kRegionBytes, &tm_q, &sm.q_full[t], r * 64, tile.h, q_row0 + tile.m0 + t * 128, tma_b);
    }
  };
  auto load_k = [&](int j, int slot) {
    mbar_expect_tx(&sm.k_full[slot], Smem::kQkTileBytes);
    for (int r = 0; r < kQkRegions; ++r)
      tma_load_4d(sm.k[slot] + r * kRegionBytes, &tm_k, &sm.k_full[slot], r * 64, tile.hk, k_row0 + j * 128, tma_b);
  };
  auto load_v = [&](int j, int slot) {
    mbar_expect_tx(&sm.v_full[slot], Smem::kVTileBytes);
    for (int r = 0; r < kRegions; ++r)
      tma_load_4d(sm.v[slot] + r * kRegionBytes, &tm_v, &sm.v_full[slot], r * 64, tile.hk, k_row0 + j * 128, tma_b);
  };

  if (tid == 0) {
    sm.ctl.abort_flag = 0;
    sm.ctl.launch_epoch = (int)p.epoch;
    for (int t = 0; t < 2; ++t) {
      mbar_init(&sm.s_full[t], 1);
      mbar_init(&sm.p_full[t], 8);  // 4 softmax warps + 4 correction warps
      mbar_init(&sm.p_last[t], 4);
      mbar_init(&sm.o_full[t], 1);
      mbar_init(&sm.o_staged[t], 4);
      for (int w = 0; w < 4; ++w) mbar_init(&sm.stat_full[t][w], 1);
      for (int w = 0; w < 4; ++w) mbar_init(&sm.fin_full[t][w], 1);
    }
    for (int s = 0; s < kKStages; ++s) mbar_init(&sm.k_empty[s], 1);
    for (int s = 0; s < kVStages; ++s) mbar_init(&sm.v_empty[s], 1);
    mbar_init(&sm.s_free, 4);
    fence_barrier_init();
  }
  if (warp == 12) {
    tmem_alloc(&sm.tmem_base, 512);
    tmem_relinquish();
  }
  if (warp == 13 && lane == 0) {
    // The producer arms the barriers its loads complete on by itself and sends the first loads off at
    // once, while tensor memory is still being allocated: what the first products need first.
    for (int t = 0; t < 2; ++t) mbar_init(&sm.q_full[t], 1);
    for (int s = 0; s < kKStages; ++s) mbar_init(&sm.k_full[s], 1);
    for (int s = 0; s < kVStages; ++s) mbar_init(&sm.v_full[s], 1);
    fence_barrier_init();
    if (n_max > 0) {
      load_q(0);
      load_k(0, 0);
      load_q(1);
      load_v(0, 0);
      for (int j = 1; j < kKStages && j < n_max; ++j) load_k(j, j);
      for (int j = 1; j < kVStages && j < n_max; ++j) load_v(j, j);
    }
    tma_prefetch_desc(&tm_o);
  }
  tc_fence_before();
  __syncthreads();
  tc_fence_after();
  const uint32_t tmem = sm.tmem_base;

  if (warp < 8) {
    // ============================================================ softmax warpgroups
    reg_alloc<192>();
    const int t = warp >> 2, w = warp & 3;
    const int r_in_tile = w * 32 + lane;
    const int row = tile.m0 + t * 128 + r_in_tile;
    // Tensor memory: one score buffer [0,128) shared by both tiles, P_0 [128,192), P_1 [192,256),
    // O_0 [256,384), O_1 [384,512).  The score buffer is free again as soon as its reader holds the
    // scores in registers, and P_t has a place of its own, so S_t(j+1) is formed while the softmax
    // of S_t(j) is still running and the softmax warps never wait for a product.
    const uint32_t s_addr = tmem + ((uint32_t)(w * 32) << 16);
    const uint32_t p_addr = s_addr + 128u + (uint32_t)(t * 64);
    const float c = p.scale_log2;
    const int shift = Sk - Sq;
    const int row_limit = p.causal ? min(Sk - 1, row + shift) : Sk - 1;  // last visible key
    const int tile_first_limit = p.causal ? min(Sk - 1, tile.m0 + t * 128 + shift) : Sk - 1;
    // l_run: FP32 sum of the unrounded probabilities (gives the LSE).  l_fix: what rounding to 16 bits
    // added to the LARGEST probability of every block.  O is divided by l_run + l_fix: the products see
    // the rounded probabilities, and in a row whose weight sits on one key the rounding of that one
    // probability (up to 2^-9 relative when the running maximum is stale, Eq. 6) would otherwise show
    // in O undiminished.  One exponential per row and block instead of a second sum over all elements.
    float m_run = -INFINITY, l_run = 0.0f, l_fix = 0.0f;
    bool ok = true;

    for (int j = 0; j < n_blk_mine; ++j) {
      ok = __all_sync(0xffffffffu, mbar_wait(&sm.s_full[t], j & 1, abort_flag, __LINE__));
      if (!ok) break;
      tc_fence_after();
      uint32_t s[4][32];
      // The second half of the scores is fetched while the maxima of the first half are taken.
      tmem_ld32(s_addr, s[0]);
      tmem_ld32(s_addr + 32, s[1]);
      tmem_wait_ld();
      tmem_ld32(s_addr + 64, s[2]);
      tmem_ld32(s_addr + 96, s[3]);

      const int j0 = j * 128;
      const bool masked = j0 + 127 > tile_first_limit;  // block touches the mask of some row of this tile
      const int lim = row_limit - j0;
      float mx[4] = {-INFINITY, -INFINITY, -INFINITY, -INFINITY};
#pragma unroll
      for (int q4 = 0; q4 < 4; ++q4) {
        if (q4 == 2) {
          tmem_wait_ld();
          tc_fence_before();
          __syncwarp();
          if (lane == 0) mbar_arrive(&sm.s_free);
        }
        if (masked) {
#pragma unroll
          for (int i = 0; i < 32; ++i)
            if (q4 * 32 + i > lim) s[q4][i] = 0xff800000u;  // -inf
        }
#pragma unroll
        for (int i = 0; i < 32; i += 8) {
          mx[0] = max3(mx[0], __uint_as_float(s[q4][i]), __uint_as_float(s[q4][i + 1]));
          mx[1] = max3(mx[1], __uint_as_float(s[q4][i + 2]), __uint_as_float(s[q4][i + 3]));
          mx[2] = max3(mx[2], __uint_as_float(s[q4][i + 4]), __uint_as_float(s[q4][i + 5]));
          mx[3] = max3(mx[3], __uint_as_float(s[q4][i + 6]), __uint_as_float(s[q4][i + 7]));
        }
      }
      const float m_blk = fmaxf(max3(mx[0], mx[1], mx[2]), mx[3]);
      const float m_new = fmaxf(m_run, m_blk);
      // Conditional rescale (Eq. 6): only when the maximum grew by more than tau in the base-2
      // domain; the decision is taken for the whole warp (Section 3.1.4, last sentence).
      const bool need = (m_new - m_run) * c > p.tau;
      float f = 1.0f;
      if (__any_sync(0xffffffffu, need)) {
        f = (m_run == -INFINITY) ? 0.0f : ex2_approx((m_run - m_new) * c);
        l_run *= f;
        l_fix *= f;
        m_run = m_new;
      }
      if (j > 0) {
        // O_t += P_t(j-1) V_{j-1} has retired: P_t may be overwritten, and the correction warp has
        // read the previous block's factors (its arrival preceded that product).  Waiting here, before
        // this block's factors are published, also keeps p_full sound: a correction warp arrives for
        // block j only after every softmax warp of the tile has finished block j - 1, so no arrival
        // can land in the previous phase.
        ok = __all_sync(0xffffffffu, mbar_wait(&sm.o_full[t], (j - 1) & 1, abort_flag, __LINE__));
        if (!ok) break;
      }
      sm.scale[t][r_in_tile] = f;
      __syncwarp();
      if (lane == 0) mbar_arrive(&sm.stat_full[t][w]);

      const float neg_mc = (m_run == -INFINITY) ? 0.0f : -m_run * c;
      const float x_top = fmaf(m_blk, c, neg_mc);  // exponent of the block's largest probability, as formed below
      bool top_emulated = false;
      float2 sum2 = make_float2(0.0f, 0.0f);
#pragma unroll
      for (int q4 = 0; q4 < 4; ++q4) {
        uint32_t pk[16];
        softmax_exp_chunk<D, kEmuPer8, kF16>(s[q4], pk, c, neg_mc, sum2, x_top, top_emulated);
        tmem_st16(p_addr + q4 * 16, pk);
        if (q4 == 2) {
          // staged store: three quarters of P are enough to start O += P V
          tmem_wait_st();
          tc_fence_before();
          __syncwarp();
          if (lane == 0) mbar_arrive(&sm.p_full[t]);
        }
      }
      l_run += sum2.x + sum2.y;
      l_fix += top_rounding_excess<kEmuPer8, kF16>(x_top, top_emulated);
      tmem_wait_st();
      tc_fence_before();
      __syncwarp();
      if (lane == 0) mbar_arrive(&sm.p_last[t]);
    }

    if (ok && valid[t]) {
      // Hand 1/l to the correction warp and write the LSE.  This uses a barrier of its own: nothing
      // orders it after the correction warp's wait for the last block's statistics, so an extra
      // phase of stat_full could run two phases ahead of a slow waiter and strand it.
      sm.inv_l[t][r_in_tile] = l_run > 0.0f ? 1.0f / (l_run + l_fix) : 0.0f;
      __syncwarp();
      if (lane == 0) mbar_arrive(&sm.fin_full[t][w]);
      if (row < Sq) lse_rows[row] = l_run > 0.0f ? (m_run * c + log2f(l_run)) * kLn2 : -INFINITY;
    }
  } else if (warp < 12) {
    // ============================================================ correction warpgroup
    reg_dealloc<80>();
    const int w = warp & 3;
    const int r_in_tile = w * 32 + lane;
    bool ok = true;
    for (int j = 0; j < n_max && ok; ++j) {
      for (int t = 0; t < 2; ++t) {
        if (j >= n_blk[t]) continue;
        ok = __all_sync(0xffffffffu, mbar_wait(&sm.stat_full[t][w], j & 1, abort_flag, __LINE__));
        if (!ok) break;
        const float f = sm.scale[t][r_in_tile];
        if (j > 0 && __any_sync(0xffffffffu, f != 1.0f)) {
          ok = __all_sync(0xffffffffu, mbar_wait(&sm.o_full[t], (j - 1) & 1, abort_flag, __LINE__));
          if (!ok) break;
          tc_fence_after();
          const uint32_t o_addr = tmem + 256u + (uint32_t)(t * 128) + ((uint32_t)(w * 32) << 16);
#pragma unroll
          for (int cc = 0; cc < D / 32; ++cc) {
            uint32_t r[32];
            tmem_ld32(o_addr + cc * 32, r);
            tmem_wait_ld();
#pragma unroll
            for (int i = 0; i < 32; ++i) r[i] = __float_as_uint(__uint_as_float(r[i]) * f);
            tmem_st32(o_addr + cc * 32, r);
          }
          tmem_wait_st();
          tc_fence_before();
        }
        __syncwarp();
        if (lane == 0) mbar_arrive(&sm.p_full[t]);
      }
    }
    // epilogue: O_t / l -> bf16 -> shared memory (128-byte swizzle) -> TMA store
    for (int t = 0; t < 2 && ok; ++t) {
      if (!valid[t]) continue;
      const int n = n_blk[t];
      ok = __all_sync(0xffffffffu, mbar_wait(&sm.fin_full[t][w], 0, abort_flag, __LINE__));
      if (!ok) break;
      const float inv_l = sm.inv_l[t][r_in_tile];
      if (n > 0) {
        ok = __all_sync(0xffffffffu, mbar_wait(&sm.o_full[t], (n - 1) & 1, abort_flag, __LINE__));
        if (!ok) break;
        tc_fence_after();
      }
      const uint32_t o_addr = tmem + 256u + (uint32_t)(t * 128) + ((uint32_t)(w * 32) << 16);
      uint8_t* stage = sm.q[t];
      // In a packed batch the rows after a sequence's last one belong to the next sequence, so a tile
      // that overhangs the end cannot leave through a 128-row TMA store: its rows are written one by one.
      const int row = tile.m0 + t * 128 + r_in_tile;
      const bool row_by_row = p.cu_q != nullptr && tile.m0 + t * 128 + 128 > Sq;
      __nv_bfloat16* o_row = p.o + ((size_t)(q_row0 + min(row, Sq - 1)) * p.H + tile.h) * D;
#pragma unroll
      for (int cc = 0; cc < D / 32; ++cc) {
        uint32_t r[32];
        if (n > 0) {
          tmem_ld32(o_addr + cc * 32, r);
          tmem_wait_ld();
        } else {
#pragma unroll
          for (int i = 0; i < 32; ++i) r[i] = 0u;
        }
        // 32 columns = 64 bytes = four 16-byte chunks of this row inside 64-column region cc / 2
        uint8_t* region = stage + (cc >> 1) * kRegionBytes + r_in_tile * 128;
#pragma unroll
        for (int i = 0; i < 4; ++i) {
          uint4 v4;
          v4.x = pack2<kF16>(__uint_as_float(r[8 * i + 0]) * inv_l, __uint_as_float(r[8 * i + 1]) * inv_l);
          v4.y = pack2<kF16>(__uint_as_float(r[8 * i + 2]) * inv_l, __uint_as_float(r[8 * i + 3]) * inv_l);
          v4.z = pack2<kF16>(__uint_as_float(r[8 * i + 4]) * inv_l, __uint_as_float(r[8 * i + 5]) * inv_l);
          v4.w = pack2<kF16>(__uint_as_float(r[8 * i + 6]) * inv_l, __uint_as_float(r[8 * i + 7]) * inv_l);
          const int chunk = (cc & 1) * 4 + i;
          if (row_by_row) {
            if (row < Sq) reinterpret_cast<uint4*>(o_row + cc * 32)[i] = v4;
          } else {
            *reinterpret_cast<uint4*>(region + ((chunk ^ (r_in_tile & 7)) << 4)) = v4;
          }
        }
      }
      if (row_by_row) continue;  // (warp-uniform) nothing to hand to the storing thread
      fence_proxy_async_smem();
      __syncwarp();
      if (lane == 0) mbar_arrive(&sm.o_staged[t]);
      if (warp == 8) {
        ok = __all_sync(0xffffffffu, mbar_wait(&sm.o_staged[t], 0, abort_flag, __LINE__));
        if (!ok) break;
        if (lane == 0) {
          for (int r = 0; r < kRegions; ++r)
            tma_store_4d(&tm_o, stage + r * kRegionBytes, r * 64, tile.h, q_row0 + tile.m0 + t * 128, tma_b);
          tma_commit_group();
        }
      }
    }
    if (warp == 8 && lane == 0) tma_wait_group_read<0>();
  } else if (warp == 12) {
    // ============================================================ MMA issuer
    // The whole warp walks the role in lock step so that every descriptor word is warp-uniform
    // (and can live in uniform registers); one elected lane issues.  Descriptors are kept as
    // 32-bit low words (start address) and advanced by adding constants.
    reg_dealloc<48>();
    if (n_max > 0) {
      constexpr uint32_t kQkStep = Smem::kQkTileBytes >> 4, kVStep = Smem::kVTileBytes >> 4;
      const uint32_t q_lo0 = desc_lo(smem_u32(sm.q[0]), 16);
      const uint32_t k_lo0 = desc_lo(smem_u32(sm.k[0]), 16);
      const uint32_t v_lo0 = desc_lo(smem_u32(sm.v[0]), kRegionBytes);
      const int n0 = n_blk[0], n1 = n_blk[1];
      auto wait_bar = [&](uint64_t* bar, uint32_t parity) {
        return __all_sync(0xffffffffu, mbar_wait(bar, parity, abort_flag, __LINE__));
      };
      auto issue_s = [&](int t, int slot) {  // S_t = Q_t K^T
        const uint32_t a_lo = q_lo0 + t * kQkStep, b_lo = k_lo0 + slot * kQkStep;
        const uint32_t d_addr = tmem;
        if (elect_one()) {
#pragma unroll
          for (int kk = 0; kk < DQK / 16; ++kk) {
            const uint32_t off = ((kk / 4) * kRegionBytes + (kk % 4) * 32) >> 4;
            mma_ss_lohi(d_addr, a_lo + off, b_lo + off, kDescHiSw128, kIdescS, kk > 0);
          }
          mma_commit(&sm.s_full[t]);
        }
        __syncwarp();
      };
      auto issue_pv = [&](int t, int slot, uint32_t accumulate, int k_first, int k_last) {  // O_t += P_t V
        const uint32_t b_lo = v_lo0 + slot * kVStep;
        const uint32_t d_addr = tmem + 256u + t * 128, p_addr = tmem + 128u + t * 64;
        if (elect_one()) {
#pragma unroll
          for (int kk = 0; kk < 8; ++kk) {
            if (kk >= k_first && kk < k_last)
              mma_ts_lohi(d_addr, p_addr + kk * 8, b_lo + ((kk * 2048) >> 4), kDescHiSw128, kIdescO,
                          kk > 0 ? 1u : accumulate);
          }
          if (k_last == 8) mma_commit(&sm.o_full[t]);
        }
        __syncwarp();
      };
      // Issue order: S_0(0), S_1(0), S_0(1), then per block j: O_0 += P_0(j) V_j, S_1(j+1),
      // O_1 += P_1(j) V_j, S_0(j+2).  Every score product but the first waits until the previous
      // one has been read out of the shared buffer.  K_j is used by tile 0 first, then by tile 1.
      int uses = 0;
      auto do_s = [&](int t, int j) -> bool {
        const bool first = t == 0 || j >= n0, last = t == 1 || j >= n1;
        const int slot = j % kKStages;
        if (first && !wait_bar(&sm.k_full[slot], (uint32_t)((j / kKStages) & 1))) return false;
        if (uses > 0) {
          if (!wait_bar(&sm.s_free, (uint32_t)((uses - 1) & 1))) return false;
          tc_fence_after();
        }
        ++uses;
        issue_s(t, slot);
        if (last) {
          if (elect_one()) mma_commit(&sm.k_empty[slot]);
          __syncwarp();
        }
        return true;
      };
      auto do_pv = [&](int t, int j, int slot_v) -> bool {
        if (!wait_bar(&sm.p_full[t], j & 1)) return false;
        tc_fence_after();
        issue_pv(t, slot_v, j > 0 ? 1u : 0u, 0, 6);
        if (!wait_bar(&sm.p_last[t], j & 1)) return false;
        tc_fence_after();
        issue_pv(t, slot_v, 1u, 6, 8);
        return true;
      };
      do {
        if (n0 > 0 && !(wait_bar(&sm.q_full[0], 0) && do_s(0, 0))) break;
        if (n1 > 0 && !(wait_bar(&sm.q_full[1], 0) && do_s(1, 0))) break;
        if (n0 > 1 && !do_s(0, 1)) break;
        int slot_v = 0;
        uint32_t ph_v = 0;
        for (int j = 0; j < n_max; ++j) {
          if (!wait_bar(&sm.v_full[slot_v], ph_v)) break;  // V_j
          if (j < n0 && !do_pv(0, j, slot_v)) break;
          if (j + 1 < n1 && !do_s(1, j + 1)) break;
          if (j < n1 && !do_pv(1, j, slot_v)) break;
          if (j + 2 < n0 && !do_s(0, j + 2)) break;
          if (elect_one()) mma_commit(&sm.v_empty[slot_v]);
          __syncwarp();
          if (++slot_v == kVStages) { slot_v = 0; ph_v ^= 1; }
        }
      } while (false);
    }
    __syncwarp();
  } else if (warp == 13) {
    // ============================================================ TMA producer
    reg_dealloc<48>();
    if (n_max > 0 && lane == 0) {
      // (the rings were filled before the CTA-wide barrier, see above)
      // Steady state, in the order in which the MMA warp releases stages: K_0's after the first S
      // products, then for every block j K_{j+1}'s (S_1(j+1) issued) and V_j's (both P V_j issued).
      int next_k = kKStages, next_v = kVStages;
      bool ok = true;
      if (next_k < n_max) {
        ok = mbar_wait(&sm.k_empty[0], 0, abort_flag, __LINE__);
        if (ok) load_k(next_k++, 0);
      }
      int slot_k = kKStages > 1 ? 1 : 0, slot_v = 0;
      uint32_t ph_k = kKStages > 1 ? 0u : 1u, ph_v = 0;
      while (ok && (next_k < n_max || next_v < n_max)) {
        if (next_k < n_max) {
          if (!(ok = mbar_wait(&sm.k_empty[slot_k], ph_k, abort_flag, __LINE__))) break;
          load_k(next_k++, slot_k);
        }
        if (next_v < n_max) {
          if (!(ok = mbar_wait(&sm.v_empty[slot_v], ph_v, abort_flag, __LINE__))) break;
          load_v(next_v++, slot_v);
        }
        if (++slot_v == kVStages) { slot_v = 0; ph_v ^= 1; }
        if (++slot_k == kKStages) { slot_k = 0; ph_k ^= 1; }
      }
    }
    __syncwarp();
  } else {
    reg_dealloc<48>();
  }

  tc_fence_before();
  __syncthreads();
  if (warp == 12) tmem_dealloc(tmem, 512);
}

}  // namespace fa

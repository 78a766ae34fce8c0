// Forward kernel for short sequences: one 128-row tile per CTA, two CTAs resident per SM.
//
// The pipelined kernel (fa_fwd_pipe.cuh) overlaps the products of one 128-row tile with the softmax of
// another inside one CTA, which owns the whole SM; the set-up, the first loads and the epilogue of a CTA
// overlap with nothing, and with a few key blocks per tile (short or causal sequences) that is a large
// part of its life.  Here the two tiles that share an SM are CTAs of their own: each takes half of the
// tensor memory (256 columns), under half of the shared memory and of the registers, and the hardware
// interleaves them, so one CTA's set-up and epilogue run under the other's main loop (the role a
// persistent tile scheduler plays in Section 3.3).  The price is that K and V are fetched once per 128 rows
// instead of once per 256, so the launch code uses this kernel only where the pipelined one is far from
// its steady state.
//
//   warps 0-3  softmax (one thread per row, Section 3.1.2), the conditional rescale of O (Section 3.1.4) and
//              the epilogue (O / l -> 16 bits -> shared memory -> TMA store)
//   warp 4     issues every tcgen05.mma:  S = Q K_j^T,  O += P V_j  (P read from tensor memory)
//   warp 5     TMA producer: Q once, then K_j and V_j through mbarrier rings
//   warps 6-7  idle (they only donate registers)
// Tensor memory (256 columns), D = 128: S [0,128), overwritten in place by the 16-bit P [0,64) once a thread
// holds its row of scores in registers (the paper's layout); O [128,256).  S(j+1) is issued behind O += P(j) V_j
// on the same in-order pipe, so it cannot overtake the read of P(j), and its completion implies that of
// that product: the softmax warps need no further barrier before they touch O.
// D = 64: O takes 64 columns, which leaves P a place of its own: S [0,128), P [128,192), O [192,256).  S(j+1) is
// then issued as soon as S(j) has been read into registers (s_free), i.e. under the softmax of block j, and the
// softmax warps wait for O += P(j-1) V_{j-1} (o_full) before they rescale O or overwrite P.
#pragma once

#include "fa_fwd_pipe.cuh"

namespace fa {

template <int D>
struct FwdTileSmem {
  static constexpr int kTileBytes = 128 * D * 2;
  static constexpr int kStages = D == 128 ? 1 : 2;
  alignas(1024) uint8_t q[kTileBytes];  // reused as the O staging buffer in the epilogue
  alignas(1024) uint8_t k[kStages][kTileBytes];
  alignas(1024) uint8_t v[kStages][kTileBytes];
  alignas(8) uint64_t q_full;
  uint64_t k_full[kStages], k_empty[kStages];
  uint64_t v_full[kStages], v_empty[kStages];
  uint64_t s_full;    // MMA -> softmax: S(j) is in tensor memory (D = 128: and O += P(j-1) V_{j-1} has finished)
  uint64_t s_free;    // softmax -> MMA (D = 64): S(j) has been read into registers
  uint64_t p_full;    // softmax -> MMA: P(j) stored, O rescaled if that was needed
  uint64_t o_full;    // MMA -> softmax: O += P(j) V_j has finished
  uint64_t o_staged;  // softmax warps -> storing thread: the O tile is in shared memory
  uint32_t tmem_base;
  WaitCtl ctl;  // abort flag and launch epoch, read by every bounded wait
};
// Dynamic shared memory asked for: the structure plus room to align it to 1024 bytes (the second CTA of an
// SM does not start on such a boundary by itself).
template <int D>
constexpr int fwd_tile_smem_bytes() { return (int)sizeof(FwdTileSmem<D>) + 1024; }

template <int D, int kEmuPer8, bool kF16 = false>
__global__ void __launch_bounds__(256, 2)
fwd_tile_kernel(const __grid_constant__ CUtensorMap tm_q, const __grid_constant__ CUtensorMap tm_k,
                const __grid_constant__ CUtensorMap tm_v, const __grid_constant__ CUtensorMap tm_o,
                const FwdParams p, const int n_mblocks) {
  extern __shared__ uint8_t smem_raw[];
  using Smem = FwdTileSmem<D>;
  Smem& sm = *reinterpret_cast<Smem*>(smem_raw + ((1024u - (smem_u32(smem_raw) & 1023u)) & 1023u));
  constexpr int kStages = Smem::kStages;
  constexpr int kRegions = D / 64;
  constexpr int kRegionBytes = 128 * 128;
  constexpr uint32_t kIdescS = make_idesc(128, 128, false, false, kF16);
  constexpr uint32_t kIdescO = make_idesc(128, D, false, true, kF16);
  constexpr bool kSeparateP = D == 64;  // P in columns of its own (see the layout above)
  constexpr uint32_t kColP = kSeparateP ? 128u : 0u, kColO = kSeparateP ? 192u : 128u;

  const int tid = threadIdx.x, warp = tid >> 5, lane = tid & 31;
  volatile int* abort_flag = &sm.ctl.abort_flag;

  // Work decode: batches outermost, then sections of heads whose K and V fit in L2 together, then
  // 128-row tiles from the LAST one down (longest causal tiles first, Section 3.3), the heads of the
  // section fastest so the heads sharing K/V run together.
  int Sq = p.Sq, Sk = p.Sk;   // for a variable-length batch: this sequence's lengths (set below)
  int b, h, hk, m0;
  int q_row0 = 0, k_row0 = 0;  // token-axis origin of this sequence in the tensor maps
  float* lse_rows;             // LSE of (this sequence, this head), indexed by the row inside the sequence
  {
    const int idx = blockIdx.x;
    const int hs = p.heads_per_section > 0 ? p.heads_per_section : p.H;
    const int per_batch = p.H * n_mblocks, per_section = hs * n_mblocks;
    b = idx / per_batch;
    const int r = idx % per_batch;
    const int r2 = r % per_section;
    h = (r / per_section) * hs + r2 % hs;
    m0 = (n_mblocks - 1 - r2 / hs) * 128;
    hk = h / (p.H / p.Hkv);
    if (p.cu_q != nullptr) {
      // Packed sequences (Section 3.3, variable sequence length): virtual batch index -> sequence in
      // longest-first order; tiles past the end of a short sequence leave at once.
      const int seq = p.order != nullptr ? p.order[b] : b;
      q_row0 = p.cu_q[seq];
      k_row0 = p.cu_k[seq];
      Sq = p.cu_q[seq + 1] - q_row0;
      Sk = p.cu_k[seq + 1] - k_row0;
      if (m0 >= Sq) return;
      b = 0;  // batch coordinate of the packed tensors
      lse_rows = p.lse + (size_t)h * p.total_q + q_row0;
    } else {
      lse_rows = p.lse + ((size_t)b * p.H + h) * Sq;
    }
  }
  const int n = fwd_num_blocks(Sq, Sk, p.causal, m0);

  auto load_k = [&](int j, int slot) {
    mbar_expect_tx(&sm.k_full[slot], Smem::kTileBytes);
    for (int r = 0; r < kRegions; ++r)
      tma_load_4d(sm.k[slot] + r * kRegionBytes, &tm_k, &sm.k_full[slot], r * 64, hk, k_row0 + j * 128, b);
  };
  auto load_v = [&](int j, int slot) {
    mbar_expect_tx(&sm.v_full[slot], Smem::kTileBytes);
    for (int r = 0; r < kRegions; ++r)
      tma_load_4d(sm.v[slot] + r * kRegionBytes, &tm_v, &sm.v_full[slot], r * 64, hk, k_row0 + j * 128, b);
  };

  if (tid == 0) {
    sm.ctl.abort_flag = 0;
    sm.ctl.launch_epoch = (int)p.epoch;
    mbar_init(&sm.s_full, 1);
    mbar_init(&sm.s_free, 4);
    mbar_init(&sm.p_full, 4);
    mbar_init(&sm.o_full, 1);
    mbar_init(&sm.o_staged, 4);
    for (int s = 0; s < kStages; ++s) {
      mbar_init(&sm.k_empty[s], 1);
      mbar_init(&sm.v_empty[s], 1);
    }
    fence_barrier_init();
  }
  if (warp == 4) {
    tmem_alloc(&sm.tmem_base, 256);
    tmem_relinquish();
  }
  if (warp == 5 && lane == 0) {
    // The producer arms the barriers its loads complete on by itself and sends the first loads off at
    // once, while tensor memory is still being allocated.
    mbar_init(&sm.q_full, 1);
    for (int s = 0; s < kStages; ++s) {
      mbar_init(&sm.k_full[s], 1);
      mbar_init(&sm.v_full[s], 1);
    }
    fence_barrier_init();
    if (n > 0) {
      mbar_expect_tx(&sm.q_full, Smem::kTileBytes);
      for (int r = 0; r < kRegions; ++r) tma_load_4d(sm.q + r * kRegionBytes, &tm_q, &sm.q_full, r * 64, h, q_row0 + m0, b);
      for (int j = 0; j < kStages && j < n; ++j) load_k(j, j);
      for (int j = 0; j < kStages && j < n; ++j) load_v(j, j);
    }
    tma_prefetch_desc(&tm_o);
  }
  tc_fence_before();
  __syncthreads();
  tc_fence_after();
  const uint32_t tmem = sm.tmem_base;

  if (warp < 4) {
    // ============================================================ softmax, rescale, epilogue
    reg_alloc<208>();
    const int w = warp;
    const int r_in_tile = w * 32 + lane;
    const int row = m0 + r_in_tile;
    const uint32_t s_addr = tmem + ((uint32_t)(w * 32) << 16);
    const uint32_t p_addr = s_addr + kColP, o_addr = s_addr + kColO;
    const float c = p.scale_log2;
    const int shift = Sk - Sq;
    const int row_limit = p.causal ? min(Sk - 1, row + shift) : Sk - 1;  // last visible key
    const int tile_first_limit = p.causal ? min(Sk - 1, m0 + shift) : Sk - 1;
    // l_run: FP32 sum of the unrounded probabilities (gives the LSE).  l_fix: what rounding to 16 bits
    // added to the largest probability of every block; O is divided by l_run + l_fix (see fa_fwd_pipe.cuh).
    float m_run = -INFINITY, l_run = 0.0f, l_fix = 0.0f;
    bool ok = true;

    for (int j = 0; j < n; ++j) {
      ok = __all_sync(0xffffffffu, mbar_wait(&sm.s_full, j & 1, abort_flag, __LINE__));
      if (!ok) break;
      tc_fence_after();
      uint32_t s[4][32];
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
          if (kSeparateP) {  // the score buffer may be overwritten by the next block's product
            tc_fence_before();
            __syncwarp();
            if (lane == 0) mbar_arrive(&sm.s_free);
          }
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
      if (kSeparateP && j > 0) {
        // O += P(j-1) V_{j-1} has finished: O may be rescaled and P overwritten
        ok = __all_sync(0xffffffffu, mbar_wait(&sm.o_full, (j - 1) & 1, abort_flag, __LINE__));
        if (!ok) break;
        tc_fence_after();
      }
      if (__any_sync(0xffffffffu, need)) {
        const float f = (m_run == -INFINITY) ? 0.0f : ex2_approx((m_run - m_new) * c);
        l_run *= f;
        l_fix *= f;
        m_run = m_new;
        if (j > 0) {  // O holds the sum over blocks 0..j-1
#pragma unroll
          for (int cc = 0; cc < D / 32; ++cc) {
            uint32_t r[32];
            tmem_ld32(o_addr + cc * 32, r);
            tmem_wait_ld();
#pragma unroll
            for (int i = 0; i < 32; ++i) r[i] = __float_as_uint(__uint_as_float(r[i]) * f);
            tmem_st32(o_addr + cc * 32, r);
          }
        }
      }
      const float neg_mc = (m_run == -INFINITY) ? 0.0f : -m_run * c;
      const float x_top = fmaf(m_blk, c, neg_mc);  // exponent of the block's largest probability, as formed below
      bool top_emulated = false;
      float2 sum2 = make_float2(0.0f, 0.0f);
#pragma unroll
      for (int q4 = 0; q4 < 4; ++q4) {
        uint32_t pk[16];
        softmax_exp_chunk<D, kEmuPer8, kF16>(s[q4], pk, c, neg_mc, sum2, x_top, top_emulated);
        tmem_st16(p_addr + q4 * 16, pk);  // (D = 128: over the first half of this row's scores, all in registers)
      }
      l_run += sum2.x + sum2.y;
      l_fix += top_rounding_excess<kEmuPer8, kF16>(x_top, top_emulated);
      tmem_wait_st();
      tc_fence_before();
      __syncwarp();
      if (lane == 0) mbar_arrive(&sm.p_full);
    }

    if (ok && m0 < Sq) {
      const float inv_l = l_run > 0.0f ? 1.0f / (l_run + l_fix) : 0.0f;
      if (row < Sq) lse_rows[row] = l_run > 0.0f ? (m_run * c + log2f(l_run)) * kLn2 : -INFINITY;
      if (n > 0) {
        ok = __all_sync(0xffffffffu, mbar_wait(&sm.o_full, (n - 1) & 1, abort_flag, __LINE__));
        tc_fence_after();
      }
      if (ok) {
        uint8_t* stage = sm.q;  // no product reads Q any more
        // In a packed batch the rows after a sequence's last one belong to the next sequence, so a tile
        // that overhangs the end cannot leave through a 128-row TMA store: its rows are written one by one.
        const bool row_by_row = p.cu_q != nullptr && m0 + 128 > Sq;
        __nv_bfloat16* o_row = p.o + ((size_t)(q_row0 + min(row, Sq - 1)) * p.H + h) * D;
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
        if (!row_by_row) {  // (warp-uniform)
          fence_proxy_async_smem();
          __syncwarp();
          if (lane == 0) mbar_arrive(&sm.o_staged);
          if (w == 0) {
            ok = __all_sync(0xffffffffu, mbar_wait(&sm.o_staged, 0, abort_flag, __LINE__));
            if (ok && lane == 0) {
              for (int r = 0; r < kRegions; ++r)
                tma_store_4d(&tm_o, stage + r * kRegionBytes, r * 64, h, q_row0 + m0, b);
              tma_commit_group();
              tma_wait_group_read<0>();
            }
          }
        }
      }
    }
  } else if (warp == 4) {
    // ============================================================ MMA issue
    reg_dealloc<48>();
    if (n > 0) {
      const uint32_t q_lo = desc_lo(smem_u32(sm.q), 0), k_lo0 = desc_lo(smem_u32(sm.k[0]), 0);
      const uint32_t v_lo0 = desc_lo(smem_u32(sm.v[0]), kRegionBytes);
      constexpr uint32_t kStep = Smem::kTileBytes >> 4;
      auto wait_bar = [&](uint64_t* bar, uint32_t parity) -> bool {
        return __all_sync(0xffffffffu, mbar_wait(bar, parity, abort_flag, __LINE__));
      };
      auto do_s = [&](int j) -> bool {  // S = Q K_j^T
        const int slot = j % kStages;
        if (!wait_bar(&sm.k_full[slot], (uint32_t)((j / kStages) & 1))) return false;
        const uint32_t b_lo = k_lo0 + slot * kStep;
        if (elect_one()) {
#pragma unroll
          for (int kk = 0; kk < D / 16; ++kk) {
            const uint32_t off = ((kk / 4) * kRegionBytes + (kk % 4) * 32) >> 4;
            mma_ss_lohi(tmem, q_lo + off, b_lo + off, kDescHiSw128, kIdescS, kk > 0);
          }
          mma_commit(&sm.s_full);
          mma_commit(&sm.k_empty[slot]);
        }
        __syncwarp();
        return true;
      };
      do {
        if (!(wait_bar(&sm.q_full, 0) && do_s(0))) break;
        for (int j = 0; j < n; ++j) {
          if (kSeparateP && j + 1 < n) {  // S(j+1) under the softmax of block j
            if (!wait_bar(&sm.s_free, j & 1)) break;
            tc_fence_after();
            if (!do_s(j + 1)) break;
          }
          const int slot = j % kStages;
          if (!wait_bar(&sm.v_full[slot], (uint32_t)((j / kStages) & 1))) break;
          if (!wait_bar(&sm.p_full, j & 1)) break;
          tc_fence_after();
          const uint32_t b_lo = v_lo0 + slot * kStep;
          if (elect_one()) {  // O += P V_j
#pragma unroll
            for (int kk = 0; kk < 8; ++kk)
              mma_ts_lohi(tmem + kColO, tmem + kColP + kk * 8, b_lo + ((kk * 2048) >> 4), kDescHiSw128, kIdescO,
                          kk > 0 ? 1u : (j > 0 ? 1u : 0u));
            mma_commit(&sm.v_empty[slot]);
            mma_commit(&sm.o_full);
          }
          __syncwarp();
          if (!kSeparateP && j + 1 < n && !do_s(j + 1)) break;
        }
      } while (false);
    }
    __syncwarp();
  } else if (warp == 5) {
    // ============================================================ TMA producer
    reg_dealloc<48>();
    if (n > 0 && lane == 0) {
      // Steady state: block j reuses the stage of block j - kStages, first K's (released when S(j - kStages)
      // has finished), then V's (when O += P V_{j - kStages} has).
      for (int j = kStages; j < n; ++j) {
        const int slot = j % kStages;
        const uint32_t parity = (uint32_t)((j / kStages - 1) & 1);
        if (!mbar_wait(&sm.k_empty[slot], parity, abort_flag, __LINE__)) break;
        load_k(j, slot);
        if (!mbar_wait(&sm.v_empty[slot], parity, abort_flag, __LINE__)) break;
        load_v(j, slot);
      }
    }
    __syncwarp();
  } else {
    reg_dealloc<48>();
  }

  tc_fence_before();
  __syncthreads();
  if (warp == 4) tmem_dealloc(tmem, 256);
}

}  // namespace fa

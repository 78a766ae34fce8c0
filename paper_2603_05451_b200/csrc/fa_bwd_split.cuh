// Backward pass as two kernels without any global reduction.
//
// The paper's backward (Section 3.2) forms all five products in one kernel that owns a key/value
// tile and adds each dQ_i tile into global memory.  On this GPU those FP32 reductions are the
// limiter: 64 KiB per 128 x 128 tile pair, while the L2 reduces at most ~4.9 TB/s with nothing
// else running (3770 SM clocks per tile over 148 SMs, against 2560 clocks of MMA).  Splitting the
// work removes the reductions at the price of recomputing S and dP once more (7 MMAs instead of 5):
//
//   bwd_dkdv_kernel  CTA = one 128-row key/value tile, loops over query tiles:
//                    S^T = K Q_i^T, P^T, dP^T = V dO_i^T, dV += P^T dO_i, dS^T, dK += dS^T Q_i
//   bwd_dq_kernel    CTA = one 128-row query tile, loops over key/value tiles:
//                    S = Q K_j^T, P, dP = dO V_j^T, dS, dQ += dS K_j
//
// Both keep P / dS in tensor memory as the A operand of the accumulating product, use the same
// roles as the forward kernel (two compute warpgroups with one thread per row and half of the
// columns each, one MMA-issuing warp, one TMA warp) and talk through mbarriers with bounded
// waits.  dQ, dK and dV are written once, in a fixed summation order: the whole backward is
// bit-reproducible, and the only scratch left is the two FP32 row vectors (Delta and LSE*log2e).
#pragma once

#include "fa_bwd_kernels.cuh"

namespace fa {

// ============================================================================ dK / dV
template <int D>
struct BwdDkdvSmem {
  static constexpr int kTileBytes = 128 * D * 2;
  alignas(1024) uint8_t k[kTileBytes];
  alignas(1024) uint8_t v[kTileBytes];
  alignas(1024) uint8_t q[2][kTileBytes];    // Q_i stages; q[0] stages dK in the epilogue
  alignas(1024) uint8_t d_o[2][kTileBytes];  // dO_i stages; d_o[0] stages dV in the epilogue
  alignas(16) float lse2[2][128];
  alignas(16) float delta[2][128];
  alignas(8) uint64_t kv_full;
  uint64_t q_full[2], do_full[2], stage_empty[2];
  uint64_t s_full, p_ready, dp_full, ds_ready, acc_full, out_staged;
  uint32_t tmem_base;
  WaitCtl ctl;  // abort flag and launch epoch, read by every bounded wait
};

template <int D, bool kF16 = false>
__global__ void __launch_bounds__(512, 1)
bwd_dkdv_kernel(const __grid_constant__ CUtensorMap tm_q, const __grid_constant__ CUtensorMap tm_k,
                const __grid_constant__ CUtensorMap tm_v, const __grid_constant__ CUtensorMap tm_do,
                const __grid_constant__ CUtensorMap tm_dk, const __grid_constant__ CUtensorMap tm_dv,
                const BwdParams p, const int n_kv_tiles) {
  extern __shared__ __align__(1024) uint8_t smem_raw[];
  using Smem = BwdDkdvSmem<D>;
  Smem& sm = *reinterpret_cast<Smem*>(smem_raw);
  if ((smem_u32(smem_raw) & 1023u) != 0) {
    if (threadIdx.x == 0) record_device_status(5, __LINE__, p.epoch);
    return;
  }
  constexpr int kRegions = D / 64;
  constexpr int kRegionBytes = 128 * 128;
  constexpr uint32_t kIdescSS = make_idesc(128, 128, false, false, kF16);  // S^T, dP^T: both operands K-major
  constexpr uint32_t kIdescAcc = make_idesc(128, D, false, true, kF16);    // dV, dK: A in TMEM, B MN-major
  constexpr uint32_t kColR0 = 0, kColR1 = 128, kColDv = 256, kColDk = 384;

  const int tid = threadIdx.x, warp = tid >> 5, lane = tid & 31;
  volatile int* abort_flag = &sm.ctl.abort_flag;

  // work decode: key tiles ascending (with a causal mask the first tile sees the most queries), kv heads, batches
  const int n_tile = blockIdx.x % n_kv_tiles;
  const int hk = (blockIdx.x / n_kv_tiles) % p.Hkv;
  const int b = blockIdx.x / (n_kv_tiles * p.Hkv);
  const int j0 = n_tile * 128;
  const int group = p.H / p.Hkv;
  const int shift = p.Sk - p.Sq;
  const int n_q_tiles = (p.Sq + 127) / 128;
  const int q_first = p.causal ? max(0, j0 - shift) : 0;  // first query that sees key j0
  const int i_first = min(n_q_tiles, q_first / 128);
  const int iters_per_head = n_q_tiles - i_first;
  const int n_iter = iters_per_head * group;

  if (tid == 0) {
    sm.ctl.abort_flag = 0;
    sm.ctl.launch_epoch = (int)p.epoch;
    mbar_init(&sm.kv_full, 1);
    for (int s = 0; s < 2; ++s) {
      mbar_init(&sm.q_full[s], 1);
      mbar_init(&sm.do_full[s], 1);
      mbar_init(&sm.stage_empty[s], 1);
    }
    mbar_init(&sm.s_full, 1);
    mbar_init(&sm.p_ready, 8);
    mbar_init(&sm.dp_full, 1);
    mbar_init(&sm.ds_ready, 8);
    mbar_init(&sm.acc_full, 1);
    mbar_init(&sm.out_staged, 8);
    fence_barrier_init();
  }
  if (warp == 12) {
    tmem_alloc(&sm.tmem_base, 512);
    tmem_relinquish();
  }
  tc_fence_before();
  __syncthreads();
  tc_fence_after();
  const uint32_t tmem = sm.tmem_base;

  if (warp < 8) {
    // ------------------------------------------------------------ compute warpgroups (thread = key row)
    reg_alloc<192>();
    const int wg = warp >> 2, w = warp & 3;
    const int r = w * 32 + lane;
    const int key = j0 + r;
    const uint32_t lane_base = (uint32_t)(w * 32) << 16;
    // each warpgroup works on its own 64 fp32 columns and writes its packed bf16 results over their first half
    const uint32_t s_addr = tmem + kColR0 + lane_base + wg * 64;
    const uint32_t dp_addr = tmem + kColR1 + lane_base + wg * 64;
    const float c = p.scale_log2;
    bool ok = true;
    for (int it = 0; it < n_iter; ++it) {
      const int stage = it & 1;
      const int i = i_first + it % iters_per_head;
      const int q0 = i * 128 + wg * 64;
      ok = __all_sync(0xffffffffu, mbar_wait(&sm.s_full, it & 1, abort_flag));
      if (!ok) break;
      tc_fence_after();
      uint32_t s[2][32];
      tmem_ld32(s_addr, s[0]);
      tmem_ld32(s_addr + 32, s[1]);
      tmem_wait_ld();
      const bool masked = p.causal && (j0 + 127 > i * 128 + shift);  // key `key` is visible to query q iff key <= q + shift
      if (masked) {  // only tiles on the diagonal pay for the test
        const int first_visible = key - q0 - shift;  // columns below it are queries that do not see this key
#pragma unroll
        for (int h2 = 0; h2 < 2; ++h2) {
#pragma unroll
          for (int col = 0; col < 32; ++col)
            if (h2 * 32 + col < first_visible) s[h2][col] = 0xff800000u;  // -inf
        }
      }
      float pr[2][32];
      const float4* lse4 = reinterpret_cast<const float4*>(&sm.lse2[stage][wg * 64]);
#pragma unroll
      for (int h2 = 0; h2 < 2; ++h2) {
#pragma unroll
        for (int g = 0; g < 8; ++g) {
          const float4 l4 = lse4[h2 * 8 + g];
          const float ls[4] = {l4.x, l4.y, l4.z, l4.w};
#pragma unroll
          for (int e = 0; e < 4; ++e) {
            const int col = g * 4 + e;
            pr[h2][col] = ex2_approx(fmaf(__uint_as_float(s[h2][col]), c, -ls[e]));
          }
        }
        uint32_t pk[16];
#pragma unroll
        for (int e = 0; e < 16; ++e) pk[e] = pack2<kF16>(pr[h2][2 * e], pr[h2][2 * e + 1]);
        tmem_st16(s_addr + h2 * 16, pk);
      }
      tmem_wait_st();
      tc_fence_before();
      __syncwarp();
      if (lane == 0) mbar_arrive(&sm.p_ready);

      ok = __all_sync(0xffffffffu, mbar_wait(&sm.dp_full, it & 1, abort_flag));
      if (!ok) break;
      tc_fence_after();
      uint32_t dp[2][32];
      tmem_ld32(dp_addr, dp[0]);
      tmem_ld32(dp_addr + 32, dp[1]);
      tmem_wait_ld();
      const float4* dl4 = reinterpret_cast<const float4*>(&sm.delta[stage][wg * 64]);
#pragma unroll
      for (int h2 = 0; h2 < 2; ++h2) {
        uint32_t pk[16];
#pragma unroll
        for (int g = 0; g < 8; ++g) {
          const float4 d4 = dl4[h2 * 8 + g];
          const float d0 = pr[h2][g * 4 + 0] * (__uint_as_float(dp[h2][g * 4 + 0]) - d4.x);
          const float d1 = pr[h2][g * 4 + 1] * (__uint_as_float(dp[h2][g * 4 + 1]) - d4.y);
          const float d2 = pr[h2][g * 4 + 2] * (__uint_as_float(dp[h2][g * 4 + 2]) - d4.z);
          const float d3 = pr[h2][g * 4 + 3] * (__uint_as_float(dp[h2][g * 4 + 3]) - d4.w);
          pk[g * 2] = pack2<kF16>(d0, d1);
          pk[g * 2 + 1] = pack2<kF16>(d2, d3);
        }
        tmem_st16(dp_addr + h2 * 16, pk);
      }
      tmem_wait_st();
      tc_fence_before();
      __syncwarp();
      if (lane == 0) mbar_arrive(&sm.ds_ready);
    }

    // epilogue: dV and dK * scale -> bf16 -> shared memory (swizzled) -> TMA store
    if (ok) {
      if (n_iter > 0) {
        ok = __all_sync(0xffffffffu, mbar_wait(&sm.acc_full, 0, abort_flag));
        tc_fence_after();
      }
      if (ok) {
        constexpr int kHalf = D / 2;
#pragma unroll
        for (int which = 0; which < 2; ++which) {
          const uint32_t acc_addr = tmem + (which == 0 ? kColDv : kColDk) + lane_base + wg * kHalf;
          uint8_t* stage_buf = which == 0 ? sm.d_o[0] : sm.q[0];
          const float mul = which == 0 ? 1.0f : p.scale;
#pragma unroll
          for (int cc = 0; cc < kHalf / 32; ++cc) {
            uint32_t v[32];
            if (n_iter > 0) {
              tmem_ld32(acc_addr + cc * 32, v);
              tmem_wait_ld();
            } else {
#pragma unroll
              for (int e = 0; e < 32; ++e) v[e] = 0u;
            }
            const int col0 = wg * kHalf + cc * 32;
            uint8_t* row_ptr = stage_buf + (col0 / 64) * kRegionBytes + r * 128;
#pragma unroll
            for (int ch = 0; ch < 4; ++ch) {
              uint4 w4;
              w4.x = pack2<kF16>(__uint_as_float(v[8 * ch + 0]) * mul, __uint_as_float(v[8 * ch + 1]) * mul);
              w4.y = pack2<kF16>(__uint_as_float(v[8 * ch + 2]) * mul, __uint_as_float(v[8 * ch + 3]) * mul);
              w4.z = pack2<kF16>(__uint_as_float(v[8 * ch + 4]) * mul, __uint_as_float(v[8 * ch + 5]) * mul);
              w4.w = pack2<kF16>(__uint_as_float(v[8 * ch + 6]) * mul, __uint_as_float(v[8 * ch + 7]) * mul);
              const int chunk = (col0 % 64) / 8 + ch;
              *reinterpret_cast<uint4*>(row_ptr + ((chunk ^ (r & 7)) << 4)) = w4;
            }
          }
        }
        fence_proxy_async_smem();
        __syncwarp();
        if (lane == 0) mbar_arrive(&sm.out_staged);
        if (warp == 0) {
          ok = __all_sync(0xffffffffu, mbar_wait(&sm.out_staged, 0, abort_flag));
          if (ok && lane == 0) {
            for (int rg = 0; rg < kRegions; ++rg) {
              tma_store_4d(&tm_dv, sm.d_o[0] + rg * kRegionBytes, rg * 64, hk, j0, b);
              tma_store_4d(&tm_dk, sm.q[0] + rg * kRegionBytes, rg * 64, hk, j0, b);
            }
            tma_commit_group();
            tma_wait_group_read<0>();
          }
        }
      }
    }
  } else if (warp == 12) {
    // ------------------------------------------------------------ MMA issuer (warp-uniform, elected lane issues)
    reg_dealloc<48>();
    if (n_iter > 0) {
      constexpr uint32_t kStageStep = Smem::kTileBytes >> 4;
      const uint32_t k_lo = desc_lo(smem_u32(sm.k), 16), v_lo = desc_lo(smem_u32(sm.v), 16);
      const uint32_t q_lo0 = desc_lo(smem_u32(sm.q[0]), 16), do_lo0 = desc_lo(smem_u32(sm.d_o[0]), 16);
      const uint32_t q_mn_lo0 = desc_lo(smem_u32(sm.q[0]), kRegionBytes);     // Q_i as MN-major B of dK
      const uint32_t do_mn_lo0 = desc_lo(smem_u32(sm.d_o[0]), kRegionBytes);  // dO_i as MN-major B of dV
      auto wait_bar = [&](uint64_t* bar, uint32_t parity) {
        return __all_sync(0xffffffffu, mbar_wait(bar, parity, abort_flag));
      };
      auto ss_kmajor = [&](uint32_t d_col, uint32_t a_lo, uint32_t b_lo, uint64_t* bar) {
        if (elect_one()) {
#pragma unroll
          for (int kk = 0; kk < D / 16; ++kk) {
            const uint32_t off = ((kk / 4) * kRegionBytes + (kk % 4) * 32) >> 4;
            mma_ss_lohi(tmem + d_col, a_lo + off, b_lo + off, kDescHiSw128, kIdescSS, kk > 0);
          }
          mma_commit(bar);
        }
        __syncwarp();
      };
      auto ts_acc = [&](uint32_t d_col, uint32_t a_col, uint32_t b_mn_lo, uint32_t accumulate) {
        if (elect_one()) {
#pragma unroll
          for (int kk = 0; kk < 8; ++kk)
            mma_ts_lohi(tmem + d_col, tmem + a_col + (kk / 4) * 64 + (kk % 4) * 8, b_mn_lo + ((kk * 2048) >> 4),
                        kDescHiSw128, kIdescAcc, kk > 0 ? 1u : accumulate);
        }
        __syncwarp();
      };
      do {
        if (!wait_bar(&sm.kv_full, 0)) break;
        if (!wait_bar(&sm.q_full[0], 0)) break;
        ss_kmajor(kColR0, k_lo, q_lo0, &sm.s_full);  // S^T(0)
        bool ok = true;
        for (int it = 0; it < n_iter; ++it) {
          const int stage = it & 1;
          const uint32_t sphase = (it >> 1) & 1;
          if (!(ok = wait_bar(&sm.do_full[stage], sphase))) break;
          ss_kmajor(kColR1, v_lo, do_lo0 + stage * kStageStep, &sm.dp_full);  // dP^T(it): after dK(it-1) in issue order
          if (!(ok = wait_bar(&sm.p_ready, it & 1))) break;
          tc_fence_after();
          ts_acc(kColDv, kColR0, do_mn_lo0 + stage * kStageStep, it > 0 ? 1u : 0u);  // dV += P^T dO
          if (it + 1 < n_iter) {
            if (!(ok = wait_bar(&sm.q_full[stage ^ 1], ((it + 1) >> 1) & 1))) break;
            ss_kmajor(kColR0, k_lo, q_lo0 + (stage ^ 1) * kStageStep, &sm.s_full);  // S^T(it + 1)
          }
          if (!(ok = wait_bar(&sm.ds_ready, it & 1))) break;
          tc_fence_after();
          ts_acc(kColDk, kColR1, q_mn_lo0 + stage * kStageStep, it > 0 ? 1u : 0u);  // dK += dS^T Q
          if (elect_one()) mma_commit(&sm.stage_empty[stage]);
          __syncwarp();
        }
        if (ok) {
          if (elect_one()) mma_commit(&sm.acc_full);
          __syncwarp();
        }
      } while (false);
    }
  } else if (warp == 13) {
    // ------------------------------------------------------------ TMA producer
    reg_dealloc<48>();
    if (n_iter > 0 && lane == 0) {
      mbar_expect_tx(&sm.kv_full, 2 * Smem::kTileBytes);
      for (int rg = 0; rg < kRegions; ++rg) {
        tma_load_4d(sm.k + rg * kRegionBytes, &tm_k, &sm.kv_full, rg * 64, hk, j0, b);
        tma_load_4d(sm.v + rg * kRegionBytes, &tm_v, &sm.kv_full, rg * 64, hk, j0, b);
      }
      for (int it = 0; it < n_iter; ++it) {
        const int stage = it & 1;
        const int h = hk * group + it / iters_per_head;
        const int i = i_first + it % iters_per_head;
        if (it >= 2 && !mbar_wait(&sm.stage_empty[stage], ((it >> 1) - 1) & 1, abort_flag)) break;
        const size_t row_off = ((size_t)b * p.H + h) * p.Sq_pad + (size_t)i * 128;
        mbar_expect_tx(&sm.q_full[stage], Smem::kTileBytes + 512);
        for (int rg = 0; rg < kRegions; ++rg)
          tma_load_4d(sm.q[stage] + rg * kRegionBytes, &tm_q, &sm.q_full[stage], rg * 64, h, i * 128, b);
        bulk_load_1d(sm.lse2[stage], p.lse2 + row_off, 512, &sm.q_full[stage]);
        mbar_expect_tx(&sm.do_full[stage], Smem::kTileBytes + 512);
        for (int rg = 0; rg < kRegions; ++rg)
          tma_load_4d(sm.d_o[stage] + rg * kRegionBytes, &tm_do, &sm.do_full[stage], rg * 64, h, i * 128, b);
        bulk_load_1d(sm.delta[stage], p.delta + row_off, 512, &sm.do_full[stage]);
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

// ============================================================================ dQ
template <int D>
struct BwdDqSmem {
  static constexpr int kTileBytes = 128 * D * 2;
  alignas(1024) uint8_t q[kTileBytes];       // resident; stages dQ in the epilogue
  alignas(1024) uint8_t d_o[kTileBytes];     // resident
  alignas(1024) uint8_t k[2][kTileBytes];    // K_j stages
  alignas(1024) uint8_t v[2][kTileBytes];    // V_j stages
  alignas(16) float lse2[128];
  alignas(16) float delta[128];
  alignas(8) uint64_t q_full;
  uint64_t kv_full[2], kv_empty[2];
  uint64_t s_full, s_free, dp_full[2], ds_ready, acc_full, out_staged;  // dp_full: one per ping-pong region
  uint32_t tmem_base;
  WaitCtl ctl;  // abort flag and launch epoch, read by every bounded wait
};

template <int D, bool kF16 = false>
__global__ void __launch_bounds__(512, 1)
bwd_dq_kernel(const __grid_constant__ CUtensorMap tm_q, const __grid_constant__ CUtensorMap tm_k,
              const __grid_constant__ CUtensorMap tm_v, const __grid_constant__ CUtensorMap tm_do,
              const __grid_constant__ CUtensorMap tm_dq, const BwdParams p, const int n_q_tiles) {
  extern __shared__ __align__(1024) uint8_t smem_raw[];
  using Smem = BwdDqSmem<D>;
  Smem& sm = *reinterpret_cast<Smem*>(smem_raw);
  if ((smem_u32(smem_raw) & 1023u) != 0) {
    if (threadIdx.x == 0) record_device_status(5, __LINE__, p.epoch);
    return;
  }
  constexpr int kRegions = D / 64;
  constexpr int kRegionBytes = 128 * 128;
  constexpr uint32_t kIdescSS = make_idesc(128, 128, false, false, kF16);  // S, dP: both operands K-major
  constexpr uint32_t kIdescAcc = make_idesc(128, D, false, true, kF16);    // dQ: A (dS) in TMEM, B (K_j) MN-major
  // tensor memory: S [0,128); dP/dS ping-pong [128,256) and [256,384); dQ accumulator [384, 384+D)
  constexpr uint32_t kColS = 0, kColDp0 = 128, kColDq = 384;

  const int tid = threadIdx.x, warp = tid >> 5, lane = tid & 31;
  volatile int* abort_flag = &sm.ctl.abort_flag;

  // work decode: batches outermost, query tiles from the LAST one down (longest first under a causal mask), heads fastest
  const int h = blockIdx.x % p.H;
  const int rest = blockIdx.x / p.H;
  const int i = n_q_tiles - 1 - rest % n_q_tiles;
  const int b = rest / n_q_tiles;
  const int hk = h / (p.H / p.Hkv);
  const int q0 = i * 128;
  const int shift = p.Sk - p.Sq;
  const int n_kv_tiles = (p.Sk + 127) / 128;
  // key tiles that some row of this query tile can see
  int n_iter = n_kv_tiles;
  if (p.causal) {
    const int last_key = min(p.Sk - 1, q0 + 127 + shift);
    n_iter = last_key >= 0 ? min(n_kv_tiles, last_key / 128 + 1) : 0;
  }

  if (tid == 0) {
    sm.ctl.abort_flag = 0;
    sm.ctl.launch_epoch = (int)p.epoch;
    mbar_init(&sm.q_full, 1);
    for (int s = 0; s < 2; ++s) {
      mbar_init(&sm.kv_full[s], 1);
      mbar_init(&sm.kv_empty[s], 1);
    }
    mbar_init(&sm.s_full, 1);
    mbar_init(&sm.s_free, 8);
    mbar_init(&sm.dp_full[0], 1);
    mbar_init(&sm.dp_full[1], 1);
    mbar_init(&sm.ds_ready, 8);
    mbar_init(&sm.acc_full, 1);
    mbar_init(&sm.out_staged, 8);
    fence_barrier_init();
  }
  if (warp == 12) {
    tmem_alloc(&sm.tmem_base, 512);
    tmem_relinquish();
  }
  tc_fence_before();
  __syncthreads();
  tc_fence_after();
  const uint32_t tmem = sm.tmem_base;

  if (warp < 8) {
    // ------------------------------------------------------------ compute warpgroups (thread = query row)
    reg_alloc<192>();
    const int wg = warp >> 2, w = warp & 3;
    const int r = w * 32 + lane;
    const int row = q0 + r;
    const uint32_t lane_base = (uint32_t)(w * 32) << 16;
    const uint32_t s_addr = tmem + kColS + lane_base + wg * 64;
    const float c = p.scale_log2;
    bool ok = true;
    float my_lse2 = INFINITY, my_delta = 0.0f;
    if (n_iter > 0) {
      ok = __all_sync(0xffffffffu, mbar_wait(&sm.q_full, 0, abort_flag));
      if (ok) {
        my_lse2 = sm.lse2[r];
        my_delta = sm.delta[r];
      }
    }
    for (int j = 0; j < n_iter && ok; ++j) {
      const uint32_t dp_addr = tmem + kColDp0 + (j & 1) * 128 + lane_base + wg * 64;
      const int key0 = j * 128 + wg * 64;
      ok = __all_sync(0xffffffffu, mbar_wait(&sm.s_full, j & 1, abort_flag));
      if (!ok) break;
      tc_fence_after();
      uint32_t s[2][32];
      tmem_ld32(s_addr, s[0]);
      tmem_ld32(s_addr + 32, s[1]);
      tmem_wait_ld();
      // the scores are in registers: S_{j+1} may be written
      tc_fence_before();
      __syncwarp();
      if (lane == 0) mbar_arrive(&sm.s_free);
      const bool masked = p.causal && (j * 128 + 127 > q0 + shift);  // key visible to `row` iff key <= row + shift
      if (masked) {  // only tiles on the diagonal pay for the test
        const int last_visible = row + shift - key0;  // columns above it are keys this query does not see
#pragma unroll
        for (int h2 = 0; h2 < 2; ++h2)
#pragma unroll
          for (int e = 0; e < 32; ++e)
            if (h2 * 32 + e > last_visible) s[h2][e] = 0xff800000u;  // -inf
      }
      float pr[2][32];
#pragma unroll
      for (int h2 = 0; h2 < 2; ++h2)
#pragma unroll
        for (int e = 0; e < 32; ++e) pr[h2][e] = ex2_approx(fmaf(__uint_as_float(s[h2][e]), c, -my_lse2));
      ok = __all_sync(0xffffffffu, mbar_wait(&sm.dp_full[j & 1], (j >> 1) & 1, abort_flag));
      if (!ok) break;
      tc_fence_after();
      uint32_t dp[2][32];
      tmem_ld32(dp_addr, dp[0]);
      tmem_ld32(dp_addr + 32, dp[1]);
      tmem_wait_ld();
#pragma unroll
      for (int h2 = 0; h2 < 2; ++h2) {
        uint32_t pk[16];
#pragma unroll
        for (int e = 0; e < 16; ++e)
          pk[e] = pack2<kF16>(pr[h2][2 * e] * (__uint_as_float(dp[h2][2 * e]) - my_delta),
                              pr[h2][2 * e + 1] * (__uint_as_float(dp[h2][2 * e + 1]) - my_delta));
        tmem_st16(dp_addr + h2 * 16, pk);
      }
      tmem_wait_st();
      tc_fence_before();
      __syncwarp();
      if (lane == 0) mbar_arrive(&sm.ds_ready);
    }

    // epilogue: dQ * scale -> bf16 -> shared memory (swizzled) -> TMA store
    if (ok) {
      if (n_iter > 0) {
        ok = __all_sync(0xffffffffu, mbar_wait(&sm.acc_full, 0, abort_flag));
        tc_fence_after();
      }
      if (ok) {
        constexpr int kHalf = D / 2;
        const uint32_t acc_addr = tmem + kColDq + lane_base + wg * kHalf;
#pragma unroll
        for (int cc = 0; cc < kHalf / 32; ++cc) {
          uint32_t v[32];
          if (n_iter > 0) {
            tmem_ld32(acc_addr + cc * 32, v);
            tmem_wait_ld();
          } else {
#pragma unroll
            for (int e = 0; e < 32; ++e) v[e] = 0u;
          }
          const int col0 = wg * kHalf + cc * 32;
          uint8_t* row_ptr = sm.q + (col0 / 64) * kRegionBytes + r * 128;
#pragma unroll
          for (int ch = 0; ch < 4; ++ch) {
            uint4 w4;
            w4.x = pack2<kF16>(__uint_as_float(v[8 * ch + 0]) * p.scale, __uint_as_float(v[8 * ch + 1]) * p.scale);
            w4.y = pack2<kF16>(__uint_as_float(v[8 * ch + 2]) * p.scale, __uint_as_float(v[8 * ch + 3]) * p.scale);
            w4.z = pack2<kF16>(__uint_as_float(v[8 * ch + 4]) * p.scale, __uint_as_float(v[8 * ch + 5]) * p.scale);
            w4.w = pack2<kF16>(__uint_as_float(v[8 * ch + 6]) * p.scale, __uint_as_float(v[8 * ch + 7]) * p.scale);
            const int chunk = (col0 % 64) / 8 + ch;
            *reinterpret_cast<uint4*>(row_ptr + ((chunk ^ (r & 7)) << 4)) = w4;
          }
        }
        fence_proxy_async_smem();
        __syncwarp();
        if (lane == 0) mbar_arrive(&sm.out_staged);
        if (warp == 0) {
          ok = __all_sync(0xffffffffu, mbar_wait(&sm.out_staged, 0, abort_flag));
          if (ok && lane == 0) {
            for (int rg = 0; rg < kRegions; ++rg) tma_store_4d(&tm_dq, sm.q + rg * kRegionBytes, rg * 64, h, q0, b);
            tma_commit_group();
            tma_wait_group_read<0>();
          }
        }
      }
    }
  } else if (warp == 12) {
    // ------------------------------------------------------------ MMA issuer
    reg_dealloc<48>();
    if (n_iter > 0) {
      constexpr uint32_t kStageStep = Smem::kTileBytes >> 4;
      const uint32_t q_lo = desc_lo(smem_u32(sm.q), 16), do_lo = desc_lo(smem_u32(sm.d_o), 16);
      const uint32_t k_lo0 = desc_lo(smem_u32(sm.k[0]), 16), v_lo0 = desc_lo(smem_u32(sm.v[0]), 16);
      const uint32_t k_mn_lo0 = desc_lo(smem_u32(sm.k[0]), kRegionBytes);  // K_j as MN-major B of dQ
      auto wait_bar = [&](uint64_t* bar, uint32_t parity) {
        return __all_sync(0xffffffffu, mbar_wait(bar, parity, abort_flag));
      };
      auto ss_kmajor = [&](uint32_t d_col, uint32_t a_lo, uint32_t b_lo, uint64_t* bar) {
        if (elect_one()) {
#pragma unroll
          for (int kk = 0; kk < D / 16; ++kk) {
            const uint32_t off = ((kk / 4) * kRegionBytes + (kk % 4) * 32) >> 4;
            mma_ss_lohi(tmem + d_col, a_lo + off, b_lo + off, kDescHiSw128, kIdescSS, kk > 0);
          }
          mma_commit(bar);
        }
        __syncwarp();
      };
      do {
        if (!wait_bar(&sm.q_full, 0)) break;
        if (!wait_bar(&sm.kv_full[0], 0)) break;
        ss_kmajor(kColS, q_lo, k_lo0, &sm.s_full);      // S(0)
        ss_kmajor(kColDp0, do_lo, v_lo0, &sm.dp_full[0]);  // dP(0)
        bool ok = true;
        for (int j = 0; j < n_iter; ++j) {
          const int stage = j & 1;
          if (j + 1 < n_iter) {
            // next block's S and dP go out before this block's dS is waited for, so the tensor pipe stays busy
            if (!(ok = wait_bar(&sm.kv_full[stage ^ 1], ((j + 1) >> 1) & 1))) break;
            if (!(ok = wait_bar(&sm.s_free, j & 1))) break;
            tc_fence_after();
            ss_kmajor(kColS, q_lo, k_lo0 + (stage ^ 1) * kStageStep, &sm.s_full);
            // dP(j+1) lands in the other ping-pong region; its previous user dQ(j-1) precedes it in issue order
            ss_kmajor(kColDp0 + ((j + 1) & 1) * 128, do_lo, v_lo0 + (stage ^ 1) * kStageStep,
                      &sm.dp_full[(j + 1) & 1]);
          }
          if (!(ok = wait_bar(&sm.ds_ready, j & 1))) break;
          tc_fence_after();
          if (elect_one()) {
            const uint32_t a_col = kColDp0 + (j & 1) * 128;
            const uint32_t b_lo = k_mn_lo0 + stage * kStageStep;
#pragma unroll
            for (int kk = 0; kk < 8; ++kk)  // dQ += dS K_j, reduction over the block's 128 keys
              mma_ts_lohi(tmem + kColDq, tmem + a_col + (kk / 4) * 64 + (kk % 4) * 8, b_lo + ((kk * 2048) >> 4),
                          kDescHiSw128, kIdescAcc, (j > 0 || kk > 0) ? 1u : 0u);
            mma_commit(&sm.kv_empty[stage]);
          }
          __syncwarp();
        }
        if (ok) {
          if (elect_one()) mma_commit(&sm.acc_full);
          __syncwarp();
        }
      } while (false);
    }
  } else if (warp == 13) {
    // ------------------------------------------------------------ TMA producer
    reg_dealloc<48>();
    if (n_iter > 0 && lane == 0) {
      const size_t row_off = ((size_t)b * p.H + h) * p.Sq_pad + (size_t)q0;
      mbar_expect_tx(&sm.q_full, 2 * Smem::kTileBytes + 1024);
      for (int rg = 0; rg < kRegions; ++rg) {
        tma_load_4d(sm.q + rg * kRegionBytes, &tm_q, &sm.q_full, rg * 64, h, q0, b);
        tma_load_4d(sm.d_o + rg * kRegionBytes, &tm_do, &sm.q_full, rg * 64, h, q0, b);
      }
      bulk_load_1d(sm.lse2, p.lse2 + row_off, 512, &sm.q_full);
      bulk_load_1d(sm.delta, p.delta + row_off, 512, &sm.q_full);
      for (int j = 0; j < n_iter; ++j) {
        const int stage = j & 1;
        if (j >= 2 && !mbar_wait(&sm.kv_empty[stage], ((j >> 1) - 1) & 1, abort_flag)) break;
        mbar_expect_tx(&sm.kv_full[stage], 2 * Smem::kTileBytes);
        for (int rg = 0; rg < kRegions; ++rg) {
          tma_load_4d(sm.k[stage] + rg * kRegionBytes, &tm_k, &sm.kv_full[stage], rg * 64, hk, j * 128, b);
          tma_load_4d(sm.v[stage] + rg * kRegionBytes, &tm_v, &sm.kv_full[stage], rg * 64, hk, j * 128, b);
        }
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

// Backward main kernel on CTA pairs (paper Section 3.2, "2-CTA" backward) for head dimension 128.
//
// A cluster of two CTAs owns 256 key rows of one (batch, kv head): CTA `rank` holds K, V and the
// dK/dV accumulators of key rows [128 rank, 128 rank + 128).  For every query tile Q_i (128 rows)
// the even CTA issues, for both SMs at once (tcgen05 cta_group::2):
//   S^T  = K Q_i^T        M = 256 keys, N = 128 queries     (each CTA stages 64 query rows of Q_i)
//   dP^T = V dO_i^T       M = 256,      N = 128             (each CTA stages 64 rows of dO_i)
//   dV  += P^T dO_i       M = 256,      N = 128 head dims   (each CTA stages 64 columns of dO_i)
//   dK  += dS^T Q_i       M = 256,      N = 128             (each CTA stages 64 columns of Q_i)
//   dQ^T = K^T dS^T       M = 128 head dims (64 per CTA), N = 128 queries, reduction over all 256 keys
// so each SM reads only half of every B operand from its shared memory, and each CTA reduces a
// 64 x 128 half of dQ_i per 256 keys instead of a full tile per 128 keys (Table 3).  For the last
// product a CTA needs dS^T of the pair's 256 keys for its 64 query columns: the half computed by the
// other CTA arrives through distributed shared memory stores.
//
// Shared-memory descriptors of a pair MMA are offsets that both CTAs apply to their own memory,
// hence every operand buffer sits at the same offset in the two CTAs and the Q_i / dO_i tiles are
// staged twice (by rows for the first two products, by columns for the next two).
#pragma once

#include "fa_bwd_fused.cuh"

namespace fa {

struct BwdPairSmem {
  static constexpr int kTileBytes = 128 * 128 * 2;
  static constexpr int kHalfBytes = kTileBytes / 2;
  alignas(1024) uint8_t k[kTileBytes];        // own K rows: two [128][64] regions
  alignas(1024) uint8_t v[kTileBytes];        // own V rows
  alignas(1024) uint8_t k_dq[kTileBytes];     // K rows of the whole pair, this CTA's 64 head dims: [256][64]
  alignas(1024) uint8_t q_rows[2][kHalfBytes];  // Q_i rows [64 rank, +64): two [64][64] regions (two stages);
                                                // both stages together stage dK in the epilogue
  alignas(1024) uint8_t q_cols[kHalfBytes];   // Q_i, this CTA's 64 head dims: [128][64]
  alignas(1024) uint8_t do_rows[kHalfBytes];  // dO_i rows [64 rank, +64); with do_cols stages dV in the epilogue
  alignas(1024) uint8_t do_cols[kHalfBytes];  // dO_i, this CTA's 64 head dims
  alignas(1024) uint8_t ds[kTileBytes];       // dS^T of the pair, this CTA's 64 queries: [256 keys][64]
  alignas(1024) float red_slot[4][32 * 32];   // [warp][query][head dim]: one 4 KiB bulk reduce each
  alignas(16) float lse2[2][128];
  alignas(16) float delta[2][128];
  // barriers marked (L) are used in the leader CTA only and collect arrivals or bytes from both
  // CTAs; the others are signalled in both CTAs by one multicast commit, or are local
  alignas(8) uint64_t kv_full;             // (L)
  uint64_t qr_full[2], qc_full, do_full;   // (L)
  uint64_t qr_empty[2], qc_empty, do_empty;
  uint64_t stat_full[2];                   // local: lse2/delta of a stage have landed
  uint64_t s_full, dp_full, dq_full, acc_full;
  uint64_t p_ready, ds_ready, dq_drained;  // (L)
  uint64_t ds_in;                          // local: the other CTA's half of dS^T has landed in `ds`
  uint64_t out_staged;                     // local
  uint32_t tmem_base;
  WaitCtl ctl;  // abort flag and launch epoch, read by every bounded wait
};
static_assert(sizeof(BwdPairSmem) <= 227 * 1024, "pair kernel shared memory");


__global__ void __cluster_dims__(2, 1, 1) __launch_bounds__(512, 1)
bwd_pair_kernel(const __grid_constant__ CUtensorMap tm_q, const __grid_constant__ CUtensorMap tm_q64,
                const __grid_constant__ CUtensorMap tm_k, const __grid_constant__ CUtensorMap tm_v,
                const __grid_constant__ CUtensorMap tm_do, const __grid_constant__ CUtensorMap tm_do64,
                const __grid_constant__ CUtensorMap tm_dk, const __grid_constant__ CUtensorMap tm_dv,
                const BwdParams p, const int n_kv_pairs) {
  constexpr int D = 128;
  extern __shared__ __align__(1024) uint8_t smem_raw[];
  using Smem = BwdPairSmem;
  Smem& sm = *reinterpret_cast<Smem*>(smem_raw);
  if ((smem_u32(smem_raw) & 1023u) != 0) {  // same in both CTAs of a pair, so both leave
    if (threadIdx.x == 0) record_device_status(5, __LINE__, p.epoch);
    return;
  }
  constexpr int kRegionBytes = 128 * 128;  // [128 rows][64 bf16]
  constexpr int kHalfRegionBytes = 64 * 128;  // [64 rows][64 bf16]
  constexpr uint32_t kIdescSS = make_idesc(256, 128, false, false);
  constexpr uint32_t kIdescAcc = make_idesc(256, D, false, true);
  constexpr uint32_t kIdescDqT = make_idesc(128, 128, true, true);
  // Tensor-memory columns.  R0: S^T (fp32), then P^T (bf16) in [0,32) and [64,96).  R1: dP^T (fp32),
  // then dS^T (bf16) in [128,160) (queries 0-63) and [224,256) (queries 64-127), which leaves
  // [160,224) for dQ^T while dK += dS^T Q still reads dS^T.
  constexpr uint32_t kColR0 = 0, kColR1 = 128, kColDq = 160, kColDv = 256, kColDk = 384;

  const int tid = threadIdx.x, warp = tid >> 5, lane = tid & 31;
  volatile int* abort_flag = &sm.ctl.abort_flag;
  const uint32_t rank = cluster_cta_rank();
  const bool leader = rank == 0;

  const int pair = (blockIdx.x >> 1) % n_kv_pairs;
  const int hk = ((blockIdx.x >> 1) / n_kv_pairs) % p.Hkv;
  const int b = (blockIdx.x >> 1) / (n_kv_pairs * p.Hkv);
  const int j0_pair = pair * 256;
  const int j0 = j0_pair + (int)rank * 128;  // first key row of this CTA
  const int group = p.H / p.Hkv;
  const int shift = p.Sk - p.Sq;
  const int n_q_tiles = (p.Sq + 127) / 128;
  const int q_first = p.causal ? max(0, j0_pair - shift) : 0;
  const int i_first = min(n_q_tiles, q_first / 128);
  const int iters_per_head = n_q_tiles - i_first;
  const int n_iter = iters_per_head * group;
  // neighbouring pairs start at different query tiles so that they do not reduce into the same rows at the same time
  const int q_rot = iters_per_head > 0 ? pair % iters_per_head : 0;

  if (tid == 0) {
    sm.ctl.abort_flag = 0;
    sm.ctl.launch_epoch = (int)p.epoch;
    mbar_init(&sm.kv_full, 1);
    for (int s = 0; s < 2; ++s) {
      mbar_init(&sm.qr_full[s], 1);
      mbar_init(&sm.qr_empty[s], 1);
      mbar_init(&sm.stat_full[s], 1);
    }
    mbar_init(&sm.qc_full, 1);
    mbar_init(&sm.qc_empty, 1);
    mbar_init(&sm.do_full, 1);
    mbar_init(&sm.do_empty, 1);
    mbar_init(&sm.s_full, 1);
    mbar_init(&sm.dp_full, 1);
    mbar_init(&sm.dq_full, 1);
    mbar_init(&sm.acc_full, 1);
    mbar_init(&sm.p_ready, 16);    // 8 compute warps of each CTA
    mbar_init(&sm.ds_ready, 17);   // compute warps of both CTAs + the other CTA's "half has landed" relay
    mbar_init(&sm.ds_in, 1);
    mbar_init(&sm.dq_drained, 8);  // 4 reduction warps of each CTA
    mbar_init(&sm.out_staged, 8);
    fence_barrier_init();
  }
  if (warp == 12) {
    tmem_alloc_pair(&sm.tmem_base, 512);
    tmem_relinquish_pair();
  }
  tc_fence_before();
  __syncthreads();
  cluster_sync_all();  // the other CTA's barriers are initialised before anything signals them
  tc_fence_after();
  const uint32_t tmem = sm.tmem_base;
  // leader-side barriers as seen from this CTA
  const uint32_t bar_p_ready = map_to_cta(smem_u32(&sm.p_ready), 0);
  const uint32_t bar_ds_ready = map_to_cta(smem_u32(&sm.ds_ready), 0);
  const uint32_t bar_dq_drained = map_to_cta(smem_u32(&sm.dq_drained), 0);

  if (warp < 8) {
    // ============================================================ compute warpgroups (thread = key row)
    reg_alloc<192>();
    const int wg = warp >> 2, w = warp & 3;
    const int r = w * 32 + lane;
    const int key = j0 + r;
    const uint32_t lane_base = (uint32_t)(w * 32) << 16;
    const uint32_t s_addr = tmem + kColR0 + lane_base + wg * 64;
    const uint32_t dp_addr = tmem + kColR1 + lane_base + wg * 64;
    // this warpgroup's 64 query columns belong to CTA `wg` of the pair: row (128 rank + r) of its dS^T buffer
    const uint32_t ds_row = map_to_cta(smem_u32(sm.ds) + (rank * 128 + r) * 128, (uint32_t)wg);
    uint8_t* ds_row_local = sm.ds + (rank * 128 + r) * 128;
    const bool ds_is_local = wg == (int)rank;
    const uint32_t bar_ds_in_peer = map_to_cta(smem_u32(&sm.ds_in), rank ^ 1u);
    const float c = p.scale_log2;
    bool ok = true;
    for (int it = 0; it < n_iter; ++it) {
      const int stage = it & 1;
      const int i = i_first + (it % iters_per_head + q_rot) % iters_per_head;
      const int q0 = i * 128 + wg * 64;
      ok = __all_sync(0xffffffffu, mbar_wait(&sm.s_full, it & 1, abort_flag, __LINE__));
      if (!ok) break;
      ok = __all_sync(0xffffffffu, mbar_wait(&sm.stat_full[stage], (it >> 1) & 1, abort_flag, __LINE__));
      if (!ok) break;
      tc_fence_after();
      uint32_t s[2][32];
      tmem_ld32(s_addr, s[0]);
      tmem_ld32(s_addr + 32, s[1]);
      tmem_wait_ld();
      const bool masked = p.causal && (j0 + 127 > i * 128 + shift);
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
        for (int e = 0; e < 16; ++e) pk[e] = pack_bf16x2(pr[h2][2 * e], pr[h2][2 * e + 1]);
        tmem_st16(s_addr + h2 * 16, pk);
      }
      tmem_wait_st();
      tc_fence_before();
      __syncwarp();
      if (lane == 0) mbar_arrive_cluster(bar_p_ready);

      ok = __all_sync(0xffffffffu, mbar_wait(&sm.dp_full, it & 1, abort_flag, __LINE__));
      if (!ok) break;
      tc_fence_after();
      uint32_t dp[2][32];
      tmem_ld32(dp_addr, dp[0]);
      tmem_ld32(dp_addr + 32, dp[1]);
      tmem_wait_ld();
      const float4* dl4 =reinterpret_cast<const float4*>(&sm.delta[stage][wg * 64]);
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
          pk[g * 2] = pack_bf16x2(d0, d1);
          pk[g * 2 + 1] = pack_bf16x2(d2, d3);
        }
        tmem_st16(dp_addr + wg * 32 + h2 * 16, pk);
#pragma unroll
        for (int ch = 0; ch < 4; ++ch) {
          const int chunk = h2 * 4 + ch;
          const uint4 v4 = make_uint4(pk[ch * 4], pk[ch * 4 + 1], pk[ch * 4 + 2], pk[ch * 4 + 3]);
          const uint32_t off = (uint32_t)((chunk ^ (r & 7)) << 4);
          // the other CTA's columns travel as asynchronous stores counted on its ds_in barrier
          if (ds_is_local) *reinterpret_cast<uint4*>(ds_row_local + off) = v4;
          else st_async_v4(ds_row + off, v4, bar_ds_in_peer);
        }
      }
      tmem_wait_st();
      tc_fence_before();
      if (ds_is_local) fence_proxy_async_smem();
      __syncwarp();
      if (lane == 0) mbar_arrive_cluster(bar_ds_ready);
    }

    // ---- epilogue: dV and dK * scale of this CTA's key rows -> bf16 -> shared memory (swizzled) -> TMA store
    if (ok) {
      if (n_iter > 0) {
        ok = __all_sync(0xffffffffu, mbar_wait(&sm.acc_full, 0, abort_flag, __LINE__));
        tc_fence_after();
      }
      if (ok) {
#pragma unroll
        for (int which = 0; which < 2; ++which) {
          const uint32_t acc_addr = tmem + (which == 0 ? kColDv : kColDk) + lane_base + wg * 64;
          uint8_t* stage_buf = which == 0 ? sm.do_rows : sm.q_rows[0];  // 32 KiB each with the buffer that follows
          const float mul = which == 0 ? 1.0f : p.scale;
#pragma unroll
          for (int cc = 0; cc < 2; ++cc) {
            uint32_t v[32];
            if (n_iter > 0) {
              tmem_ld32(acc_addr + cc * 32, v);
              tmem_wait_ld();
            } else {
#pragma unroll
              for (int e = 0; e < 32; ++e) v[e] = 0u;
            }
            uint8_t* row_ptr = stage_buf + wg * kRegionBytes + r * 128;
#pragma unroll
            for (int ch = 0; ch < 4; ++ch) {
              uint4 w4;
              w4.x = pack_bf16x2(__uint_as_float(v[8 * ch + 0]) * mul, __uint_as_float(v[8 * ch + 1]) * mul);
              w4.y = pack_bf16x2(__uint_as_float(v[8 * ch + 2]) * mul, __uint_as_float(v[8 * ch + 3]) * mul);
              w4.z = pack_bf16x2(__uint_as_float(v[8 * ch + 4]) * mul, __uint_as_float(v[8 * ch + 5]) * mul);
              w4.w = pack_bf16x2(__uint_as_float(v[8 * ch + 6]) * mul, __uint_as_float(v[8 * ch + 7]) * mul);
              const int chunk = cc * 4 + ch;
              *reinterpret_cast<uint4*>(row_ptr + ((chunk ^ (r & 7)) << 4)) = w4;
            }
          }
        }
        fence_proxy_async_smem();
        __syncwarp();
        if (lane == 0) mbar_arrive(&sm.out_staged);
        if (warp == 0) {
          ok = __all_sync(0xffffffffu, mbar_wait(&sm.out_staged, 0, abort_flag, __LINE__));
          if (ok && lane == 0 && j0 < p.Sk) {
            for (int rg = 0; rg < 2; ++rg) {
              tma_store_4d(&tm_dv, sm.do_rows + rg * kRegionBytes, rg * 64, hk, j0, b);
              tma_store_4d(&tm_dk, sm.q_rows[0] + rg * kRegionBytes, rg * 64, hk, j0, b);
            }
            tma_commit_group();
            tma_wait_group_read<0>();
          }
        }
      }
    }
  } else if (warp < 12) {
    // ============================================================ dQ reduction warps
    // dQ^T of the pair product has 64 head-dim rows per CTA, laid out in tensor memory as lanes
    // 0-63 = queries 0-63 and lanes 64-127 = queries 64-127 (64 columns each).  Warp w therefore
    // owns head dims [64 rank + 32 (w & 1), +32) of queries [64 (w >> 1), +64): two 4 KiB chunks.
    reg_dealloc<80>();
    const int w = warp & 3;
    const uint32_t addr = tmem + kColDq + ((uint32_t)(w * 32) << 16);
    const int d_chunk = 2 * (int)rank + (w & 1);
    float* slot = sm.red_slot[w];
    bool ok = true;
    for (int it = 0; it < n_iter && ok; ++it) {
      const int h = hk * group + it / iters_per_head;
      const int i = i_first + (it % iters_per_head + q_rot) % iters_per_head;
      ok = __all_sync(0xffffffffu, mbar_wait(&sm.dq_full, it & 1, abort_flag, __LINE__));
      if (!ok) break;
      tc_fence_after();
      uint32_t v[2][32];
      tmem_ld32(addr, v[0]);
      tmem_ld32(addr + 32, v[1]);
      tmem_wait_ld();
      // everything is in registers: the next dP^T may overwrite the region
      tc_fence_before();
      __syncwarp();
      if (lane == 0) mbar_arrive_cluster(bar_dq_drained);
      float* dst = p.dq_acc +
                   ((((size_t)b * p.H + h) * (p.Sq_pad / 32) + (size_t)i * 4 + 2 * (w >> 1)) * 4 + d_chunk) * 1024;
#pragma unroll
      for (int cc = 0; cc < 2; ++cc) {
        // the previous bulk reduce has to be done reading the slot
        if (lane == 0) tma_wait_group_read<0>();
        __syncwarp();
#pragma unroll
        for (int e = 0; e < 32; ++e) slot[e * 32 + lane] = __uint_as_float(v[cc][e]);
        fence_proxy_async_smem();
        __syncwarp();
        if (lane == 0) {
          asm volatile("cp.reduce.async.bulk.global.shared::cta.bulk_group.add.f32 [%0], [%1], %2;" ::"l"(
                           dst + (size_t)cc * 4096),
                       "r"(smem_u32(slot)), "r"(4096)
                       : "memory");
          tma_commit_group();
        }
      }
    }
    if (lane == 0) tma_wait_group<0>();  // all reductions have landed before the CTA exits
    __syncwarp();
  } else if (warp == 12) {
    // ============================================================ MMA issuer (leader CTA only; warp-uniform, one lane issues)
    reg_dealloc<48>();
    if (leader && n_iter > 0) {
      const uint32_t k_lo = desc_lo(smem_u32(sm.k), 16), v_lo = desc_lo(smem_u32(sm.v), 16);
      const uint32_t kdq_lo = desc_lo(smem_u32(sm.k_dq), kRegionBytes);
      const uint32_t qr_lo0 = desc_lo(smem_u32(sm.q_rows[0]), 16), dor_lo = desc_lo(smem_u32(sm.do_rows), 16);
      const uint32_t qc_lo = desc_lo(smem_u32(sm.q_cols), kRegionBytes);
      const uint32_t doc_lo = desc_lo(smem_u32(sm.do_cols), kRegionBytes);
      const uint32_t ds_lo = desc_lo(smem_u32(sm.ds), kRegionBytes);
      constexpr uint32_t kQrStageStep = Smem::kHalfBytes >> 4;
      auto wait_bar = [&](uint64_t* bar, uint32_t parity, int site) {
        return __all_sync(0xffffffffu, mbar_wait_cluster(bar, parity, abort_flag, site));
      };
      // D[256 x 128] = A[256 x 128] B^T, both K-major: A = own [128][128] tile, B = [64][128] rows tile
      auto ss_kmajor = [&](uint32_t d_col, uint32_t a_lo, uint32_t b_lo) {
        if (elect_one()) {
#pragma unroll
          for (int kk = 0; kk < D / 16; ++kk) {
            const uint32_t a_off = ((kk / 4) * kRegionBytes + (kk % 4) * 32) >> 4;
            const uint32_t b_off = ((kk / 4) * kHalfRegionBytes + (kk % 4) * 32) >> 4;
            mma_pair_ss_lohi(tmem + d_col, a_lo + a_off, b_lo + b_off, kDescHiSw128, kIdescSS, kk > 0);
          }
        }
        __syncwarp();
      };
      // D[256 x 128] (+)= A[tmem, 256 x 128 queries] B[128 queries x 128], B = [128][64] columns tile
      // (`a_half` = column distance between the bf16 blocks of queries 0-63 and 64-127)
      auto ts_acc = [&](uint32_t d_col, uint32_t a_col, uint32_t a_half, uint32_t b_mn_lo, uint32_t accumulate) {
        if (elect_one()) {
#pragma unroll
          for (int kk = 0; kk < 8; ++kk)
            mma_pair_ts_lohi(tmem + d_col, tmem + a_col + (kk / 4) * a_half + (kk % 4) * 8, b_mn_lo + ((kk * 2048) >> 4),
                             kDescHiSw128, kIdescAcc, kk > 0 ? 1u : accumulate);
        }
        __syncwarp();
      };
      auto commit = [&](uint64_t* bar) {
        if (elect_one()) mma_pair_commit(bar);
        __syncwarp();
      };
      do {
        if (!wait_bar(&sm.kv_full, 0, __LINE__)) break;
        if (!wait_bar(&sm.qr_full[0], 0, __LINE__)) break;
        ss_kmajor(kColR0, k_lo, qr_lo0);  // S^T(0)
        commit(&sm.s_full);
        commit(&sm.qr_empty[0]);
        if (elect_one()) mbar_expect_tx(&sm.ds_in, Smem::kHalfBytes);
        __syncwarp();
        bool ok = true;
        for (int it = 0; it < n_iter; ++it) {
          const int stage = it & 1;
          if (!(ok = wait_bar(&sm.do_full, it & 1, __LINE__))) break;
          if (it > 0 && !(ok = wait_bar(&sm.dq_drained, (it - 1) & 1, __LINE__))) break;
          tc_fence_after();
          ss_kmajor(kColR1, v_lo, dor_lo);  // dP^T(it)
          commit(&sm.dp_full);
          if (!(ok = wait_bar(&sm.p_ready, it & 1, __LINE__))) break;
          tc_fence_after();
          ts_acc(kColDv, kColR0, 64, doc_lo, it > 0 ? 1u : 0u);  // dV += P^T dO
          commit(&sm.do_empty);
          if (it + 1 < n_iter) {
            if (!(ok = wait_bar(&sm.qr_full[stage ^ 1], ((it + 1) >> 1) & 1, __LINE__))) break;
            ss_kmajor(kColR0, k_lo, qr_lo0 + (stage ^ 1) * kQrStageStep);  // S^T(it + 1)
            commit(&sm.s_full);
            commit(&sm.qr_empty[stage ^ 1]);
          }
          if (!(ok = wait_bar(&sm.ds_ready, it & 1, __LINE__))) break;
          if (!(ok = wait_bar(&sm.ds_in, it & 1, __LINE__))) break;
          tc_fence_after();
          // dQ^T first: its drain and the hand-back of the region then overlap with the dK product
          if (elect_one()) {
            if (it + 1 < n_iter) mbar_expect_tx(&sm.ds_in, Smem::kHalfBytes);
#pragma unroll
            for (int kk = 0; kk < 16; ++kk)  // dQ^T = K^T dS^T over the pair's 256 keys
              mma_pair_ss_lohi(tmem + kColDq, kdq_lo + ((kk * 2048) >> 4), ds_lo + ((kk * 2048) >> 4), kDescHiSw128,
                               kIdescDqT, kk > 0);
          }
          __syncwarp();
          commit(&sm.dq_full);
          if (!(ok = wait_bar(&sm.qc_full, it & 1, __LINE__))) break;
          ts_acc(kColDk, kColR1, 96, qc_lo, it > 0 ? 1u : 0u);  // dK += dS^T Q
          commit(&sm.qc_empty);
        }
        if (ok) commit(&sm.acc_full);
      } while (false);
    } else if (n_iter > 0 && lane == 0) {
      // other CTA: tell the leader when this CTA's copy of dS^T has received the leader's half
      for (int it = 0; it < n_iter; ++it) {
        mbar_expect_tx(&sm.ds_in, Smem::kHalfBytes);
        if (!mbar_wait(&sm.ds_in, it & 1, abort_flag, __LINE__)) break;
        mbar_arrive_cluster(bar_ds_ready);
      }
    }
    __syncwarp();
  } else if (warp == 13) {
    // ============================================================ TMA producer (both CTAs, each into its own memory)
    reg_dealloc<48>();
    if (n_iter > 0 && lane == 0) {
      const int d_half = (int)rank * 64;   // this CTA's head-dim columns
      const int row_half = (int)rank * 64;  // this CTA's rows of a query tile
      const uint32_t bar_kv = map_to_cta(smem_u32(&sm.kv_full), 0);
      const uint32_t bar_qr[2] = {map_to_cta(smem_u32(&sm.qr_full[0]), 0), map_to_cta(smem_u32(&sm.qr_full[1]), 0)};
      const uint32_t bar_qc = map_to_cta(smem_u32(&sm.qc_full), 0);
      const uint32_t bar_do = map_to_cta(smem_u32(&sm.do_full), 0);
      auto tile_of = [&](int it, int& h, int& i) {
        h = hk * group + it / iters_per_head;
        i = i_first + (it % iters_per_head + q_rot) % iters_per_head;
      };
      auto load_q_rows_and_stats = [&](int it) {
        int h, i;
        tile_of(it, h, i);
        const int stage = it & 1;
        if (leader) mbar_expect_tx(&sm.qr_full[stage], 2 * Smem::kHalfBytes);
        for (int rg = 0; rg < 2; ++rg)
          tma_load_4d_pair(sm.q_rows[stage] + rg * kHalfRegionBytes, &tm_q64, bar_qr[stage], rg * 64, h,
                           i * 128 + row_half, b);
        const size_t row_off = ((size_t)b * p.H + h) * p.Sq_pad + (size_t)i * 128;
        mbar_expect_tx(&sm.stat_full[stage], 1024);
        bulk_load_1d(sm.lse2[stage], p.lse2 + row_off, 512, &sm.stat_full[stage]);
        bulk_load_1d(sm.delta[stage], p.delta + row_off, 512, &sm.stat_full[stage]);
      };
      if (leader) mbar_expect_tx(&sm.kv_full, 2 * 3 * Smem::kTileBytes);
      for (int rg = 0; rg < 2; ++rg) {
        tma_load_4d_pair(sm.k + rg * kRegionBytes, &tm_k, bar_kv, rg * 64, hk, j0, b);
        tma_load_4d_pair(sm.v + rg * kRegionBytes, &tm_v, bar_kv, rg * 64, hk, j0, b);
        tma_load_4d_pair(sm.k_dq + rg * kRegionBytes, &tm_k, bar_kv, d_half, hk, j0_pair + rg * 128, b);
      }
      load_q_rows_and_stats(0);
      for (int it = 0; it < n_iter; ++it) {
        int h, i;
        tile_of(it, h, i);
        if (it >= 1 && !mbar_wait(&sm.do_empty, (it - 1) & 1, abort_flag, __LINE__)) break;
        if (leader) mbar_expect_tx(&sm.do_full, 2 * Smem::kTileBytes);
        for (int rg = 0; rg < 2; ++rg)
          tma_load_4d_pair(sm.do_rows + rg * kHalfRegionBytes, &tm_do64, bar_do, rg * 64, h, i * 128 + row_half, b);
        tma_load_4d_pair(sm.do_cols, &tm_do, bar_do, d_half, h, i * 128, b);
        if (it >= 1 && !mbar_wait(&sm.qc_empty, (it - 1) & 1, abort_flag, __LINE__)) break;
        if (leader) mbar_expect_tx(&sm.qc_full, 2 * Smem::kHalfBytes);
        tma_load_4d_pair(sm.q_cols, &tm_q, bar_qc, d_half, h, i * 128, b);
        if (it + 1 < n_iter) {
          const int s1 = (it + 1) & 1;
          if (it + 1 >= 2 && !mbar_wait(&sm.qr_empty[s1], (((it + 1) >> 1) - 1) & 1, abort_flag, __LINE__)) break;
          load_q_rows_and_stats(it + 1);
        }
      }
    }
    __syncwarp();
  } else {
    reg_dealloc<48>();
  }

  tc_fence_before();
  __syncthreads();
  cluster_sync_all();  // neither CTA leaves (or frees tensor memory) while the other may still touch it
  if (warp == 12) tmem_dealloc_pair(tmem, 512);
}

}  // namespace fa

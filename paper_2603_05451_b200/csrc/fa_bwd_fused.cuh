// Backward main kernel, single-kernel ("fused") form of the paper's Section 3.2 for head
// dimensions 128 and 64: five MMAs per (key tile, query tile) pair with P and dS resident in
// tensor memory, dQ reduced into an FP32 global accumulator.
//
// Differences from the generic kernel in fa_bwd_kernels.cuh:
//   * The dQ tile is drained by four warps that work independently.  A warp copies a chunk of 32
//     queries x 32 head dims (4 KiB of floats) into its private shared-memory slot with
//     conflict-free stores and hands it to the TMA unit as ONE bulk reduce-add.  The accumulator
//     layout [B][H][Sq_pad/32][D/32][32][32] makes that chunk contiguous in global memory, so the
//     L2 receives whole 128-byte lines (the pattern it reduces fastest) and the SM's load/store
//     pipe is not clogged by reduction instructions.  Slots are double-buffered per warp.
//     D = 128: the product is formed transposed, dQ^T = K^T dS^T (head dim on the tensor-memory
//     lanes, over the dP^T / dS^T region), a warp owns 32 head dims of all 128 queries and a chunk
//     is stored [query][head dim].  D = 64: dQ = dS K with the queries on the lanes, in a region
//     of its own (tensor memory has room), a warp owns 32 queries and a chunk is stored
//     [head dim][query].
//   * dO_i is single-buffered (it is free again once dV += P^T dO_i has been issued), which pays
//     for the 32 KiB of reduction slots; Delta_i travels with Q_i.
#pragma once

#include "fa_bwd_kernels.cuh"

namespace fa {

template <int D>
struct BwdFusedSmem {
  static constexpr int kTileBytes = 128 * D * 2;
  static constexpr int kDsBytes = 128 * 128 * 2;
  alignas(1024) uint8_t k[kTileBytes];
  alignas(1024) uint8_t v[kTileBytes];
  alignas(1024) uint8_t q[2][kTileBytes];  // Q_i stages; q[0] stages dK in the epilogue
  alignas(1024) uint8_t d_o[kTileBytes];   // dO_i (single stage); stages dV in the epilogue
  alignas(1024) uint8_t ds[kDsBytes];      // dS^T tile, [key row][query], 128-byte swizzle
  alignas(1024) float red_slot[4][2][32 * 32];  // [warp][buffer][query][head dim]: one 4 KiB bulk reduce each
  alignas(16) float lse2[2][128];
  alignas(16) float delta[2][128];
  alignas(8) uint64_t kv_full;
  uint64_t q_full[2], q_empty[2], do_full, do_empty;
  uint64_t s_full, p_ready, dp_full, dst_ready, ds_ready, dq_full, dq_drained, acc_full, out_staged;
  uint32_t tmem_base;
  WaitCtl ctl;  // abort flag and launch epoch, read by every bounded wait
};

// dQ accumulator element (b, h, q, d) in the chunked layout the bulk reductions use: chunks of 32
// queries x 32 head dims; inside a chunk [query][head dim] for D = 128, [head dim][query] for D = 64.
template <int D>
__host__ __device__ inline size_t dq_acc_chunked_index(int b, int h, int q, int d, int H, int Sq_pad) {
  const size_t chunk = (((size_t)b * H + h) * (Sq_pad / 32) + q / 32) * (D / 32) + d / 32;
  return chunk * 1024 + (D == 128 ? (size_t)(q % 32) * 32 + d % 32 : (size_t)(d % 32) * 32 + q % 32);
}

template <int D, bool kF16>
__global__ void __launch_bounds__(256)
bwd_convert_dq_chunked_kernel(const float* __restrict__ dq_acc, __nv_bfloat16* __restrict__ dq, size_t n8, float scale,
                              int H, int Sq, int Sq_pad) {
  // idx runs over groups of 8 elements of dq [B, Sq, H, D]
  const size_t idx = (size_t)blockIdx.x * blockDim.x + threadIdx.x;
  if (idx >= n8) return;
  constexpr int kSubs = D / 8;
  const int sub = (int)(idx % kSubs);
  const int h = (int)((idx / kSubs) % H);
  const int q = (int)((idx / ((size_t)kSubs * H)) % Sq);
  const int bb = (int)(idx / ((size_t)kSubs * H * Sq));
  float x[8];
  if (D == 128) {
    const float4* src = reinterpret_cast<const float4*>(dq_acc + dq_acc_chunked_index<D>(bb, h, q, sub * 8, H, Sq_pad));
    const float4 a = src[0], b = src[1];
    x[0] = a.x; x[1] = a.y; x[2] = a.z; x[3] = a.w; x[4] = b.x; x[5] = b.y; x[6] = b.z; x[7] = b.w;
  } else {
    const float* src = dq_acc + dq_acc_chunked_index<D>(bb, h, q, sub * 8, H, Sq_pad);
#pragma unroll
    for (int e = 0; e < 8; ++e) x[e] = src[e * 32];  // consecutive head dims are 32 floats apart
  }
  uint4 w;
  w.x = pack2<kF16>(x[0] * scale, x[1] * scale);
  w.y = pack2<kF16>(x[2] * scale, x[3] * scale);
  w.z = pack2<kF16>(x[4] * scale, x[5] * scale);
  w.w = pack2<kF16>(x[6] * scale, x[7] * scale);
  reinterpret_cast<uint4*>(dq)[idx] = w;
}

template <int D, bool kF16>  // kF16: inputs and outputs FP16 instead of BF16
__global__ void __launch_bounds__(512, 1)
bwd_fused_kernel(const __grid_constant__ CUtensorMap tm_q, const __grid_constant__ CUtensorMap tm_k,
                 const __grid_constant__ CUtensorMap tm_v, const __grid_constant__ CUtensorMap tm_do,
                 const __grid_constant__ CUtensorMap tm_dk, const __grid_constant__ CUtensorMap tm_dv,
                 const BwdParams p, const int n_kv_tiles) {
  extern __shared__ __align__(1024) uint8_t smem_raw[];
  using Smem = BwdFusedSmem<D>;
  Smem& sm = *reinterpret_cast<Smem*>(smem_raw);
  if ((smem_u32(smem_raw) & 1023u) != 0) {
    if (threadIdx.x == 0) record_device_status(5, __LINE__, p.epoch);
    return;
  }
  constexpr int kRegions = D / 64;
  constexpr int kRegionBytes = 128 * 128;
  constexpr uint32_t kIdescSS = make_idesc(128, 128, false, false, kF16);
  constexpr uint32_t kIdescAcc = make_idesc(128, D, false, true, kF16);
  // D = 128: dQ^T = K^T dS^T (128 head dims x 128 queries); D = 64: dQ = dS K (128 queries x 64 head dims)
  constexpr uint32_t kIdescDq = make_idesc(128, D == 128 ? 128 : 64, true, true, kF16);
  constexpr uint32_t kColR0 = 0, kColR1 = 128, kColDv = 256, kColDk = 256 + D;
  constexpr uint32_t kColDq = D == 128 ? kColR1 : 256 + 2 * D;  // D = 64: a region of its own

  const int tid = threadIdx.x, warp = tid >> 5, lane = tid & 31;
  volatile int* abort_flag = &sm.ctl.abort_flag;

  // Launch order.  Without a mask every key tile costs the same and the tiles of one (batch, head) follow each
  // other, so that the CTAs in flight stream the same Q and dO.  With the causal mask the first key tile of a
  // sequence meets every query tile and the last one a single one; a head's long tiles that start late would
  // leave the other SMs idle at the end.  The launch code then asks for sections of a few heads: inside a section
  // the key-tile index is the slow coordinate, so the section's longest tiles start first and its shortest fill the
  // tail (longest-processing-time-first, Section 3.3), while the tiles of a head still run close enough together
  // to share their Q and dO reads in L2.
  int n_tile, hk, b;
  if (p.heads_per_section > 0) {
    const int heads = p.Hkv * p.B, per_section = p.heads_per_section * n_kv_tiles;
    const int sec = blockIdx.x / per_section, r = blockIdx.x % per_section;
    const int g = min(p.heads_per_section, heads - sec * p.heads_per_section);  // the last section may be smaller
    n_tile = r / g;
    const int hb = sec * p.heads_per_section + r % g;
    hk = hb % p.Hkv;
    b = hb / p.Hkv;
  } else {
    n_tile = blockIdx.x % n_kv_tiles;
    hk = (blockIdx.x / n_kv_tiles) % p.Hkv;
    b = blockIdx.x / (n_kv_tiles * p.Hkv);
  }
  const int j0 = n_tile * 128;
  const int group = p.H / p.Hkv;
  // Dense batch: sequence b of length Sq / Sk at batch coordinate b.  Packed batch: this sequence's
  // lengths and its offsets on the token axis (batch coordinate 0) and in the workspace arrays.
  int Sq = p.Sq, Sk = p.Sk, q_row0 = 0, k_row0 = 0, tma_b = b;
  size_t acc_row0 = (size_t)b * p.H * p.Sq_pad;  // first workspace row of (this sequence, head 0)
  size_t acc_head_stride = p.Sq_pad;             // workspace rows between consecutive heads
  const bool packed = p.cu_q != nullptr;
  if (packed) {
    q_row0 = p.cu_q[b];
    k_row0 = p.cu_k[b];
    Sq = p.cu_q[b + 1] - q_row0;
    Sk = p.cu_k[b + 1] - k_row0;
    if (j0 >= Sk) return;  // this key tile does not exist in this sequence
    tma_b = 0;
    acc_row0 = p.pad_off[b];
    acc_head_stride = p.total_pad;
  }
  const bool kv_tail = packed && j0 + 128 > Sk;  // rows past the end hold the next sequence's keys: mask them
  const int shift = Sk - Sq;
  const int n_q_tiles = (Sq + 127) / 128;
  const int q_first = p.causal ? max(0, j0 - shift) : 0;
  const int i_first = min(n_q_tiles, q_first / 128);
  const int iters_per_head = n_q_tiles - i_first;
  const int n_iter = iters_per_head * group;
  // neighbouring CTAs start at different query tiles so that they do not reduce into the same rows at the same time
  const int q_rot = iters_per_head > 0 ? n_tile % iters_per_head : 0;

  if (tid == 0) {
    sm.ctl.abort_flag = 0;
    sm.ctl.launch_epoch = (int)p.epoch;
    mbar_init(&sm.kv_full, 1);
    for (int s = 0; s < 2; ++s) {
      mbar_init(&sm.q_full[s], 1);
      mbar_init(&sm.q_empty[s], 1);
    }
    mbar_init(&sm.do_full, 1);
    mbar_init(&sm.do_empty, 1);
    mbar_init(&sm.s_full, 1);
    mbar_init(&sm.p_ready, 8);
    mbar_init(&sm.dp_full, 1);
    mbar_init(&sm.dst_ready, 8);  // dS^T in tensor memory (for dK)
    mbar_init(&sm.ds_ready, 8);   // dS^T in shared memory (for dQ^T)
    mbar_init(&sm.dq_full, 1);
    mbar_init(&sm.dq_drained, 4);
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
    // ============================================================ compute warpgroups (thread = key row)
    reg_alloc<192>();
    const int wg = warp >> 2, w = warp & 3;
    const int r = w * 32 + lane;
    const int key = j0 + r;
    const uint32_t lane_base = (uint32_t)(w * 32) << 16;
    const uint32_t s_addr = tmem + kColR0 + lane_base + wg * 64;
    const uint32_t dp_addr = tmem + kColR1 + lane_base + wg * 64;
    uint8_t* ds_row = sm.ds + wg * kRegionBytes + r * 128;
    const float c = p.scale_log2;
    bool ok = true;
    for (int it = 0; it < n_iter; ++it) {
      const int stage = it & 1;
      const int i = i_first + (it % iters_per_head + q_rot) % iters_per_head;
      const int q0 = i * 128 + wg * 64;
      ok = __all_sync(0xffffffffu, mbar_wait(&sm.s_full, it & 1, abort_flag));
      if (!ok) break;
      tc_fence_after();
      uint32_t s[2][32];
      tmem_ld32(s_addr, s[0]);
      tmem_ld32(s_addr + 32, s[1]);
      tmem_wait_ld();
      const bool masked = p.causal && (j0 + 127 > i * 128 + shift);
      // Tiles on the diagonal and the last key tile of a packed sequence: masked scores become -inf here, so that
      // the loop below carries no per-element test for all the other tiles.
      if (masked) {
        const int first_visible = key - q0 - shift;  // columns below it are queries that do not see this key
#pragma unroll
        for (int h2 = 0; h2 < 2; ++h2) {
#pragma unroll
          for (int col = 0; col < 32; ++col)
            if (h2 * 32 + col < first_visible) s[h2][col] = 0xff800000u;
        }
      }
      if (kv_tail && key >= Sk) {
#pragma unroll
        for (int h2 = 0; h2 < 2; ++h2) {
#pragma unroll
          for (int col = 0; col < 32; ++col) s[h2][col] = 0xff800000u;
        }
      }
      float pr[2][32];
      const float4* lse4 = reinterpret_cast<const float4*>(&sm.lse2[stage][wg * 64]);
#pragma unroll
      for (int h2 = 0; h2 < 2; ++h2) {
#pragma unroll
        for (int g = 0; g < 8; ++g) {
          const float4 l4 = lse4[h2 * 8 + g];
          // two scores per instruction on the packed FP32 pipe
          const float2 x01 = __ffma2_rn(make_float2(__uint_as_float(s[h2][g * 4 + 0]), __uint_as_float(s[h2][g * 4 + 1])),
                                        make_float2(c, c), make_float2(-l4.x, -l4.y));
          const float2 x23 = __ffma2_rn(make_float2(__uint_as_float(s[h2][g * 4 + 2]), __uint_as_float(s[h2][g * 4 + 3])),
                                        make_float2(c, c), make_float2(-l4.z, -l4.w));
          const float xs[4] = {x01.x, x01.y, x23.x, x23.y};
#pragma unroll
          for (int e = 0; e < 4; ++e) {
            const int col = g * 4 + e;
            pr[h2][col] = ex2_approx(xs[e]);
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
      uint32_t pk[2][16];
#pragma unroll
      for (int h2 = 0; h2 < 2; ++h2) {
#pragma unroll
        for (int g = 0; g < 8; ++g) {
          const float4 d4 = dl4[h2 * 8 + g];
          const float2 t01 = __fadd2_rn(make_float2(__uint_as_float(dp[h2][g * 4 + 0]), __uint_as_float(dp[h2][g * 4 + 1])),
                                        make_float2(-d4.x, -d4.y));
          const float2 t23 = __fadd2_rn(make_float2(__uint_as_float(dp[h2][g * 4 + 2]), __uint_as_float(dp[h2][g * 4 + 3])),
                                        make_float2(-d4.z, -d4.w));
          const float2 d01 = __fmul2_rn(make_float2(pr[h2][g * 4 + 0], pr[h2][g * 4 + 1]), t01);
          const float2 d23 = __fmul2_rn(make_float2(pr[h2][g * 4 + 2], pr[h2][g * 4 + 3]), t23);
          pk[h2][g * 2] = pack2<kF16>(d01.x, d01.y);
          pk[h2][g * 2 + 1] = pack2<kF16>(d23.x, d23.y);
        }
        tmem_st16(dp_addr + h2 * 16, pk[h2]);
      }
      // dS^T is in tensor memory: dK += dS^T Q can start while the shared-memory copy (for dQ) is written
      tmem_wait_st();
      tc_fence_before();
      __syncwarp();
      if (lane == 0) mbar_arrive(&sm.dst_ready);
#pragma unroll
      for (int chunk = 0; chunk < 8; ++chunk) {
        const int h2 = chunk >> 2, ch = chunk & 3;
        *reinterpret_cast<uint4*>(ds_row + ((chunk ^ (r & 7)) << 4)) =
            make_uint4(pk[h2][ch * 4], pk[h2][ch * 4 + 1], pk[h2][ch * 4 + 2], pk[h2][ch * 4 + 3]);
      }
      fence_proxy_async_smem();
      __syncwarp();
      if (lane == 0) mbar_arrive(&sm.ds_ready);
    }

    // ---- epilogue: dV and dK * scale -> bf16 -> shared memory (swizzled) -> TMA store
    if (ok) {
      if (n_iter > 0) {
        ok = __all_sync(0xffffffffu, mbar_wait(&sm.acc_full, 0, abort_flag));
        tc_fence_after();
      }
      if (ok) {
#pragma unroll
        for (int which = 0; which < 2; ++which) {
          const uint32_t acc_addr = tmem + (which == 0 ? kColDv : kColDk) + lane_base + wg * (D / 2);
          uint8_t* stage_buf = which == 0 ? sm.d_o : sm.q[0];
          const float mul = which == 0 ? 1.0f : p.scale;
#pragma unroll
          for (int cc = 0; cc < D / 64; ++cc) {
            uint32_t v[32];
            if (n_iter > 0) {
              tmem_ld32(acc_addr + cc * 32, v);
              tmem_wait_ld();
            } else {
#pragma unroll
              for (int e = 0; e < 32; ++e) v[e] = 0u;
            }
            // this warpgroup's half of the head dims: a 64-column region of its own (D = 128) or half a region (D = 64)
            uint8_t* row_ptr = stage_buf + (D == 128 ? wg * kRegionBytes : 0) + r * 128;
#pragma unroll
            for (int ch = 0; ch < 4; ++ch) {
              uint4 w4;
              w4.x = pack2<kF16>(__uint_as_float(v[8 * ch + 0]) * mul, __uint_as_float(v[8 * ch + 1]) * mul);
              w4.y = pack2<kF16>(__uint_as_float(v[8 * ch + 2]) * mul, __uint_as_float(v[8 * ch + 3]) * mul);
              w4.z = pack2<kF16>(__uint_as_float(v[8 * ch + 4]) * mul, __uint_as_float(v[8 * ch + 5]) * mul);
              w4.w = pack2<kF16>(__uint_as_float(v[8 * ch + 6]) * mul, __uint_as_float(v[8 * ch + 7]) * mul);
              const int chunk = D == 128 ? cc * 4 + ch : wg * 4 + ch;  // 16-byte chunk inside the 128-byte row
              if (kv_tail) {
                // the rows after this sequence's last key belong to the next sequence: no 128-row TMA store,
                // every valid row is written on its own
                __nv_bfloat16* out = (which == 0 ? p.dv : p.dk) +
                                     ((size_t)(k_row0 + min(key, Sk - 1)) * p.Hkv + hk) * D + (D == 128 ? wg * 64 : 0) + chunk * 8;
                if (key < Sk) *reinterpret_cast<uint4*>(out) = w4;
              } else {
                *reinterpret_cast<uint4*>(row_ptr + ((chunk ^ (r & 7)) << 4)) = w4;
              }
            }
          }
        }
        fence_proxy_async_smem();
        __syncwarp();
        if (lane == 0) mbar_arrive(&sm.out_staged);
        if (warp == 0) {
          ok = __all_sync(0xffffffffu, mbar_wait(&sm.out_staged, 0, abort_flag));
          if (ok && lane == 0 && !kv_tail) {
            for (int rg = 0; rg < kRegions; ++rg) {
              tma_store_4d(&tm_dv, sm.d_o + rg * kRegionBytes, rg * 64, hk, k_row0 + j0, tma_b);
              tma_store_4d(&tm_dk, sm.q[0] + rg * kRegionBytes, rg * 64, hk, k_row0 + j0, tma_b);
            }
            tma_commit_group();
            tma_wait_group_read<0>();
          }
        }
      }
    }
  } else if (warp < 12) {
    // ============================================================ dQ reduction warps (independent of one another)
    reg_dealloc<80>();
    const int w = warp & 3;
    // this thread: head-dim row 32w + lane of dQ^T (D = 128), query 32w + lane of dQ (D = 64)
    const uint32_t addr = tmem + kColDq + ((uint32_t)(w * 32) << 16);
    bool ok = true;
    for (int it = 0; it < n_iter && ok; ++it) {
      const int h = hk * group + it / iters_per_head;
      const int i = i_first + (it % iters_per_head + q_rot) % iters_per_head;
      ok = __all_sync(0xffffffffu, mbar_wait(&sm.dq_full, it & 1, abort_flag));
      if (!ok) break;
      tc_fence_after();
      // first 32-query chunk of the tile in the accumulator (chunks of 4 KiB, D / 32 per 32 queries)
      float* tile_dst = p.dq_acc + ((acc_row0 + (size_t)h * acc_head_stride) / 32 + (size_t)i * 4) * (D / 32) * 1024;
      // two chunks (both slots) per round
#pragma unroll
      for (int half = 0; half < D / 64; ++half) {
        uint32_t v[2][32];
        tmem_ld32(addr + half * 64, v[0]);
        tmem_ld32(addr + half * 64 + 32, v[1]);
        tmem_wait_ld();
        if (half == D / 64 - 1) {
          // everything is in registers: the region may be overwritten
          tc_fence_before();
          __syncwarp();
          if (lane == 0) mbar_arrive(&sm.dq_drained);
        }
        // the bulk reduces of the previous round have to be done reading the slots
        if (lane == 0) tma_wait_group_read<0>();
        __syncwarp();
#pragma unroll
        for (int s2 = 0; s2 < 2; ++s2) {
          float* slot = sm.red_slot[w][s2];
#pragma unroll
          for (int e = 0; e < 32; ++e) slot[e * 32 + lane] = __uint_as_float(v[s2][e]);
        }
        fence_proxy_async_smem();
        __syncwarp();
        if (lane == 0) {
#pragma unroll
          for (int s2 = 0; s2 < 2; ++s2) {
            // D = 128: queries [32 (2 half + s2), +32) x this warp's head dims; D = 64: this warp's queries x head dims [32 s2, +32)
            float* dst = D == 128 ? tile_dst + ((size_t)(half * 2 + s2) * 4 + w) * 1024
                                  : tile_dst + ((size_t)w * 2 + s2) * 1024;
            asm volatile("cp.reduce.async.bulk.global.shared::cta.bulk_group.add.f32 [%0], [%1], %2;" ::"l"(dst),
                         "r"(smem_u32(sm.red_slot[w][s2])), "r"(4096)
                         : "memory");
          }
          tma_commit_group();
        }
      }
    }
    if (lane == 0) tma_wait_group<0>();  // all reductions have landed before the CTA exits
    __syncwarp();
  } else if (warp == 12) {
    // ============================================================ MMA issuer (warp-uniform, one elected lane issues)
    reg_dealloc<48>();
    if (n_iter > 0) {
      constexpr uint32_t kStageStep = Smem::kTileBytes >> 4;
      const uint32_t k_lo = desc_lo(smem_u32(sm.k), 16), v_lo = desc_lo(smem_u32(sm.v), 16);
      const uint32_t k_mn_lo = desc_lo(smem_u32(sm.k), kRegionBytes);
      const uint32_t q_lo0 = desc_lo(smem_u32(sm.q[0]), 16), do_lo = desc_lo(smem_u32(sm.d_o), 16);
      const uint32_t q_mn_lo0 = desc_lo(smem_u32(sm.q[0]), kRegionBytes);
      const uint32_t do_mn_lo = desc_lo(smem_u32(sm.d_o), kRegionBytes);
      const uint32_t ds_mn_lo = desc_lo(smem_u32(sm.ds), kRegionBytes);
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
          if (!(ok = wait_bar(&sm.do_full, it & 1))) break;
          // D = 128: dQ^T of the previous tile sits in this region until the drain warps hold it in registers
          if (D == 128 && it > 0 && !(ok = wait_bar(&sm.dq_drained, (it - 1) & 1))) break;
          tc_fence_after();
          ss_kmajor(kColR1, v_lo, do_lo, &sm.dp_full);  // dP^T(it)
          if (!(ok = wait_bar(&sm.p_ready, it & 1))) break;
          tc_fence_after();
          ts_acc(kColDv, kColR0, do_mn_lo, it > 0 ? 1u : 0u);  // dV += P^T dO
          if (elect_one()) mma_commit(&sm.do_empty);           // dO_i is free once these MMAs retire
          __syncwarp();
          if (it + 1 < n_iter) {
            if (!(ok = wait_bar(&sm.q_full[stage ^ 1], ((it + 1) >> 1) & 1))) break;
            ss_kmajor(kColR0, k_lo, q_lo0 + (stage ^ 1) * kStageStep, &sm.s_full);  // S^T(it + 1)
          }
          if (!(ok = wait_bar(&sm.dst_ready, it & 1))) break;
          tc_fence_after();
          ts_acc(kColDk, kColR1, q_mn_lo0 + stage * kStageStep, it > 0 ? 1u : 0u);  // dK += dS^T Q
          if (!(ok = wait_bar(&sm.ds_ready, it & 1))) break;
          tc_fence_after();
          // D = 64: dQ has a region of its own, free again once the drain warps hold the previous tile
          if (D == 64 && it > 0 && !(ok = wait_bar(&sm.dq_drained, (it - 1) & 1))) break;
          if (D == 64) tc_fence_after();
          if (elect_one()) {
#pragma unroll
            for (int kk = 0; kk < 8; ++kk) {
              if (D == 128)  // dQ^T = K^T dS^T: rows = head dim, columns = queries
                mma_ss_lohi(tmem + kColDq, k_mn_lo + ((kk * 2048) >> 4), ds_mn_lo + ((kk * 2048) >> 4), kDescHiSw128,
                            kIdescDq, kk > 0);
              else  // dQ = dS K: rows = queries (A = dS^T read transposed), columns = head dim
                mma_ss_lohi(tmem + kColDq, ds_mn_lo + ((kk * 2048) >> 4), k_mn_lo + ((kk * 2048) >> 4), kDescHiSw128,
                            kIdescDq, kk > 0);
            }
            mma_commit(&sm.dq_full);
            mma_commit(&sm.q_empty[stage]);
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
    // ============================================================ TMA producer
    reg_dealloc<48>();
    if (n_iter > 0 && lane == 0) {
      mbar_expect_tx(&sm.kv_full, 2 * Smem::kTileBytes);
      for (int rg = 0; rg < kRegions; ++rg) {
        tma_load_4d(sm.k + rg * kRegionBytes, &tm_k, &sm.kv_full, rg * 64, hk, k_row0 + j0, tma_b);
        tma_load_4d(sm.v + rg * kRegionBytes, &tm_v, &sm.kv_full, rg * 64, hk, k_row0 + j0, tma_b);
      }
      for (int it = 0; it < n_iter; ++it) {
        const int stage = it & 1;
        const int h = hk * group + it / iters_per_head;
        const int i = i_first + (it % iters_per_head + q_rot) % iters_per_head;
        if (it >= 2 && !mbar_wait(&sm.q_empty[stage], ((it >> 1) - 1) & 1, abort_flag)) break;
        const size_t row_off = acc_row0 + (size_t)h * acc_head_stride + (size_t)i * 128;
        mbar_expect_tx(&sm.q_full[stage], Smem::kTileBytes + 1024);
        for (int rg = 0; rg < kRegions; ++rg)
          tma_load_4d(sm.q[stage] + rg * kRegionBytes, &tm_q, &sm.q_full[stage], rg * 64, h, q_row0 + i * 128, tma_b);
        bulk_load_1d(sm.lse2[stage], p.lse2 + row_off, 512, &sm.q_full[stage]);
        bulk_load_1d(sm.delta[stage], p.delta + row_off, 512, &sm.q_full[stage]);
        if (it >= 1 && !mbar_wait(&sm.do_empty, (it - 1) & 1, abort_flag)) break;
        mbar_expect_tx(&sm.do_full, Smem::kTileBytes);
        for (int rg = 0; rg < kRegions; ++rg)
          tma_load_4d(sm.d_o + rg * kRegionBytes, &tm_do, &sm.do_full, rg * 64, h, q_row0 + i * 128, tma_b);
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

// Matmuls of 129..256 rows with few output columns (O-proj and down of batched decode steps), the
// weights as the MMA's 128-row operand: D[n, m] = sum_k W[n, k] X[m, k].
//
// Why.  With X as the 128-row operand a 256-row matmul is two row tiles, every 128-column tile of W is
// multiplied twice, and a matrix of 28-36 column tiles gives 56-72 tiles for 148 SMs, which the unit-range
// kernel then splits along K with partial tiles through L2 (measured 40-72 us against 7-25 us of weight
// streaming).  Here one accumulator of 128 lanes (rows of W) x up to 256 columns (all rows of X) holds a
// whole column tile of the output; a cluster of C CTAs owns the tile and splits K, so every weight
// byte crosses the L2 fabric once and T * C CTAs stream at the same time.
//
// Reduction.  After its last MMA a CTA's ring is idle, and the partial sums are staged there: for each
// peer r' the columns [r' * Mc, (r' + 1) * Mc) (Mc = columns / C rows of X) of this CTA's accumulator,
// as [Mc / 4][128 lanes][4] floats (16-byte stores and loads of consecutive lanes never collide).  One
// cluster barrier; then CTA r adds, for its own Mc columns, the partials of all ranks in rank order (its
// own straight from tensor memory, the others through remote loads) and runs the epilogue; a second
// cluster barrier keeps every CTA until its peers have read its staging area.
//
// Epilogue.  A thread holds one output column n (its TMEM lane) for 32 rows m at a time, so stores of
// one row are contiguous over the warp.  Residual update with bf16 copy and the sums of squares of
// 32-column chunks (one warp = one chunk: shuffle tree); fp32 / bf16 output.  Row factors of the folded
// RMSNorm of the CTA's rows are prepared in shared memory while the MMAs run.  (A RoPE + cache-write
// epilogue in this orientation -- a tile is one head, the members of a RoPE pair in neighbouring lanes,
// two-byte stores per row -- measured slower than the unit-range kernel's and is not kept.)
//
// Warp roles: 0 requests weights (one bulk copy of a 16 KB block per K slab) and activations (one TMA
// tile of all rows), 1 issues tcgen05.mma (128 x columns x 16) and owns tensor memory, 2-5 epilogue.
#pragma once
#include <cuda.h>

#include "common.cuh"
#include "gemm_tc.cuh"
#include "ptx_sm100.cuh"

namespace d3 {
namespace tc {

constexpr int XT_THREADS = 192;

struct XtSplit {
  int C;       // CTAs per cluster = K parts (1, 2, 4 or 8)
  int n_cols;  // columns of the accumulator: rows of X rounded up to a multiple of 32 * C, at most 256
};

inline size_t gemm_xt_smem_bytes(int n_cols, int stages) {
  return 1024 + static_cast<size_t>(stages) * (128 * 128 + static_cast<size_t>(n_cols) * 128) + (2 * stages + 2) * 8 + 64 +
         2 * 256 * 4;
}

// grid = (N / 128) * C, cluster dims (C, 1, 1).  Dynamic shared memory: [stages x 16 KB] W slabs,
// [stages x n_cols x 128 B] X slabs (both reused as the staging area), barriers, row tables.
template <int EPI>
__global__ void __launch_bounds__(XT_THREADS, 1)
gemm_xt_kernel(const __grid_constant__ CUtensorMap tmap_x, const GemmParams p, const XtSplit xs) {
  if (p.skip_flag != nullptr && *p.skip_flag != 0) return;
  grid_dep_launch();
  extern __shared__ uint8_t smem_raw[];
  uint8_t* smem = reinterpret_cast<uint8_t*>((reinterpret_cast<uintptr_t>(smem_raw) + 1023) & ~uintptr_t(1023));
  const int stages = p.stages;
  constexpr uint32_t w_stage_bytes = 128u * 128u;
  const uint32_t x_stage_bytes = static_cast<uint32_t>(xs.n_cols) * 128u;
  uint8_t* smem_w = smem;
  uint8_t* smem_x = smem + static_cast<size_t>(stages) * w_stage_bytes;
  uint8_t* tail = smem_x + static_cast<size_t>(stages) * x_stage_bytes;
  uint64_t* full_bar = reinterpret_cast<uint64_t*>(tail);
  uint64_t* empty_bar = full_bar + stages;
  uint64_t* acc_full = empty_bar + stages;
  uint32_t* tmem_slot = reinterpret_cast<uint32_t*>(acc_full + 1);
  volatile int* abort_flag = reinterpret_cast<volatile int*>(tmem_slot + 1);
  float* rs_sm = reinterpret_cast<float*>(tmem_slot + 4);  // [256] row factor of every row of X this CTA finishes

  const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
  const int C = xs.C;
  const int rank = C > 1 ? static_cast<int>(cluster_ctarank()) : 0;
  const int tile = blockIdx.x / C;  // 128 rows of W
  const int KC = p.k_chunks;
  const int kc0 = KC * rank / C, n_k = KC * (rank + 1) / C - kc0;
  const int Mc = xs.n_cols / C;     // columns this CTA finishes: a multiple of 32
  constexpr uint32_t TMEM_COLS = 256;

  if (threadIdx.x == 0) {
    prefetch_tensormap(&tmap_x);
    for (int s = 0; s < stages; ++s) {
      mbar_init(&full_bar[s], 1);
      mbar_init(&empty_bar[s], 1);
    }
    mbar_init(acc_full, 1);
    *abort_flag = 0;
    fence_barrier_init();
  }
  if (warp == 1) {
    tmem_alloc<TMEM_COLS>(tmem_slot);
    tmem_relinquish();
  }
  tc_fence_before();
  __syncthreads();
  tc_fence_after();
  const uint32_t tmem_base = *tmem_slot;
  bool alive = true;  // epilogue warps: the accumulator is complete

  if (warp == 0) {
    // ---------------- requests: weights of the first ring lap before the dependency wait, activations after it
    if (lane == 0) {
      const __nv_bfloat16* wsrc = p.w_packed + (static_cast<long long>(tile) * KC + kc0) * (128 * 64);
      const uint32_t tx = w_stage_bytes + x_stage_bytes;
      const int pre = n_k < stages ? n_k : stages;
      for (int i = 0; i < pre; ++i) {
        mbar_arrive_expect_tx(&full_bar[i], tx);
        bulk_load_1d(smem_w + static_cast<size_t>(i) * w_stage_bytes, wsrc + static_cast<size_t>(i) * (128 * 64), w_stage_bytes, &full_bar[i]);
      }
      grid_dep_wait();
      for (int i = 0; i < pre; ++i)
        tma_load_2d(smem_x + static_cast<size_t>(i) * x_stage_bytes, &tmap_x, &full_bar[i], (kc0 + i) * BLOCK_K, 0);
      int s = 0;
      uint32_t ph = 0;
      for (int i = pre; i < n_k; ++i) {
        if (!mbar_wait(&empty_bar[s], ph, abort_flag, p.error_word)) break;
        mbar_arrive_expect_tx(&full_bar[s], tx);
        bulk_load_1d(smem_w + static_cast<size_t>(s) * w_stage_bytes, wsrc + static_cast<size_t>(i) * (128 * 64), w_stage_bytes, &full_bar[s]);
        tma_load_2d(smem_x + static_cast<size_t>(s) * x_stage_bytes, &tmap_x, &full_bar[s], (kc0 + i) * BLOCK_K, 0);
        if (++s == stages) { s = 0; ph ^= 1u; }
      }
    }
  } else if (warp == 1) {
    // ---------------- MMA issue: A = weights (128 rows), B = activations (n_cols rows)
    if (lane == 0) {
      const uint32_t idesc = make_idesc(128, xs.n_cols);
      const uint64_t adesc0 = make_smem_desc(smem_u32(smem_w)), bdesc0 = make_smem_desc(smem_u32(smem_x));
      const uint64_t a_step = w_stage_bytes >> 4, b_step = x_stage_bytes >> 4;
      int s = 0;
      uint32_t ph = 0;
      bool ok = true;
      for (int i = 0; i < n_k; ++i) {
        if (!mbar_wait(&full_bar[s], ph, abort_flag, p.error_word)) { ok = false; break; }
        tc_fence_after();
        const uint64_t adesc = adesc0 + a_step * static_cast<uint64_t>(s), bdesc = bdesc0 + b_step * static_cast<uint64_t>(s);
#pragma unroll
        for (int kk = 0; kk < BLOCK_K / UMMA_K; ++kk)
          umma_bf16(tmem_base, adesc + static_cast<uint64_t>(2 * kk), bdesc + static_cast<uint64_t>(2 * kk), idesc,
                    (i > 0 || kk > 0) ? 1u : 0u);
        umma_commit(&empty_bar[s]);
        if (++s == stages) { s = 0; ph ^= 1u; }
      }
      if (ok) umma_commit(acc_full);
    }
  } else {
    // ---------------- epilogue warps, part 1: tables, then the peers' columns into the staging area
    grid_dep_wait();
    const int et = threadIdx.x - 64;  // 0..127 = TMEM lane = row of W inside the tile
    const int lg = warp & 3;
    // rows of X this CTA finishes: their row factor (folded RMSNorm) and, for the QKV epilogue, cache slot
    for (int j = et; j < Mc; j += 128) {
      const int m = rank * Mc + j;
      float rs = 1.f;
      if (m < p.M && EPI != EPI_RESID && p.ep.ssq_in != nullptr) rs = row_rstd(p.ep, m);
      rs_sm[j] = rs;
    }
    bool ok = mbar_wait(acc_full, 0u, abort_flag, p.error_word);
    alive = __all_sync(0xffffffffu, ok);
    tc_fence_after();
    if (alive && C > 1) {
      // (the ring is idle: every copy into it was consumed by an MMA that has completed)
      const uint32_t lane_addr = tmem_base + (static_cast<uint32_t>(((warp & 3) * 32)) << 16);
      float4* stage4 = reinterpret_cast<float4*>(smem);
      for (int r2 = 0; r2 < C; ++r2) {
        if (r2 == rank) continue;
        for (int c = 0; c < Mc; c += 32) {
          float v[32];
          tmem_ld_32x32(lane_addr + static_cast<uint32_t>(r2 * Mc + c), v);
          tmem_ld_wait();
          float4* dst = stage4 + (static_cast<size_t>(r2) * (Mc / 4) + c / 4) * 128 + (lg * 32 + lane);
#pragma unroll
          for (int q = 0; q < 8; ++q) dst[static_cast<size_t>(q) * 128] = make_float4(v[4 * q], v[4 * q + 1], v[4 * q + 2], v[4 * q + 3]);
        }
      }
    }
    (void)et;
  }
  __syncthreads();
  if (C > 1) cluster_sync_all();  // every CTA's staging area is complete
  if (warp >= 2) {
    // ---------------- epilogue warps, part 2: this CTA's columns, partials added in rank order
    const int lg = warp & 3;
    const int n_local = lg * 32 + lane;
    const int n = tile * 128 + n_local;
    const uint32_t lane_addr = tmem_base + (static_cast<uint32_t>(lg * 32) << 16);
    const uint32_t stage_addr = smem_u32(smem);
    alive = alive && (*abort_flag == 0);
    for (int c = 0; c < Mc && alive; c += 32) {
      float own[32], acc[32];
      tmem_ld_32x32(lane_addr + static_cast<uint32_t>(rank * Mc + c), own);
      tmem_ld_wait();
#pragma unroll
      for (int j = 0; j < 32; ++j) acc[j] = 0.f;
      for (int s2 = 0; s2 < C; ++s2) {
        if (s2 == rank) {
#pragma unroll
          for (int j = 0; j < 32; ++j) acc[j] += own[j];
        } else {
          const uint32_t base = map_to_cta(stage_addr + static_cast<uint32_t>(((rank * (Mc / 4) + c / 4) * 128 + n_local) * 16), static_cast<uint32_t>(s2));
          float4 part[8];
#pragma unroll
          for (int q = 0; q < 8; ++q) part[q] = ld_cluster_f4(base + static_cast<uint32_t>(q * 128 * 16));
#pragma unroll
          for (int q = 0; q < 8; ++q) {
            acc[4 * q] += part[q].x; acc[4 * q + 1] += part[q].y; acc[4 * q + 2] += part[q].z; acc[4 * q + 3] += part[q].w;
          }
        }
      }
      const int m0 = rank * Mc + c;
      if constexpr (EPI == EPI_RESID) {
        float* y = static_cast<float*>(p.ep.y);
        const bool n_ok = n < p.N;
        float o[32];
#pragma unroll
        for (int j = 0; j < 32; ++j) o[j] = (n_ok && m0 + j < p.M) ? y[static_cast<size_t>(m0 + j) * p.ep.ldy + n] : 0.f;  // all loads in flight
#pragma unroll
        for (int j = 0; j < 32; ++j) {
          const int m = m0 + j;
          const bool live = n_ok && m < p.M;
          const float v = o[j] + acc[j];
          if (live) {
            y[static_cast<size_t>(m) * p.ep.ldy + n] = v;
            if (p.ep.yb != nullptr) p.ep.yb[static_cast<size_t>(m) * p.ep.ldy + n] = __float2bfloat16_rn(v);
          }
          // the warp's 32 lanes are the 32 columns of one chunk: sum of squares in a fixed tree
          float sq = live ? v * v : 0.f;
#pragma unroll
          for (int d = 1; d < 32; d <<= 1) sq += __shfl_xor_sync(0xffffffffu, sq, d);
          if (lane == 0 && m < p.M && p.ep.ssq_out != nullptr && tile * 128 + lg * 32 < p.N)
            p.ep.ssq_out[static_cast<size_t>(m) * ((p.N + 31) / 32) + (tile * 128 + lg * 32) / 32] = sq;
        }
      } else if constexpr (EPI == EPI_F32 || EPI == EPI_T) {
#pragma unroll
        for (int j = 0; j < 32; ++j) {
          const int m = m0 + j;
          if (n < p.N && m < p.M) {
            const float v = acc[j] * rs_sm[c + j] * (EPI == EPI_F32 ? p.ep.scale : 1.f);
            if constexpr (EPI == EPI_F32) static_cast<float*>(p.ep.y)[static_cast<size_t>(m) * p.ep.ldy + n] = v;
            else static_cast<__nv_bfloat16*>(p.ep.y)[static_cast<size_t>(m) * p.ep.ldy + n] = __float2bfloat16_rn(v);
          }
        }
      }
    }
    tc_fence_before();
  }
  __syncthreads();
  if (C > 1) cluster_sync_all();  // no CTA leaves while a peer may still read its staging area
  if (warp == 1) {
    tc_fence_after();
    tmem_dealloc<TMEM_COLS>(tmem_base);
  }
}

}  // namespace tc
}  // namespace d3

// Matmuls Y = X W^T of more than 128 rows on CTA pairs: a cluster of two CTAs owns a 256 x 256 tile of Y and
// one tcgen05.mma.cta_group::2 of M = 256 computes it.  Each CTA stages its own 128 rows of X (TMA) and its own
// 128 of the tile's 256 weight rows (one pre-swizzled 16 KB block) per 64-wide K slab, both by TMA: 32 KB of shared
// memory traffic per CTA and slab where a lone CTA with a 128 x 256 tile moves 48 KB for the same arithmetic.  The
// L2-to-shared-memory path is what paces those tiles, so the pair form gains what it saves there.
//
// Per CTA, 192 threads: warp 0 producer (one thread), warp 1 the MMA thread (in the leader, rank 0, only), warps 2-5
// epilogue (one row = one tensor-memory lane per thread).
// Hand-over per ring stage s:
//   producer (both CTAs)  waits its empty[s] and issues its two tile loads (cta_group::2 form: the bytes land in
//                         its own shared memory and are counted on the LEADER's full[s]); the leader's producer
//                         first expects the 64 KB of both CTAs there
//   MMA thread (leader)   waits full[s], issues four MMAs (K = 16 each) that read both CTAs' stages, commits to
//                         empty[s] of both CTAs (tcgen05.commit with a CTA mask)
// (A first form, in which the peer's loads were counted on its own barrier and a relay thread passed each stage on
// to the leader with a remote arrive, ran at half the speed of the single-CTA kernel: the extra hop per stage is
// longer than the six stages cover.)  The weights, pre-swizzled 128 x 64 blocks stored one after the other, are read
// through a tensor map over [blocks * 128 rows][64] without swizzle, which copies a block verbatim.
// Accumulators: two of 256 columns per CTA (all 512 columns, allocated pair-wide), so that the epilogue of a tile
// runs under the MMAs of the next one; the last commit of a tile goes to acc_full[buf] of both CTAs, and every
// epilogue warp of both CTAs arrives on the leader's acc_empty[buf] when it has read its lanes.
// Tiles are dealt round-robin to the pairs in bands of eight row tiles (2048 rows), row tiles fastest inside a band:
// the pairs of a moment share a few weight blocks, and a band's rows of X stay in L2 while all column tiles pass
// (with row tiles fastest over all of a 16384-row X, every column tile streamed X from HBM again: 17 % slower).  Epilogues are those of gemm_tc.cuh (run_epilogue on 256 columns).
#pragma once
#include "gemm_tc.cuh"

namespace d3 {
namespace tc {

constexpr int PAIR_THREADS = 192;
constexpr int PAIR_STAGES = 6;
constexpr int PAIR_BAND = 8;  // row tiles per band of the tile order
constexpr uint32_t PAIR_A_BYTES = 128u * 128u;  // [128 rows][64 bf16]
constexpr uint32_t PAIR_B_BYTES = 128u * 128u;  // one weight block
constexpr uint32_t PAIR_STAGE_BYTES = PAIR_A_BYTES + PAIR_B_BYTES;

// kind::f16 instruction descriptor of the pair MMA: D fp32, A and B bf16 K-major, N >> 3 in [17,23), M >> 4 in [24,29).
constexpr uint32_t PAIR_IDESC = (1u << 4) | (1u << 7) | (1u << 10) | (static_cast<uint32_t>(256 >> 3) << 17) |
                                (static_cast<uint32_t>(256 >> 4) << 24);

__device__ __forceinline__ void pair_tile_mn(int q, int m_tiles, int n_tiles, int& m_t, int& n_t) {
  const int band_sz = PAIR_BAND * n_tiles;
  const int band = q / band_sz, r = q - band * band_sz;
  const int rows_here = min(PAIR_BAND, m_tiles - band * PAIR_BAND);
  n_t = r / rows_here;
  m_t = band * PAIR_BAND + r % rows_here;
}

inline size_t gemm_pair_smem_bytes() { return 1024 + PAIR_STAGES * PAIR_STAGE_BYTES + (2 * PAIR_STAGES + 4) * 8 + 64; }

// grid = 2 x pairs, cluster (2, 1, 1).  p: M, N (multiple of 256), K (multiple of 64), k_chunks, w_packed (tiled
// weights), ep and, for EPI_QKV, the RoPE and cache fields.  tmap_x: X as [M, K] with boxes of 128 rows (128-byte
// swizzle); tmap_w: the weight blocks as [N / 128 * k_chunks * 128, 64] with boxes of 128 rows, no swizzle.
template <int EPI>
__global__ void __launch_bounds__(PAIR_THREADS, 1) gemm_pair_kernel(const __grid_constant__ CUtensorMap tmap_x,
                                                                    const __grid_constant__ CUtensorMap tmap_w, const GemmParams p) {
  if (p.skip_flag != nullptr && *p.skip_flag != 0) return;  // uniform over the grid
  grid_dep_launch();
  extern __shared__ uint8_t smem_raw[];
  uint8_t* smem = reinterpret_cast<uint8_t*>((reinterpret_cast<uintptr_t>(smem_raw) + 1023) & ~uintptr_t(1023));
  uint64_t* full_bar = reinterpret_cast<uint64_t*>(smem + PAIR_STAGES * PAIR_STAGE_BYTES);
  uint64_t* empty_bar = full_bar + PAIR_STAGES;
  uint64_t* acc_full = empty_bar + PAIR_STAGES;   // [2]
  uint64_t* acc_empty = acc_full + 2;             // [2], used in the leader only
  uint32_t* tmem_slot = reinterpret_cast<uint32_t*>(acc_empty + 2);
  volatile int* abort_flag = reinterpret_cast<volatile int*>(tmem_slot + 1);

  const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
  const uint32_t rank = cluster_ctarank();
  const int pair = blockIdx.x >> 1, n_pairs = gridDim.x >> 1;
  const int m_tiles = (p.M + 255) / 256, n_tiles = p.N / 256;
  const int tiles = m_tiles * n_tiles;
  const int my_tiles = pair < tiles ? (tiles - pair + n_pairs - 1) / n_pairs : 0;
  const int KC = p.k_chunks;
  // A row tile that lies wholly in the unused tail of a sequence's rows (padded prompts) is passed over by all three
  // roles alike.  (The row map was written before the forward's first kernel started: readable before the dependency wait.)
  auto tile_dead = [&](int m_t) {
    if (p.live_n_valid == nullptr) return false;
    const int row0 = m_t * 256;
    return row0 % p.live_rps >= p.live_n_valid[row0 / p.live_rps];
  };

  if (threadIdx.x == 0) {
    prefetch_tensormap(&tmap_x);
    prefetch_tensormap(&tmap_w);
    for (int s = 0; s < PAIR_STAGES; ++s) {
      mbar_init(&full_bar[s], 1);
      mbar_init(&empty_bar[s], 1);
    }
    for (int b = 0; b < 2; ++b) {
      mbar_init(&acc_full[b], 1);
      mbar_init(&acc_empty[b], 8);  // four epilogue warps of each CTA
    }
    *abort_flag = 0;
    fence_barrier_init();
  }
  if (warp == 1) {
    tmem_alloc_pair<512>(tmem_slot);
    tmem_relinquish_pair();
  }
  tc_fence_before();
  cluster_sync_all();  // barriers of both CTAs exist before either signals the other
  tc_fence_after();
  const uint32_t tmem_base = *tmem_slot;

  if (warp == 0) {
    // ------------------------------------------------------------------ producer
    if (lane == 0) {
      grid_dep_wait();  // X comes from the kernel before this one
      int it = 0;
      bool ok = true;
      for (int t = 0; t < my_tiles && ok; ++t) {
        const int q = pair + t * n_pairs;
        int m_t, n_t;
        pair_tile_mn(q, m_tiles, n_tiles, m_t, n_t);
        if (tile_dead(m_t)) continue;
        const int row0 = m_t * 256 + static_cast<int>(rank) * 128;
        const int wrow0 = (n_t * 2 + static_cast<int>(rank)) * KC * 128;  // first row of this CTA's first weight block
        for (int kc = 0; kc < KC; ++kc, ++it) {
          const int s = it % PAIR_STAGES;
          if (it >= PAIR_STAGES && !mbar_wait(&empty_bar[s], static_cast<uint32_t>(it / PAIR_STAGES - 1) & 1u, abort_flag, p.error_word)) {
            ok = false;
            break;
          }
          uint8_t* st = smem + s * PAIR_STAGE_BYTES;
          if (rank == 0) mbar_arrive_expect_tx(&full_bar[s], 2 * PAIR_STAGE_BYTES);
          const uint32_t lead_full = map_to_cta(smem_u32(&full_bar[s]), 0);
          tma_load_2d_pair(st, &tmap_x, lead_full, kc * 64, row0);
          tma_load_2d_pair(st + PAIR_A_BYTES, &tmap_w, lead_full, 0, wrow0 + kc * 128);
        }
      }
    }
  } else if (warp == 1) {
    if (lane == 0) {
      if (rank == 0) {
        // -------------------------------------------------------------- MMA issue (leader)
        const uint32_t sb = smem_u32(smem);
        int it = 0;
        bool ok = true;
        int n_done = 0;  // tiles computed so far: accumulator buffer and barrier phases
        for (int t = 0; t < my_tiles && ok; ++t) {
          int m_t, n_t;
          pair_tile_mn(pair + t * n_pairs, m_tiles, n_tiles, m_t, n_t);
          if (tile_dead(m_t)) continue;
          const int buf = n_done & 1;
          if (n_done >= 2) ok = mbar_wait_cluster(&acc_empty[buf], static_cast<uint32_t>((n_done >> 1) - 1) & 1u, abort_flag, p.error_word);
          if (!ok) break;
          tc_fence_after();
          const uint32_t tmem_d = tmem_base + static_cast<uint32_t>(buf * 256);
          for (int kc = 0; kc < KC; ++kc, ++it) {
            const int s = it % PAIR_STAGES;
            const uint32_t ph = static_cast<uint32_t>(it / PAIR_STAGES) & 1u;
            ok = mbar_wait_cluster(&full_bar[s], ph, abort_flag, p.error_word);
            if (!ok) break;
            tc_fence_after();
            const uint64_t adesc = make_smem_desc(sb + s * PAIR_STAGE_BYTES);
            const uint64_t bdesc = make_smem_desc(sb + s * PAIR_STAGE_BYTES + PAIR_A_BYTES);
#pragma unroll
            for (int kk = 0; kk < BLOCK_K / UMMA_K; ++kk)
              umma_bf16_pair(tmem_d, adesc + static_cast<uint64_t>(2 * kk), bdesc + static_cast<uint64_t>(2 * kk), PAIR_IDESC,
                             (kc > 0 || kk > 0) ? 1u : 0u);
            umma_commit_pair(&empty_bar[s], 3);
          }
          if (ok) umma_commit_pair(&acc_full[buf], 3);
          ++n_done;
        }
      }
    }
  } else {
    // ------------------------------------------------------------------ epilogue warps: lane group = warp % 4
    grid_dep_wait();  // residual rows, positions and row sums come from earlier kernels
    const int lg = warp & 3;
    const int row = lg * 32 + lane;
    int n_done = 0;
    for (int t = 0; t < my_tiles; ++t) {
      const int q = pair + t * n_pairs;
      int m_t, n_t;
      pair_tile_mn(q, m_tiles, n_tiles, m_t, n_t);
      if (tile_dead(m_t)) continue;
      const int m = m_t * 256 + static_cast<int>(rank) * 128 + row;
      const int buf = n_done & 1;
      float rs = 1.f;  // folded RMSNorm: the row's factor, fetched while the MMAs still run
      if (p.ep.ssq_in != nullptr && m < p.M) rs = row_rstd(p.ep, m);
      bool ok = mbar_wait(&acc_full[buf], static_cast<uint32_t>(n_done >> 1) & 1u, abort_flag, p.error_word);
      ok = __all_sync(0xffffffffu, ok);
      if (!ok) break;
      tc_fence_after();
      const bool warp_live = m_t * 256 + static_cast<int>(rank) * 128 + lg * 32 < p.M;  // warp-uniform
      TmemSource tsrc{tmem_base + static_cast<uint32_t>(buf * 256) + (static_cast<uint32_t>(lg * 32) << 16)};
      if (warp_live) run_epilogue<EPI, 256>(tsrc, p, m, n_t * 256, m < p.M, 0, 1, -1, rs);
      tc_fence_before();
      __syncwarp();
      if (lane == 0) mbar_arrive_remote(&acc_empty[buf], 0);
      ++n_done;
    }
  }
  // Neither CTA may leave (its shared memory is an operand of the leader's MMAs, its barriers a target of the
  // leader's commits) nor give back tensor memory before both are through.
  __syncwarp();
  tc_fence_before();
  cluster_sync_all();
  if (warp == 1) tmem_dealloc_pair<512>(tmem_base);
}

}  // namespace tc
}  // namespace d3

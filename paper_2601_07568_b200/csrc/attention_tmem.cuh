// Block-bidirectional attention (Sec. 3.2: every row of the block sees the whole prefix and the block itself,
// no causal mask) with both products on the tcgen05 tensor cores and S, P, O and Q in tensor memory.
// bf16, d_head = 128.
//
// One CTA = one (sequence, kv head, query tile, key split), 192 threads:
//   warps 0-3  softmax: thread t owns row t of the tile = tensor-memory lane t
//   warp 4     producer: K and V tiles of KT keys by TMA (128-byte swizzle) into a ring of six stages
//   warp 5     one thread issues the MMAs; the warp owns the tensor-memory allocation
// Per key tile i:  S_i = Q K_i^T   M = 128 rows, N = KT keys, K = d_head; Q is the A operand from tensor memory
//                                  (64 columns: two bf16 per column), K_i a K-major B operand in shared memory
//                  P_i = exp2(S_i * scale - m) as bf16, stored by the softmax threads over the first KT / 2 columns
//                        of S_i's own buffer (every thread has read its row of S_i before it writes there)
//                  O  += P_i V_i   N = d_head, K = KT keys; P_i is the A operand from tensor memory; V as it lies
//                                  in the cache, [key][d], is an MN-major B operand: 64 d values = one 128-byte
//                                  swizzle row, 8 keys = one 1024-byte atom
// With both A operands in tensor memory an MMA step reads 4 KB of shared memory instead of 8 (the shared-memory
// port, 128 bytes a clock, is what paces a 128 x 128 x 16 step with two shared-memory operands), and shared
// memory holds nothing but K and V tiles in flight.
// With two S buffers the first product of tile i + 1 runs under the softmax of tile i.  O accumulates over all tiles inside the MMA.  The exponentials are taken against a reference m
// that follows the row maximum lazily: it moves only when a tile's maximum exceeds it by more than 2^8, and only
// then are the row sum and the O row (tcgen05.ld, scale, tcgen05.st) rescaled.  P <= 2^8 is exact enough in bf16,
// the sums are fp32, and the quotient O / l does not depend on m.
//
// Fewer than 128 packed rows leave lanes (and whole warps, which then skip the softmax) idle; the MMAs do not care.
//
// Two shapes of the same code:  <128 keys per tile>: 448 columns of tensor memory, 192 KB of K/V in flight, one CTA
// per SM, for long key ranges;  <64>: 256 columns (Q stays in shared memory and the first product takes both
// operands from there), 64 KB in flight, two CTAs per SM, whose start-up and output overlap the other's tile loop:
// for short key ranges, where a CTA lives for a few tiles only.
//
// Key splits: as in attn_tc_kernel, the CTAs of one query tile form a cluster along z and merge their partials
// through distributed shared memory.
#pragma once
#include "attention.cuh"

namespace d3 {
namespace attn {

constexpr int TM_THREADS = 192;
constexpr float TM_SLACK_LOG2 = 8.f;           // how far a tile's maximum may exceed the reference before it moves

// K-major operand slab, 128-byte swizzle: rows of 128 bytes, 8-row atoms 1024 bytes apart (stride byte offset);
// the leading byte offset is not used by this form.  Bits: start address >> 4 in [0,14), LBO >> 4 in [16,30),
// SBO >> 4 in [32,46), descriptor version 1 in [46,48), swizzle mode 2 (128 bytes) in [61,64).
__device__ __forceinline__ uint64_t tm_desc_k(uint32_t smem_addr) {
  return static_cast<uint64_t>((smem_addr & 0x3FFFF) >> 4) | (1ull << 16) | (static_cast<uint64_t>(1024 >> 4) << 32) |
         (1ull << 46) | (2ull << 61);
}
// MN-major operand, 128-byte swizzle: 64 consecutive MN elements per 128-byte row, one row per K index, atoms of
// 8 K indices (1024 bytes) `sbo` bytes apart, blocks of 64 MN elements `lbo` bytes apart.
__device__ __forceinline__ uint64_t tm_desc_mn(uint32_t smem_addr, uint32_t lbo, uint32_t sbo) {
  return static_cast<uint64_t>((smem_addr & 0x3FFFF) >> 4) | (static_cast<uint64_t>(lbo >> 4) << 16) |
         (static_cast<uint64_t>(sbo >> 4) << 32) | (1ull << 46) | (2ull << 61);
}
// kind::f16 instruction descriptor: D fp32, A and B bf16, A K-major, B K-major or MN-major (bit 16).
__host__ __device__ constexpr uint32_t tm_idesc(int m, int n, bool b_mn) {
  return (1u << 4) | (1u << 7) | (1u << 10) | (b_mn ? (1u << 16) : 0u) | (static_cast<uint32_t>(n >> 3) << 17) |
         (static_cast<uint32_t>(m >> 4) << 24);
}


template <int KT, int SBUF>
struct TmLayout {
  static constexpr uint32_t SLAB = static_cast<uint32_t>(KT) * 128u;  // [KT keys][64 bf16], swizzled
  static constexpr uint32_t TILE = 2u * SLAB;                         // one K or V tile: d 0-63, d 64-127
  // The small shape keeps Q in shared memory (two K-major slabs of [128 rows][64 bf16]): S twice, O and Q together
  // do not fit the 256 columns that let two CTAs share an SM's tensor memory.
  static constexpr bool Q_SMEM = KT == 64;
  static constexpr int STAGES = Q_SMEM ? 4 : 6;                       // ring of K / V tiles
  static constexpr uint32_t Q_SLAB = 128u * 128u;
  static constexpr uint32_t OFF_RING = Q_SMEM ? 2u * Q_SLAB : 0u;
  static constexpr uint32_t OFF_BAR = OFF_RING + STAGES * TILE;
  static constexpr uint32_t COL_S = 0, COL_O = SBUF * KT, COL_Q = COL_O + 128;  // tensor-memory columns
  static constexpr uint32_t COLS = (Q_SMEM ? COL_Q : COL_Q + 64) <= 256 ? 256 : 512;  // allocation: a power of two
  static constexpr size_t smem_bytes() { return 1024 + OFF_BAR + (2 * STAGES + 2 * SBUF + 4) * 8 + 64; }
};

// grid (q_tiles, bs * hkv, n_splits); 128 packed rows per query tile.
template <int KT, int SBUF>
__global__ void __launch_bounds__(TM_THREADS, KT == 64 ? 2 : 1) attn_tmem_kernel(const __grid_constant__ CUtensorMap tmap_kv,
                                                                                 const AttnTcParams p) {
  using L = TmLayout<KT, SBUF>;
  constexpr int NCH = KT / 32;  // 32-column chunks of S per thread
  constexpr int BM = 128;
  extern __shared__ uint8_t smem_raw[];
  uint8_t* smem = reinterpret_cast<uint8_t*>((reinterpret_cast<uintptr_t>(smem_raw) + 1023) & ~uintptr_t(1023));
  uint64_t* kv_full = reinterpret_cast<uint64_t*>(smem + L::OFF_BAR);
  uint64_t* kv_empty = kv_full + L::STAGES;
  uint64_t* s_full = kv_empty + L::STAGES;  // [SBUF] S_i complete in tensor memory
  uint64_t* p_full = s_full + SBUF;         // [SBUF] P_i in tensor memory (over S_i), O rescaled where it had to be
  uint64_t* o_full = p_full + SBUF;         // second product of tile i complete (O updated, P_i and V_i read)
  uint64_t* q_full = o_full + 1;            // Q in tensor memory
  uint32_t* tmem_slot = reinterpret_cast<uint32_t*>(q_full + 1);
  volatile int* abort_flag = reinterpret_cast<volatile int*>(tmem_slot + 1);

  const int warp_id = threadIdx.x >> 5, lane = threadIdx.x & 31;
  const int qt = blockIdx.x, pair = blockIdx.y, split = blockIdx.z;
  const int b = pair / p.hkv, g = pair % p.hkv;
  const int group = p.hq / p.hkv;
  const int rps = p.rm.rows_per_seq;

  // The row map was written before this forward's first kernel started and cache rows below pos_base are not
  // touched by this forward: both may be read before the dependency wait.
  const int n_valid = p.rm.n_valid[b];
  const int kv_len = p.rm.kv_len[b];
  const int stable_keys = p.rm.pos_base[b];
  const int R = group * rps;
  bool work = !(qt * BM >= R || n_valid <= 0 || kv_len <= 0);
  if (work) {
    bool any = false;
    for (int pr = qt * BM; pr < min(R, (qt + 1) * BM) && !any; pr += 1) any = (pr % rps) < n_valid;
    work = any;
  }
  if (!work) {  // uniform over the CTA and over the cluster
    ptx::grid_dep_launch();
    ptx::grid_dep_wait();
    return;
  }
  if (threadIdx.x == 0) {
    ptx::prefetch_tensormap(&tmap_kv);
    for (int s = 0; s < L::STAGES; ++s) {
      ptx::mbar_init(&kv_full[s], 1);
      ptx::mbar_init(&kv_empty[s], 1);
    }
    for (int s = 0; s < SBUF; ++s) {
      ptx::mbar_init(&s_full[s], 1);
      ptx::mbar_init(&p_full[s], 128);
    }
    ptx::mbar_init(o_full, 1);
    ptx::mbar_init(q_full, 128);
    *abort_flag = 0;
    ptx::fence_barrier_init();
  }
  if (warp_id == 5) {
    ptx::tmem_alloc<L::COLS>(tmem_slot);
    ptx::tmem_relinquish();
  }
  ptx::tc_fence_before();
  __syncthreads();
  ptx::tc_fence_after();
  const uint32_t tmem_base = *tmem_slot;
  ptx::grid_dep_launch();

  const int n_tiles = (kv_len + KT - 1) / KT;
  const int tps = (n_tiles + p.n_splits - 1) / p.n_splits;
  const int t0 = split * tps, t1 = min(n_tiles, t0 + tps);
  const int n_my = max(t1 - t0, 0);
  const uint32_t sbase = ptx::smem_u32(smem);
  bool alive = true;

  // Producer and MMA thread walk the tiles in the same order: K_0 .. K_(SBUF-1), then V_j, K_(j+SBUF) for every j.
  if (warp_id == 4) {
    // ------------------------------------------------------------------ producer
    if (lane == 0) {
      const long long krow = p.k_row0 + (static_cast<long long>(b) * p.hkv + g) * p.max_seq;
      const long long vrow = p.v_row0 + (static_cast<long long>(b) * p.hkv + g) * p.max_seq;
      bool waited = false, ok = true;
      int s = 0;  // position in the ring
      auto load = [&](bool is_k, int i) {
        const int stage = s % L::STAGES;
        if (s >= L::STAGES &&
            !ptx::mbar_wait(&kv_empty[stage], static_cast<uint32_t>(s / L::STAGES - 1) & 1u, abort_flag, p.error_word))
          return false;
        const int j0 = (t0 + i) * KT;
        if (!waited && j0 + KT > stable_keys) {  // this tile holds rows the QKV kernel of this layer writes
          ptx::grid_dep_wait();
          waited = true;
        }
        uint8_t* dst = smem + L::OFF_RING + stage * L::TILE;
        const int row = static_cast<int>((is_k ? krow : vrow) + j0);
        ptx::mbar_arrive_expect_tx(&kv_full[stage], L::TILE);
        ptx::tma_load_2d(dst, &tmap_kv, &kv_full[stage], 0, row);
        ptx::tma_load_2d(dst + L::SLAB, &tmap_kv, &kv_full[stage], 64, row);
        ++s;
        return true;
      };
      for (int i = 0; i < min(SBUF, n_my) && ok; ++i) ok = load(true, i);
      for (int j = 0; j < n_my && ok; ++j) {
        ok = load(false, j);
        if (ok && j + SBUF < n_my) ok = load(true, j + SBUF);
      }
      if (!waited) ptx::grid_dep_wait();
    }
  } else if (warp_id == 5) {
    // ------------------------------------------------------------------ MMA issue
    if (lane == 0) {
      constexpr uint32_t idesc_qk = tm_idesc(128, KT, false);
      constexpr uint32_t idesc_pv = tm_idesc(128, 128, true);
      bool ok = ptx::mbar_wait(q_full, 0, abort_flag, p.error_word);
      ptx::tc_fence_after();
      int s = 0;  // position in the ring
      auto stage_ready = [&](uint32_t& addr) {
        const int stage = s % L::STAGES;
        if (!ptx::mbar_wait(&kv_full[stage], static_cast<uint32_t>(s / L::STAGES) & 1u, abort_flag, p.error_word)) return -1;
        ptx::tc_fence_after();
        addr = sbase + L::OFF_RING + stage * L::TILE;
        ++s;
        return stage;
      };
      auto qk = [&](int i) {  // S_i into S buffer i % SBUF
        uint32_t kb;
        const int stage = stage_ready(kb);
        if (stage < 0) return false;
#pragma unroll
        for (int kk = 0; kk < 8; ++kk) {  // 16 values of d_head per step = 8 columns of Q
          const uint64_t bd = tm_desc_k(kb + (kk >> 2) * L::SLAB) + static_cast<uint64_t>(2 * (kk & 3));
          const uint32_t sd = tmem_base + L::COL_S + static_cast<uint32_t>((i % SBUF) * KT);
          if constexpr (L::Q_SMEM)
            ptx::umma_bf16(sd, tm_desc_k(sbase + (kk >> 2) * L::Q_SLAB) + static_cast<uint64_t>(2 * (kk & 3)), bd, idesc_qk, kk > 0 ? 1u : 0u);
          else
            ptx::umma_bf16_ts(sd, tmem_base + L::COL_Q + kk * 8, bd, idesc_qk, kk > 0 ? 1u : 0u);
        }
        ptx::umma_commit(&kv_empty[stage]);
        ptx::umma_commit(&s_full[i % SBUF]);
        return true;
      };
      for (int i = 0; i < min(SBUF, n_my) && ok; ++i) ok = qk(i);
      for (int i = 0; i < n_my && ok; ++i) {
        ok = ptx::mbar_wait(&p_full[i % SBUF], static_cast<uint32_t>(i / SBUF) & 1u, abort_flag, p.error_word);
        if (!ok) break;
        uint32_t vb;
        const int stage = stage_ready(vb);
        if (stage < 0) break;
        const uint32_t pcol = tmem_base + L::COL_S + static_cast<uint32_t>((i % SBUF) * KT);  // P_i lies over S_i
#pragma unroll
        for (int kk = 0; kk < KT / 16; ++kk) {  // 16 keys per step = 8 columns of P
          const uint64_t bd = tm_desc_mn(vb + kk * 2048, L::SLAB, 1024);
          ptx::umma_bf16_ts(tmem_base + L::COL_O, pcol + kk * 8, bd, idesc_pv, (i > 0 || kk > 0) ? 1u : 0u);
        }
        ptx::umma_commit(&kv_empty[stage]);
        ptx::umma_commit(o_full);
        if (i + SBUF < n_my) ok = qk(i + SBUF);  // overwrites S_i / P_i: issued after the product that reads P_i
      }
    }
  }

  // ------------------------------------------------------------------ softmax warps
  const int tid = threadIdx.x;   // row of the tile and tensor-memory lane (warps 0-3)
  const int pr = qt * BM + tid;  // packed row: head_in_group * rows_per_seq + r
  const int r_seq = pr % rps;
  const bool row_ok = warp_id < 4 && pr < R && r_seq < n_valid;
  float acc[128];
  // m_run is the reference the exponentials are taken against, not the running maximum (see the head of the file)
  float m_run = -INFINITY, l_run = 0.f;
  if (warp_id < 4) {
    const uint32_t t_lane = tmem_base + (static_cast<uint32_t>(warp_id * 32) << 16);
    const uint32_t t_o = t_lane + L::COL_O;
    const bool warp_rows = __any_sync(0xffffffffu, row_ok);  // a warp without rows only keeps the barriers going
    ptx::grid_dep_wait();  // Q comes from the kernel before this one
    {  // this thread's row of Q into its lane (128 bf16 = 64 columns) or its shared-memory row; a row that does not exist is zero
      const uint4* src = reinterpret_cast<const uint4*>(p.q + (static_cast<size_t>(b) * rps + r_seq) * p.hq * 128 +
                                                        (g * group + pr / rps) * 128);
      if constexpr (L::Q_SMEM) {
        // rows of a warp without any stay as they are: nobody reads what comes of them; a CTA without tiles needs no
        // Q, and its warps write their partials over this memory without waiting for each other
        if (warp_rows && n_my > 0) {
#pragma unroll
          for (int ch = 0; ch < 16; ++ch)
            *reinterpret_cast<uint4*>(smem + (ch >> 3) * L::Q_SLAB + swz(tid, ch & 7)) = row_ok ? src[ch] : make_uint4(0u, 0u, 0u, 0u);
          ptx::fence_proxy_async();
        }
      } else {
#pragma unroll
        for (int h = 0; h < 2; ++h) {
          uint4 v[8];
#pragma unroll
          for (int j = 0; j < 8; ++j) v[j] = row_ok ? src[h * 8 + j] : make_uint4(0u, 0u, 0u, 0u);
          ptx::tmem_st_32x32(t_lane + L::COL_Q + h * 32, *reinterpret_cast<const float(*)[32]>(v));
        }
        ptx::tmem_st_wait();
        ptx::tc_fence_before();
      }
      ptx::mbar_arrive(q_full);
    }
    const int kv_lim = row_ok ? row_kv_limit(p.rm, b, r_seq, kv_len) : kv_len;
    for (int i = 0; i < n_my && alive; ++i) {
      alive = ptx::mbar_wait(&s_full[i % SBUF], static_cast<uint32_t>(i / SBUF) & 1u, abort_flag, p.error_word);
      if (!alive) break;
      // Every thread watches every phase of o_full in order (a parity wait cannot tell a phase from the one two
      // before it): the product of tile i - 1 was issued a whole tile ago, so this wait is over before it starts.
      auto seen_o = [&]() { return i == 0 || ptx::mbar_wait(o_full, static_cast<uint32_t>(i - 1) & 1u, abort_flag, p.error_word); };
      if (!warp_rows) {  // whatever these lanes of S hold is multiplied into rows nobody reads
        alive = seen_o();
        ptx::mbar_arrive(&p_full[i % SBUF]);
        continue;
      }
      ptx::tc_fence_after();
      const int j0 = (t0 + i) * KT;
      const uint32_t t_s = t_lane + L::COL_S + static_cast<uint32_t>((i % SBUF) * KT);
      float s[NCH][32];
#pragma unroll
      for (int ch = 0; ch < NCH; ++ch) ptx::tmem_ld_32x32(t_s + ch * 32, s[ch]);
      ptx::tmem_ld_wait();
      if (!__all_sync(0xffffffffu, j0 + KT <= kv_lim)) {  // a tile that reaches beyond what some row may see
#pragma unroll
        for (int ch = 0; ch < NCH; ++ch)
#pragma unroll
          for (int c = 0; c < 32; ++c)
            if (j0 + ch * 32 + c >= kv_lim) s[ch][c] = -INFINITY;
      }
      float mx4[4] = {-INFINITY, -INFINITY, -INFINITY, -INFINITY};  // four chains instead of one of KT maxima
#pragma unroll
      for (int ch = 0; ch < NCH; ++ch)
#pragma unroll
        for (int c = 0; c < 32; ++c) mx4[c & 3] = fmaxf(mx4[c & 3], s[ch][c]);
      const float mx = fmaxf(fmaxf(mx4[0], mx4[1]), fmaxf(mx4[2], mx4[3])) * p.scale_log2;
      const bool move = mx > m_run + TM_SLACK_LOG2;  // also the first tile with a visible key (m_run = -inf)
      const bool resc = move && m_run != -INFINITY;  // there is something to rescale
      if (i > 0 && __any_sync(0xffffffffu, resc)) {
        // O holds the sum over the tiles before this one: all of those products must have landed
        alive = ptx::mbar_wait(o_full, static_cast<uint32_t>(i - 1) & 1u, abort_flag, p.error_word);
        if (!alive) break;
        ptx::tc_fence_after();
        const float f = resc ? exp2f(m_run - mx) : 1.f;
#pragma unroll
        for (int c4 = 0; c4 < 4; ++c4) {
          float o[32];
          ptx::tmem_ld_32x32(t_o + c4 * 32, o);
          ptx::tmem_ld_wait();
#pragma unroll
          for (int c = 0; c < 32; ++c) o[c] *= f;
          ptx::tmem_st_32x32(t_o + c4 * 32, o);
        }
      }
      if (move) {
        if (resc) l_run *= exp2f(m_run - mx);
        m_run = mx;
      }
      const float nbase = m_run == -INFINITY ? 0.f : -m_run;  // no key seen yet: exponentials against 0 give 0, not NaN
      // ---- P = exp2(S * scale - m) as bf16, two keys per column, over the first KT / 2 columns of S_i
      float sum4[4] = {0.f, 0.f, 0.f, 0.f};
#pragma unroll
      for (int h = 0; h < NCH / 2; ++h) {  // 64 keys = 32 columns of P per store
        uint32_t v[32];
#pragma unroll
        for (int j = 0; j < 32; ++j) {
          const float p0 = ptx::ex2_approx(fmaf(s[h * 2 + (j >> 4)][(j & 15) * 2], p.scale_log2, nbase));
          const float p1 = ptx::ex2_approx(fmaf(s[h * 2 + (j >> 4)][(j & 15) * 2 + 1], p.scale_log2, nbase));
          sum4[j & 3] += p0 + p1;
          v[j] = pack_bf16(p0, p1);
        }
        ptx::tmem_st_32x32(t_s + h * 32, *reinterpret_cast<const float(*)[32]>(v));
      }
      l_run += (sum4[0] + sum4[1]) + (sum4[2] + sum4[3]);
      alive = seen_o();
      ptx::tmem_st_wait();
      ptx::tc_fence_before();
      ptx::mbar_arrive(&p_full[i % SBUF]);
    }
    // ---- the row of O, once every product has landed
    if (alive && n_my > 0) {
      alive = ptx::mbar_wait(o_full, static_cast<uint32_t>(n_my - 1) & 1u, abort_flag, p.error_word);
      ptx::tc_fence_after();
    }
    if (alive && n_my > 0 && warp_rows) {
#pragma unroll
      for (int c4 = 0; c4 < 4; ++c4) ptx::tmem_ld_32x32(t_o + c4 * 32, *reinterpret_cast<float(*)[32]>(acc + c4 * 32));
      ptx::tmem_ld_wait();
    } else {
#pragma unroll
      for (int d = 0; d < 128; ++d) acc[d] = 0.f;
    }
  }

  // ------------------------------------------------------------------ output
  auto out_ptr = [&](int prow) -> __nv_bfloat16* {
    const int hg = prow / rps, r = prow % rps;
    return p.out + (static_cast<size_t>(b) * rps + r) * p.hq * 128 + (g * group + hg) * 128;
  };
  if (p.n_splits == 1) {
    if (alive && row_ok) {
      const float inv = 1.0f / l_run;
      __nv_bfloat16* o = out_ptr(pr);
#pragma unroll
      for (int d = 0; d < 128; d += 8)
        *reinterpret_cast<uint4*>(o + d) =
            make_uint4(pack_bf16(acc[d] * inv, acc[d + 1] * inv), pack_bf16(acc[d + 2] * inv, acc[d + 3] * inv),
                       pack_bf16(acc[d + 4] * inv, acc[d + 5] * inv), pack_bf16(acc[d + 6] * inv, acc[d + 7] * inv));
    }
  } else {
    // Partials [128][PART_LD] over the ring (every load into it has been consumed once the last O is read), merged
    // over the key splits: every CTA of the cluster takes a slice of the rows.
    float* red = reinterpret_cast<float*>(smem);
    if (warp_id < 4) {
      float* rr = red + static_cast<size_t>(tid) * PART_LD;
#pragma unroll
      for (int d = 0; d < 128; d += 4) *reinterpret_cast<float4*>(rr + d) = make_float4(acc[d], acc[d + 1], acc[d + 2], acc[d + 3]);
      rr[128] = m_run;  // a split without keys leaves m = -inf, l = 0
      rr[129] = l_run;
    }
    __syncwarp();
    ptx::cluster_sync_all();
    if (warp_id < 4) {
      const int S = p.n_splits;
      const int rank = static_cast<int>(ptx::cluster_ctarank());
      const int rpr = (BM + S - 1) / S;
      const int row0 = rank * rpr, row1 = min(BM, row0 + rpr);
      const uint32_t red_addr = ptx::smem_u32(red);
      for (int e = tid; e < (row1 - row0) * 32; e += 128) {
        const int row = row0 + (e >> 5), c4 = (e & 31) * 4;
        const int prow = qt * BM + row;
        if (prow >= R || (prow % rps) >= n_valid) continue;
        const uint32_t off = static_cast<uint32_t>(row * PART_LD) * 4u;
        float ms[8], ls[8];
        float4 vs[8];
        float M = -INFINITY;
#pragma unroll
        for (int s2 = 0; s2 < 8; ++s2) {
          if (s2 < S) {
            const uint32_t a = ptx::map_to_cta(red_addr + off, static_cast<uint32_t>(s2));
            ms[s2] = ptx::ld_cluster_f(a + 128 * 4);
            ls[s2] = ptx::ld_cluster_f(a + 129 * 4);
            vs[s2] = ptx::ld_cluster_f4(a + c4 * 4);
            M = fmaxf(M, ms[s2]);
          }
        }
        float Lsum = 0.f, a0 = 0.f, a1 = 0.f, a2 = 0.f, a3 = 0.f;
#pragma unroll
        for (int s2 = 0; s2 < 8; ++s2) {  // splits in index order: fixed order of the sums
          if (s2 < S && ls[s2] != 0.f) {
            const float w = exp2f(ms[s2] - M);
            Lsum += w * ls[s2];
            a0 += w * vs[s2].x; a1 += w * vs[s2].y; a2 += w * vs[s2].z; a3 += w * vs[s2].w;
          }
        }
        const float inv = 1.0f / Lsum;
        *reinterpret_cast<uint2*>(out_ptr(prow) + c4) = make_uint2(pack_bf16(a0 * inv, a1 * inv), pack_bf16(a2 * inv, a3 * inv));
      }
    }
    __syncwarp();
    ptx::cluster_sync_all();  // no CTA may leave while a peer still reads its partial
  }
  ptx::tc_fence_before();
  __syncthreads();
  if (warp_id == 5) ptx::tmem_dealloc<L::COLS>(tmem_base);
}

static_assert(TmLayout<64, 2>::OFF_BAR >= 128 * PART_LD * 4, "the partials of the key splits overlay Q and the ring");


// ----------------------------------------------------------------------------- persistent form
// The same tile pipeline for decode-sized batches: all packed rows of a (sequence, kv head) pair fit one 128-row
// tile, a pair's keys take a few tiles only, and there are several pairs per SM.  A CTA per pair pays its fixed cost
// (tensor-memory allocation, Q, first loads, pipeline fill, output: about 7 us against 1.1 us per 64-key tile) once
// per pair, which at 32 rows x 350 keys is most of its life.  Here one CTA per SM walks through its pairs (pair
// blockIdx.x, blockIdx.x + gridDim.x, ...) and treats their key tiles as one stream: the producer runs ahead across
// pair borders (K/V ring, and the next pair's Q by TMA into the second Q buffer), the MMA thread issues the first
// products of the next pair while the softmax threads read out O of the pair before, and nothing is set up twice.
// 128-key tiles, two S buffers, Q in shared memory (two buffers of two K-major slabs), five ring stages.
// (A tile row is a tensor-memory lane and a lane quadrant belongs to one scheduler partition, so 32 live rows use a
// quarter of the SM's exponential rate: about 2200 clocks per 128-key tile on the one warp, against 2750 for the
// tile's 64 KB at an SM's share of HBM.  A form with 2 or 4 copies of the rows in the tile, each copy taking a part
// of every tile's keys, with one reference per row agreed through shared memory and the copies' parts of O added
// there after the pair's last tile, was built and passed the same tests, but was slower (77-79 and 98-103 us per
// layer against 72-73 and 92-93): a barrier per tile and eight per pair cost more than the exponentials saved.)
// Shared memory: two Q buffers of two whole 128-row slabs each (64 KB), five 32 KB ring stages, the barriers.
// (Q buffers cut down to the rows a pair has, so that the 128-row A operand reads on into the other buffer and the
// ring, made room for a sixth stage and cost 10 % of the kernel's speed; a fifth stage over four gained nothing.)
struct TmStream {
  static constexpr int KT = 128, MAX_STAGES = 5;
  static constexpr uint32_t SLAB = 128u * 128u, TILE = 2u * SLAB;
  static constexpr uint32_t COL_S = 0, COL_O = 256;
  static __host__ __device__ uint32_t q_slab(int) { return SLAB; }
  static __host__ __device__ uint32_t off_ring(int R) { return 4u * q_slab(R); }
  static __host__ __device__ int stages(int) { return MAX_STAGES; }
  static __host__ __device__ uint32_t off_bar(int R) { return off_ring(R) + static_cast<uint32_t>(stages(R)) * TILE; }
  static size_t smem_bytes(int R) { return 1024 + off_bar(R) + (2 * MAX_STAGES + 9) * 8 + 64; }
};

// Position in the stream of key tiles of this CTA's pairs: pairs without live rows or keys are passed over.
struct TmCursor {
  int w;    // pair index (sequence * hkv + kv head); >= pairs: the stream has ended
  int j;    // tile of the pair
  int n_t;  // tiles of the pair
  int qi;   // ordinal of the pair among those this CTA works on
  int g;    // ordinal of the tile in the stream
};
__device__ __forceinline__ int tm_pair_tiles(const AttnTcParams& p, int w) {
  const int b = w / p.hkv;
  const int kv = p.rm.kv_len[b];
  return (p.rm.n_valid[b] > 0 && kv > 0) ? (kv + TmStream::KT - 1) / TmStream::KT : 0;
}
__device__ __forceinline__ void tm_cursor_seek(const AttnTcParams& p, int pairs, TmCursor& c) {  // to the first pair with tiles, from c.w on
  while (c.w < pairs && (c.n_t = tm_pair_tiles(p, c.w)) == 0) c.w += gridDim.x;
  c.j = 0;
}
__device__ __forceinline__ void tm_cursor_next(const AttnTcParams& p, int pairs, TmCursor& c) {
  ++c.g;
  if (++c.j < c.n_t) return;
  c.w += gridDim.x;
  ++c.qi;
  tm_cursor_seek(p, pairs, c);
}

// grid (min(SMs, pairs)); needs group * rows_per_seq <= 128.  tmap_q: Q as [bs * rows_per_seq, hq * 128] with boxes of
// rows_per_seq rows x 64 columns (128-byte swizzle).
__global__ void __launch_bounds__(TM_THREADS, 1) attn_tmem_stream_kernel(const __grid_constant__ CUtensorMap tmap_kv,
                                                                         const __grid_constant__ CUtensorMap tmap_q,
                                                                         const AttnTcParams p) {
  using L = TmStream;
  constexpr int KT = L::KT, NCH = KT / 32;
  extern __shared__ uint8_t smem_raw[];
  uint8_t* smem = reinterpret_cast<uint8_t*>((reinterpret_cast<uintptr_t>(smem_raw) + 1023) & ~uintptr_t(1023));
  const int warp_id = threadIdx.x >> 5, lane = threadIdx.x & 31;
  const int group = p.hq / p.hkv;
  const int rps = p.rm.rows_per_seq;
  const int R = group * rps;
  const int pairs = p.rm.bs * p.hkv;
  const int n_stages = L::stages(R);
  const uint32_t q_slab = L::q_slab(R), off_ring = L::off_ring(R);
  uint64_t* kv_full = reinterpret_cast<uint64_t*>(smem + L::off_bar(R));
  uint64_t* kv_empty = kv_full + L::MAX_STAGES;
  uint64_t* s_full = kv_empty + L::MAX_STAGES;  // [2]
  uint64_t* p_full = s_full + 2;            // [2]
  uint64_t* q_full = p_full + 2;            // [2] Q of a pair in its buffer
  uint64_t* q_empty = q_full + 2;           // [2] the pair's last first product has read it
  uint64_t* o_full = q_empty + 2;
  uint32_t* tmem_slot = reinterpret_cast<uint32_t*>(o_full + 1);
  volatile int* abort_flag = reinterpret_cast<volatile int*>(tmem_slot + 1);


  if (threadIdx.x == 0) {
    ptx::prefetch_tensormap(&tmap_kv);
    ptx::prefetch_tensormap(&tmap_q);
    for (int s = 0; s < n_stages; ++s) {
      ptx::mbar_init(&kv_full[s], 1);
      ptx::mbar_init(&kv_empty[s], 1);
    }
    for (int s = 0; s < 2; ++s) {
      ptx::mbar_init(&s_full[s], 1);
      ptx::mbar_init(&p_full[s], 128);
      ptx::mbar_init(&q_full[s], 1);
      ptx::mbar_init(&q_empty[s], 1);
    }
    ptx::mbar_init(o_full, 1);
    *abort_flag = 0;
    ptx::fence_barrier_init();
  }
  if (warp_id == 5) {
    ptx::tmem_alloc<512>(tmem_slot);
    ptx::tmem_relinquish();
  }
  ptx::tc_fence_before();
  __syncthreads();
  ptx::tc_fence_after();
  const uint32_t tmem_base = *tmem_slot;
  ptx::grid_dep_launch();
  const uint32_t sbase = ptx::smem_u32(smem);

  // The row map was written before this forward's first kernel started and cache rows below pos_base are not
  // touched by this forward: both may be read before the dependency wait.
  TmCursor c0{static_cast<int>(blockIdx.x), 0, 0, 0, 0};
  tm_cursor_seek(p, pairs, c0);

  // Producer and MMA thread walk the stream in the same order: K(0), K(1), then V(g), K(g + 2) for every tile g.
  if (warp_id == 4) {
    // ------------------------------------------------------------------ producer
    if (lane == 0) {
      bool waited = false, ok = true;
      int s = 0;  // position in the ring
      auto load = [&](bool is_k, const TmCursor& c) {
        const int stage = s % n_stages;
        if (s >= n_stages &&
            !ptx::mbar_wait(&kv_empty[stage], static_cast<uint32_t>(s / n_stages - 1) & 1u, abort_flag, p.error_word))
          return false;
        const int b = c.w / p.hkv, g = c.w % p.hkv;
        const int j0 = c.j * KT;
        if (!waited && j0 + KT > p.rm.pos_base[b]) {  // this tile holds rows the QKV kernel of this layer writes
          ptx::grid_dep_wait();
          waited = true;
        }
        uint8_t* dst = smem + off_ring + stage * L::TILE;
        const long long plane = (static_cast<long long>(b) * p.hkv + g) * p.max_seq;
        const int row = static_cast<int>((is_k ? p.k_row0 : p.v_row0) + plane + j0);
        ptx::mbar_arrive_expect_tx(&kv_full[stage], L::TILE);
        ptx::tma_load_2d(dst, &tmap_kv, &kv_full[stage], 0, row);
        ptx::tma_load_2d(dst + L::SLAB, &tmap_kv, &kv_full[stage], 64, row);
        ++s;
        if (is_k && c.j == 0) {  // the pair's Q follows its first K tile
          if (!waited) {
            ptx::grid_dep_wait();
            waited = true;
          }
          const int qb = c.qi & 1;
          if (c.qi >= 2 && !ptx::mbar_wait(&q_empty[qb], static_cast<uint32_t>((c.qi >> 1) - 1) & 1u, abort_flag, p.error_word))
            return false;
          uint8_t* qd = smem + qb * 2 * q_slab;
          ptx::mbar_arrive_expect_tx(&q_full[qb], static_cast<uint32_t>(R) * 256u);
          for (int hg = 0; hg < group; ++hg)
            for (int h = 0; h < 2; ++h)
              ptx::tma_load_2d(qd + h * q_slab + hg * rps * 128, &tmap_q, &q_full[qb], (g * group + hg) * 128 + h * 64, b * rps);
        }
        return true;
      };
      TmCursor ck = c0, cv = c0;
      for (int i = 0; i < 2 && ok && ck.w < pairs; ++i) {
        ok = load(true, ck);
        tm_cursor_next(p, pairs, ck);
      }
      while (ok && cv.w < pairs) {
        ok = load(false, cv);
        tm_cursor_next(p, pairs, cv);
        if (ok && ck.w < pairs) {
          ok = load(true, ck);
          tm_cursor_next(p, pairs, ck);
        }
      }
      if (!waited) ptx::grid_dep_wait();
    }
  } else if (warp_id == 5) {
    // ------------------------------------------------------------------ MMA issue
    if (lane == 0) {
      constexpr uint32_t idesc_qk = tm_idesc(128, KT, false);
      constexpr uint32_t idesc_pv = tm_idesc(128, 128, true);
      bool ok = true;
      int s = 0;
      auto stage_ready = [&](uint32_t& addr) {
        const int stage = s % n_stages;
        if (!ptx::mbar_wait(&kv_full[stage], static_cast<uint32_t>(s / n_stages) & 1u, abort_flag, p.error_word)) return -1;
        addr = sbase + off_ring + stage * L::TILE;
        ++s;
        return stage;
      };
      auto qk = [&](const TmCursor& c) {  // S of tile c.g into S buffer c.g & 1
        uint32_t kb;
        const int stage = stage_ready(kb);
        if (stage < 0) return false;
        const int qb = c.qi & 1;
        if (c.j == 0 && !ptx::mbar_wait(&q_full[qb], static_cast<uint32_t>(c.qi >> 1) & 1u, abort_flag, p.error_word)) return false;
        ptx::tc_fence_after();
        const uint32_t qa = sbase + qb * 2 * q_slab;
        const uint32_t sd = tmem_base + L::COL_S + static_cast<uint32_t>((c.g & 1) * KT);
#pragma unroll
        for (int kk = 0; kk < 8; ++kk)
          ptx::umma_bf16(sd, tm_desc_k(qa + (kk >> 2) * q_slab) + static_cast<uint64_t>(2 * (kk & 3)),
                         tm_desc_k(kb + (kk >> 2) * L::SLAB) + static_cast<uint64_t>(2 * (kk & 3)), idesc_qk, kk > 0 ? 1u : 0u);
        ptx::umma_commit(&kv_empty[stage]);
        ptx::umma_commit(&s_full[c.g & 1]);
        if (c.j == c.n_t - 1) ptx::umma_commit(&q_empty[qb]);
        return true;
      };
      TmCursor ck = c0, cv = c0;
      for (int i = 0; i < 2 && ok && ck.w < pairs; ++i) {
        ok = qk(ck);
        tm_cursor_next(p, pairs, ck);
      }
      while (ok && cv.w < pairs) {
        ok = ptx::mbar_wait(&p_full[cv.g & 1], static_cast<uint32_t>(cv.g >> 1) & 1u, abort_flag, p.error_word);
        if (!ok) break;
        uint32_t vb;
        const int stage = stage_ready(vb);
        if (stage < 0) break;
        ptx::tc_fence_after();
        const uint32_t pcol = tmem_base + L::COL_S + static_cast<uint32_t>((cv.g & 1) * KT);  // P lies over its S
#pragma unroll
        for (int kk = 0; kk < KT / 16; ++kk)
          ptx::umma_bf16_ts(tmem_base + L::COL_O, pcol + kk * 8, tm_desc_mn(vb + kk * 2048, L::SLAB, 1024), idesc_pv,
                            (cv.j > 0 || kk > 0) ? 1u : 0u);
        ptx::umma_commit(&kv_empty[stage]);
        ptx::umma_commit(o_full);
        tm_cursor_next(p, pairs, cv);
        if (ck.w < pairs) {  // overwrites the S / P buffer of the tile just multiplied: issued after that product
          ok = qk(ck);
          tm_cursor_next(p, pairs, ck);
        }
      }
    }
  } else {
    // ------------------------------------------------------------------ softmax warps
    const int tid = threadIdx.x;  // row of the tile, tensor-memory lane, packed row head_in_group * rows_per_seq + r
    const uint32_t t_lane = tmem_base + (static_cast<uint32_t>(warp_id * 32) << 16);
    const uint32_t t_o = t_lane + L::COL_O;
    const int r_seq = tid % rps, hg = tid / rps;
    bool alive = true;
    ptx::grid_dep_wait();
    for (TmCursor c = c0; c.w < pairs && alive;) {
      const int b = c.w / p.hkv, g = c.w % p.hkv;
      const int n_valid = p.rm.n_valid[b], kv_len = p.rm.kv_len[b];
      const bool row_ok = tid < R && r_seq < n_valid;
      const bool warp_rows = __any_sync(0xffffffffu, row_ok);
      const int kv_lim = row_ok ? row_kv_limit(p.rm, b, r_seq, kv_len) : kv_len;
      const int n_t = c.n_t;
      float m_run = -INFINITY, l_run = 0.f;  // m_run: the reference of the exponentials (see the head of the file)
      for (int j = 0; j < n_t && alive; ++j, tm_cursor_next(p, pairs, c)) {
        const int gt = c.g;
        alive = ptx::mbar_wait(&s_full[gt & 1], static_cast<uint32_t>(gt >> 1) & 1u, abort_flag, p.error_word);
        if (!alive) break;
        // every thread watches every phase of o_full in order (a parity wait cannot tell a phase from the one two before)
        auto seen_o = [&]() { return gt == 0 || ptx::mbar_wait(o_full, static_cast<uint32_t>(gt - 1) & 1u, abort_flag, p.error_word); };
        if (!warp_rows) {
          alive = seen_o();
          ptx::mbar_arrive(&p_full[gt & 1]);
          continue;
        }
        ptx::tc_fence_after();
        const int j0 = j * KT;
        const uint32_t t_s = t_lane + L::COL_S + static_cast<uint32_t>((gt & 1) * KT);
        float s[NCH][32];
#pragma unroll
        for (int ch = 0; ch < NCH; ++ch) ptx::tmem_ld_32x32(t_s + ch * 32, s[ch]);
        ptx::tmem_ld_wait();
        if (!__all_sync(0xffffffffu, j0 + KT <= kv_lim)) {
#pragma unroll
          for (int ch = 0; ch < NCH; ++ch)
#pragma unroll
            for (int cc = 0; cc < 32; ++cc)
              if (j0 + ch * 32 + cc >= kv_lim) s[ch][cc] = -INFINITY;
        }
        float mx4[4] = {-INFINITY, -INFINITY, -INFINITY, -INFINITY};
#pragma unroll
        for (int ch = 0; ch < NCH; ++ch)
#pragma unroll
          for (int cc = 0; cc < 32; ++cc) mx4[cc & 3] = fmaxf(mx4[cc & 3], s[ch][cc]);
        const float mx = fmaxf(fmaxf(mx4[0], mx4[1]), fmaxf(mx4[2], mx4[3])) * p.scale_log2;
        const bool move = mx > m_run + TM_SLACK_LOG2;
        const bool resc = move && m_run != -INFINITY;
        if (j > 0 && __any_sync(0xffffffffu, resc)) {
          alive = seen_o();  // O holds the sum over the pair's tiles before this one
          if (!alive) break;
          ptx::tc_fence_after();
          const float f = resc ? exp2f(m_run - mx) : 1.f;
#pragma unroll
          for (int c4 = 0; c4 < 4; ++c4) {
            float o[32];
            ptx::tmem_ld_32x32(t_o + c4 * 32, o);
            ptx::tmem_ld_wait();
#pragma unroll
            for (int cc = 0; cc < 32; ++cc) o[cc] *= f;
            ptx::tmem_st_32x32(t_o + c4 * 32, o);
          }
        }
        if (move) {
          if (resc) l_run *= exp2f(m_run - mx);
          m_run = mx;
        }
        const float nbase = m_run == -INFINITY ? 0.f : -m_run;
        float sum4[4] = {0.f, 0.f, 0.f, 0.f};
#pragma unroll
        for (int h = 0; h < NCH / 2; ++h) {
          uint32_t v[32];
#pragma unroll
          for (int jj = 0; jj < 32; ++jj) {
            const float p0 = ptx::ex2_approx(fmaf(s[h * 2 + (jj >> 4)][(jj & 15) * 2], p.scale_log2, nbase));
            const float p1 = ptx::ex2_approx(fmaf(s[h * 2 + (jj >> 4)][(jj & 15) * 2 + 1], p.scale_log2, nbase));
            sum4[jj & 3] += p0 + p1;
            v[jj] = pack_bf16(p0, p1);
          }
          ptx::tmem_st_32x32(t_s + h * 32, *reinterpret_cast<const float(*)[32]>(v));
        }
        l_run += (sum4[0] + sum4[1]) + (sum4[2] + sum4[3]);
        alive = seen_o();
        ptx::tmem_st_wait();
        ptx::tc_fence_before();
        ptx::mbar_arrive(&p_full[gt & 1]);
      }
      if (!alive) break;
      // ---- the pair's rows of O (c now stands on the first tile of the next pair: the last tile was c.g - 1)
      alive = ptx::mbar_wait(o_full, static_cast<uint32_t>(c.g - 1) & 1u, abort_flag, p.error_word);
      if (!alive) break;
      if (warp_rows) {
        ptx::tc_fence_after();
        float acc[128];
#pragma unroll
        for (int c4 = 0; c4 < 4; ++c4) ptx::tmem_ld_32x32(t_o + c4 * 32, *reinterpret_cast<float(*)[32]>(acc + c4 * 32));
        ptx::tmem_ld_wait();
        ptx::tc_fence_before();  // the next pair's first P (and with it the product that overwrites O) comes after this
        if (row_ok) {
          const float inv = 1.0f / l_run;
          __nv_bfloat16* o = p.out + (static_cast<size_t>(b) * rps + r_seq) * p.hq * 128 + (g * group + hg) * 128;
#pragma unroll
          for (int d = 0; d < 128; d += 8)
            *reinterpret_cast<uint4*>(o + d) =
                make_uint4(pack_bf16(acc[d] * inv, acc[d + 1] * inv), pack_bf16(acc[d + 2] * inv, acc[d + 3] * inv),
                           pack_bf16(acc[d + 4] * inv, acc[d + 5] * inv), pack_bf16(acc[d + 6] * inv, acc[d + 7] * inv));
        }
      }
    }
  }
  __syncwarp();
  ptx::tc_fence_before();
  __syncthreads();
  if (warp_id == 5) ptx::tmem_dealloc<512>(tmem_base);
}

}  // namespace attn
}  // namespace d3

// Skinny decode matmuls (up to 64 rows) run as a chain: one persistent launch executes up to four
// matmuls that depend on one another -- attention output projection -> gate/up -> down -> the next
// layer's QKV -- so that weights keep streaming from HBM across the borders between them.
//
// Why.  At 32 rows every matmul of a layer is bound by weight streaming, and as separate kernels each
// of them pays, after its last weight byte has arrived, an epilogue, a kernel boundary and the first
// activation load of its successor before HBM is busy again.  Here the CTAs stay, and the thread that
// requests weights never waits for data: it walks through the CTA's share of all matmuls of the chain
// and is held back by ring space only.  While a border's dependency resolves (epilogue, reduction,
// grid-wide counter, activation load) the ring fills with the next matmul's weights.
//
// Grid: clusters of CHAIN_C = 4 CTAs, one CTA per SM, all resident at once (the host sizes the grid
// from the occupancy of clusters).  Two ways of cutting a matmul Y[M,N] = X[M,K] . W[N,K]^T:
//   * CHAIN_STRIP (QKV, gate/up: many columns): CTA i owns the column strip of units
//     [U i / n, U (i+1) / n) of 16 columns over the whole K range; the accumulator goes straight from
//     tensor memory to the epilogue (RoPE + cache write, SwiGLU).  No reduction.
//   * CHAIN_KSPLIT (O-proj, down: few columns, long K; QKV: so that a CTA does not re-read all of X
//     for a narrow strip): ks = 4 or 2 CTAs of a cluster share a strip of 32-column units and take a
//     ks-th of K each; the partial sums meet in distributed shared memory: a strip is cut into units of
//     16 rows x 32 columns, unit u belongs to the group's CTA u mod ks, every CTA pushes its partial of
//     each unit into the owner's receive buffer (remote stores) and arrives on the owner's barrier; the
//     owner adds the partials in rank order (fixed order: reproducible bits) with one (row, 4 columns)
//     element per thread and runs the epilogue (residual update, or RoPE + cache write).
// Weights come in the tiled form (contiguous pre-swizzled 128 x 64 blocks): a strip's rows are runs of
// whole 8-row swizzle groups inside the blocks it touches, copied with one bulk copy per block.
//
// Borders.  Matmul j+1 reads what matmul j wrote on other SMs, so each border is a grid-wide counter
// in global memory: a CTA adds one (release) after its last store of matmul j; the thread that loads
// activations and one epilogue thread wait for the count (acquire, bounded spin) before they touch
// matmul j+1's inputs.  Matmul 0 waits for the kernels before this launch (griddepcontrol.wait).
//
// Warp roles: 0 weights, 1 MMA issue + tensor-memory owner, 2-5 epilogue, 6 activations.
#pragma once
#include <cuda.h>

#include "common.cuh"
#include "gemm_tc.cuh"
#include "ptx_sm100.cuh"

namespace d3 {
namespace tc {

constexpr int CHAIN_MAX_OPS = 4;
constexpr int CHAIN_THREADS = 224;
constexpr int CHAIN_C = 4;
enum : int { CHAIN_STRIP = 0, CHAIN_KSPLIT = 1 };

struct ChainOp {
  int kind;   // CHAIN_STRIP / CHAIN_KSPLIT
  int epi;    // CHAIN_STRIP: EPI_QKV or EPI_SWIGLU; CHAIN_KSPLIT: EPI_RESID or EPI_QKV
  int ks;     // CHAIN_KSPLIT: CTAs of a cluster that share a column strip and split K among them (1, 2 or 4);
              // the cluster then holds 4 / ks strips side by side
  int N, K;
  int x_map;  // which of the launch's activation tensor maps this matmul reads
  const __nv_bfloat16* w;  // tiled weights
  EpiParams ep;
};

struct ChainParams {
  int n_ops;
  ChainOp op[CHAIN_MAX_OPS];
  int M;
  int a_rows;              // rows of the X box: 32 or 64
  int stages;              // ring depth
  uint32_t w_stage_bytes;  // weight part of a stage: the widest strip of the chain x 128 bytes
  unsigned int* sync;      // [CHAIN_MAX_OPS] border counters of this launch, zero on entry
  uint32_t* error_word;
  const int* skip_flag;
  // EPI_QKV
  const float* rope_cos;
  const float* rope_sin;
  const int* pos_base;
  const int* n_valid;
  int rows_per_seq;
  int n_q_heads, n_kv_heads, max_seq;
  __nv_bfloat16* k_cache;
  __nv_bfloat16* v_cache;
};

// This CTA's share of one matmul of the chain.
struct ChainShare {
  int c0, S;     // column strip [c0, c0 + S)
  int k0, n_k;   // K slabs [k0, k0 + n_k)
};
__device__ __forceinline__ ChainShare chain_share(const ChainOp& o, int cta, int n_cta, int cluster, int n_clusters, int rank) {
  ChainShare s;
  const int KC = (o.K + 63) / 64;
  if (o.kind == CHAIN_STRIP) {
    const int U = o.N / 16;
    const int u0 = static_cast<int>(static_cast<long long>(U) * cta / n_cta);
    const int u1 = static_cast<int>(static_cast<long long>(U) * (cta + 1) / n_cta);
    s.c0 = u0 * 16;
    s.S = (u1 - u0) * 16;
    s.k0 = 0;
    s.n_k = KC;
  } else {
    const int U = o.N / 32;
    const int per = CHAIN_C / o.ks;                   // strips per cluster
    const int g = cluster * per + rank / o.ks, G = n_clusters * per;
    const int kp = rank % o.ks;                       // this CTA's part of K
    const int u0 = static_cast<int>(static_cast<long long>(U) * g / G);
    const int u1 = static_cast<int>(static_cast<long long>(U) * (g + 1) / G);
    s.c0 = u0 * 32;
    s.S = (u1 - u0) * 32;
    s.k0 = KC * kp / o.ks;
    s.n_k = KC * (kp + 1) / o.ks - s.k0;
  }
  if (s.S == 0) s.n_k = 0;
  return s;
}

// Bounded spin until *ptr >= target (acquire at gpu scope).  false: gave up (error word raised) or
// another role of the CTA did.
__device__ __forceinline__ bool chain_wait_count(const unsigned int* ptr, unsigned int target, volatile int* abort_flag,
                                                 uint32_t* error_word) {
  uint64_t t0 = 0;
  for (uint32_t it = 1;; ++it) {
    unsigned int v;
    asm volatile("ld.acquire.gpu.global.u32 %0, [%1];" : "=r"(v) : "l"(ptr) : "memory");
    if (v >= target) return true;
    if ((it & 0xff) == 0) {
      if (*abort_flag) return false;
      const uint64_t now = global_ns();
      if (t0 == 0) t0 = now;
      else if (now - t0 > WAIT_LIMIT_NS) {
        *abort_flag = 1;
        atomicOr(error_word, ERRW_MBAR_TIMEOUT);
        return false;
      }
    }
  }
}
__device__ __forceinline__ void chain_arrive(unsigned int* ptr) {
  asm volatile("red.release.gpu.global.add.u32 [%0], 1;" ::"l"(ptr) : "memory");
}

// Barrier over the 128 epilogue threads that also tells every one of them whether all of them are
// still in order: a thread whose wait gave up must not leave the others at a later barrier.
__device__ __forceinline__ bool epi_all(bool ok) {
  uint32_t r;
  asm volatile(
      "{\n"
      ".reg .pred p, q;\n"
      "setp.ne.u32 q, %1, 0;\n"
      "barrier.red.and.pred p, 1, 128, q;\n"
      "selp.u32 %0, 1, 0, p;\n"
      "}\n"
      : "=r"(r)
      : "r"(static_cast<uint32_t>(ok))
      : "memory");
  return r != 0;
}

// Dynamic shared memory (1024-byte aligned inside the kernel):
//   [stages x a_rows x 128 B] X slabs, [stages x w_stage_bytes] W slabs (at least (128 - a_rows) * 128
//   bytes follow the last X slab: the MMA reads 128 rows of its A operand whatever a_rows is),
//   receive buffer [units per owner][4 sources][16 rows][32 columns] fp32, barriers.
inline size_t chain_recv_bytes(int a_rows, int max_ksplit_cols) {
  // an owner holds ceil(units / ks) units x ks sources x 2 KB: at most (units + ks - 1) x 2 KB, ks <= 4
  const int n_units = (max_ksplit_cols / 32) * (a_rows / 16);
  return static_cast<size_t>(n_units + CHAIN_C - 1) * 2048;
}
inline size_t chain_smem_bytes(int a_rows, uint32_t w_stage_bytes, int stages, int max_ksplit_cols) {
  size_t body = static_cast<size_t>(stages) * (static_cast<size_t>(a_rows) * 128 + w_stage_bytes);
  const size_t reach = static_cast<size_t>(stages - 1) * a_rows * 128 + 128 * 128;
  if (body < reach) body = reach;
  return 1024 + body + chain_recv_bytes(a_rows, max_ksplit_cols) + (2 * stages + 8) * 8 + 64;
}

__global__ void __launch_bounds__(CHAIN_THREADS, 1)
chain_kernel(const __grid_constant__ CUtensorMap tmap_x0, const __grid_constant__ CUtensorMap tmap_x1,
             const __grid_constant__ CUtensorMap tmap_x2, const ChainParams p, const int recv_bytes) {
  if (p.skip_flag != nullptr && *p.skip_flag != 0) return;
  grid_dep_launch();
  extern __shared__ uint8_t smem_raw[];
  uint8_t* smem = reinterpret_cast<uint8_t*>((reinterpret_cast<uintptr_t>(smem_raw) + 1023) & ~uintptr_t(1023));
  const int stages = p.stages;
  const uint32_t a_stage_bytes = static_cast<uint32_t>(p.a_rows) * 128u;
  const uint32_t b_stage_bytes = p.w_stage_bytes;
  uint8_t* smem_a = smem;
  uint8_t* smem_b = smem + static_cast<size_t>(stages) * a_stage_bytes;
  size_t body = static_cast<size_t>(stages) * (a_stage_bytes + b_stage_bytes);
  const size_t reach = static_cast<size_t>(stages - 1) * a_stage_bytes + 128 * 128;
  if (body < reach) body = reach;
  float* recv = reinterpret_cast<float*>(smem + body);
  uint64_t* full_bar = reinterpret_cast<uint64_t*>(smem + body + recv_bytes);
  uint64_t* empty_bar = full_bar + stages;
  uint64_t* acc_full = empty_bar + stages;   // [2]
  uint64_t* acc_empty = acc_full + 2;        // [2]
  uint64_t* ready_bar = acc_empty + 2;       // all four partials of this CTA's units have arrived
  uint32_t* tmem_slot = reinterpret_cast<uint32_t*>(ready_bar + 1);
  volatile int* abort_flag = reinterpret_cast<volatile int*>(tmem_slot + 1);

  const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
  const int cta = blockIdx.x, n_cta = gridDim.x;
  const int rank = static_cast<int>(cluster_ctarank());
  const int cluster = cta / CHAIN_C, n_clusters = n_cta / CHAIN_C;
  // One accumulator of up to 256 columns.  A second one would buy nothing: the MMAs of matmul j+1 need
  // activations that exist only after every CTA has finished the epilogue of matmul j.  And two CTAs
  // of chain launches that share an SM must both get their tensor memory (512 columns per SM): a CTA
  // that waited for the other's columns while the other waits for it at a border would never run.
  constexpr uint32_t TMEM_COLS = 256;

  if (threadIdx.x == 0) {
    prefetch_tensormap(&tmap_x0);
    prefetch_tensormap(&tmap_x1);
    prefetch_tensormap(&tmap_x2);
    for (int s = 0; s < stages; ++s) {
      mbar_init(&full_bar[s], 2);  // the weight thread and the activation thread each announce their own bytes
      mbar_init(&empty_bar[s], 1);
    }
    for (int b = 0; b < 2; ++b) {
      mbar_init(&acc_full[b], 1);
      mbar_init(&acc_empty[b], 128);
    }
    mbar_init(ready_bar, CHAIN_C);
    *abort_flag = 0;
    fence_barrier_init();
  }
  if (warp == 1) {
    tmem_alloc<TMEM_COLS>(tmem_slot);
    tmem_relinquish();
  }
  tc_fence_before();
  __syncthreads();
  cluster_sync_all();  // every CTA's barriers exist before a peer arrives on them
  tc_fence_after();
  const uint32_t tmem_base = *tmem_slot;

  auto x_map_of = [&](int i) -> const CUtensorMap* { return i == 0 ? &tmap_x0 : (i == 1 ? &tmap_x1 : &tmap_x2); };

  if (warp == 0) {
    // ---------------- weights: never waits for data, only for ring space
    if (lane == 0) {
      int s = 0;
      uint32_t ph = 1;  // parity to wait for on the empty barrier (first lap: passes at once)
      bool ok = true;
      for (int j = 0; j < p.n_ops && ok; ++j) {
        const ChainOp& o = p.op[j];
        const ChainShare sh = chain_share(o, cta, n_cta, cluster, n_clusters, rank);
        if (sh.n_k == 0) continue;
        const int KC = (o.K + 63) / 64;
        // the strip's rows inside the 128-row blocks it touches: up to three runs of whole 8-row groups
        const __nv_bfloat16* piece_src[3];
        uint32_t piece_bytes[3], piece_dst[3];
        {
          int row = sh.c0, left = sh.S;
          uint32_t off = 0;
#pragma unroll
          for (int q = 0; q < 3; ++q) {
            const int blk = row >> 7, r0 = row & 127;
            const int n = left < 128 - r0 ? left : 128 - r0;
            piece_src[q] = o.w + (static_cast<long long>(blk) * KC * 128 + r0) * 64;
            piece_bytes[q] = static_cast<uint32_t>(n) * 128u;
            piece_dst[q] = off;
            off += static_cast<uint32_t>(n) * 128u;
            row += n;
            left -= n;
          }
        }
        const uint32_t tx = static_cast<uint32_t>(sh.S) * 128u;
        for (int i = 0; i < sh.n_k; ++i) {
          if (!mbar_wait(&empty_bar[s], ph, abort_flag, p.error_word)) { ok = false; break; }
          mbar_arrive_expect_tx(&full_bar[s], tx);
          uint8_t* dst = smem_b + static_cast<size_t>(s) * b_stage_bytes;
          const size_t slab = static_cast<size_t>(sh.k0 + i) * (128 * 64);
#pragma unroll
          for (int q = 0; q < 3; ++q)
            if (piece_bytes[q] != 0) bulk_load_1d(dst + piece_dst[q], piece_src[q] + slab, piece_bytes[q], &full_bar[s]);
          if (++s == stages) { s = 0; ph ^= 1u; }
        }
      }
    }
  } else if (warp == 6) {
    // ---------------- activations: behind the border of each matmul
    if (lane == 0) {
      int s = 0;
      uint32_t ph = 1;
      bool ok = true;
      grid_dep_wait();
      for (int j = 0; j < p.n_ops && ok; ++j) {
        const ChainOp& o = p.op[j];
        const ChainShare sh = chain_share(o, cta, n_cta, cluster, n_clusters, rank);
        if (j > 0) {
          if (!chain_wait_count(p.sync + (j - 1), static_cast<unsigned int>(n_cta), abort_flag, p.error_word)) break;
          fence_proxy_async_all();  // the rows were written with ordinary stores; the loads below go through the async proxy
        }
        const CUtensorMap* tm = x_map_of(o.x_map);
        for (int i = 0; i < sh.n_k; ++i) {
          // the stage's previous use must be over (the weight thread waits for the same phase)
          if (!mbar_wait(&empty_bar[s], ph, abort_flag, p.error_word)) { ok = false; break; }
          mbar_arrive_expect_tx(&full_bar[s], a_stage_bytes);
          tma_load_2d(smem_a + static_cast<size_t>(s) * a_stage_bytes, tm, &full_bar[s], (sh.k0 + i) * BLOCK_K, 0);
          if (++s == stages) { s = 0; ph ^= 1u; }
        }
      }
    }
  } else if (warp == 1) {
    // ---------------- MMA issue
    if (lane == 0) {
      const uint64_t adesc0 = make_smem_desc(smem_u32(smem_a)), bdesc0 = make_smem_desc(smem_u32(smem_b));
      const uint64_t a_step = a_stage_bytes >> 4, b_step = b_stage_bytes >> 4;
      int s = 0;
      uint32_t ph = 0;
      int n_acc = 0;  // accumulators produced so far
      bool ok = true;
      for (int j = 0; j < p.n_ops && ok; ++j) {
        const ChainShare sh = chain_share(p.op[j], cta, n_cta, cluster, n_clusters, rank);
        if (sh.n_k == 0) continue;
        // the epilogue of the matmul before this one has drained the accumulator
        if (!mbar_wait(&acc_empty[0], (static_cast<uint32_t>(n_acc) & 1u) ^ 1u, abort_flag, p.error_word)) break;
        tc_fence_after();
        const uint32_t idesc = make_idesc(BLOCK_M, sh.S);
        const uint32_t tmem_d = tmem_base;
        for (int i = 0; i < sh.n_k; ++i) {
          if (!mbar_wait(&full_bar[s], ph, abort_flag, p.error_word)) { ok = false; break; }
          tc_fence_after();
          const uint64_t adesc = adesc0 + a_step * static_cast<uint64_t>(s), bdesc = bdesc0 + b_step * static_cast<uint64_t>(s);
#pragma unroll
          for (int kk = 0; kk < BLOCK_K / UMMA_K; ++kk)
            umma_bf16(tmem_d, adesc + static_cast<uint64_t>(2 * kk), bdesc + static_cast<uint64_t>(2 * kk), idesc,
                      (i > 0 || kk > 0) ? 1u : 0u);
          umma_commit(&empty_bar[s]);
          if (++s == stages) { s = 0; ph ^= 1u; }
        }
        if (ok) umma_commit(&acc_full[0]);
        ++n_acc;
      }
    }
  } else if (warp >= 2 && warp <= 5) {
    // ---------------- epilogue warps: TMEM lane group = warp % 4
    grid_dep_wait();
    const int lg = warp & 3;
    const int row = lg * 32 + lane;
    const int et = threadIdx.x - 64;  // 0..127
    const bool warp_live = lg * 32 < p.a_rows && lg * 32 < p.M;
    const uint32_t recv_addr = smem_u32(recv);
    const int RS = p.a_rows / 16;
    const int e_j = et & 7, e_row = et >> 3;
    int n_acc = 0, n_ks = 0;
    bool alive = true;
    for (int j = 0; j < p.n_ops && alive; ++j) {
      const ChainOp& o = p.op[j];
      const ChainShare sh = chain_share(o, cta, n_cta, cluster, n_clusters, rank);
      if (j > 0) {  // rows, chunk sums and residual values written by the matmul before this one, on any SM
        bool ok = true;
        if (et == 0) ok = chain_wait_count(p.sync + (j - 1), static_cast<unsigned int>(n_cta), abort_flag, p.error_word);
        if (!epi_all(ok)) { alive = false; break; }
      }
      if (sh.n_k > 0) {
        constexpr int buf = 0;
        const uint32_t acc_par = static_cast<uint32_t>(n_acc) & 1u;
        ++n_acc;
        // the matmul's parameters in the form the shared epilogue code reads
        GemmParams gp{};
        gp.M = p.M; gp.N = o.N; gp.K = o.K;
        gp.a_rows = p.a_rows;
        gp.error_word = p.error_word;
        gp.ep = o.ep;
        gp.rope_cos = p.rope_cos; gp.rope_sin = p.rope_sin; gp.pos_base = p.pos_base; gp.n_valid = p.n_valid;
        gp.rows_per_seq = p.rows_per_seq; gp.n_q_heads = p.n_q_heads; gp.n_kv_heads = p.n_kv_heads; gp.max_seq = p.max_seq;
        gp.k_cache = p.k_cache; gp.v_cache = p.v_cache;
        const uint32_t lane_addr = tmem_base + (static_cast<uint32_t>(lg * 32) << 16);
        if (o.kind == CHAIN_STRIP) {
          const float rs = (warp_live && row < p.M && o.ep.ssq_in != nullptr) ? row_rstd(o.ep, row) : 1.f;
          bool ok = mbar_wait(&acc_full[buf], acc_par, abort_flag, p.error_word);
          if (!epi_all(ok)) { alive = false; break; }
          tc_fence_after();
          if (warp_live) {
            TmemSource tsrc{lane_addr};
            if (o.epi == EPI_QKV) run_epilogue<EPI_QKV, 256>(tsrc, gp, row, sh.c0, row < p.M, 0, 1, sh.c0 + sh.S, rs);
            else run_epilogue<EPI_SWIGLU, 256>(tsrc, gp, row, sh.c0, row < p.M, 0, 1, sh.c0 + sh.S, rs);
          }
          tc_fence_before();
          mbar_arrive(&acc_empty[buf]);
        } else {
          // ---- K-split: push this lane's row of every 32-column chunk to the chunk's owner
          const int ks = o.ks;
          const int gbase = (rank / ks) * ks, kp = rank % ks;  // first CTA of this strip's group, this CTA's K part
          const int n_chunks = sh.S / 32;
          const int n_units = n_chunks * RS;
          const int n_owners = n_units < ks ? n_units : ks;
          const bool owner_here = kp < n_units;
          const uint32_t ready_par = static_cast<uint32_t>(n_ks) & 1u;  // phases of ready_bar advance only when this CTA owns units
          if (owner_here) ++n_ks;
          // what this thread needs besides the sums, in flight while the MMAs still run: the residual
          // values it will update (first PRE units it owns), or the row factors of the folded norm
          // (a thread meets RS <= 4 different rows)
          constexpr int PRE = 4;
          float4 y_pre[PRE];
          float rs_row[4];
#pragma unroll
          for (int q = 0; q < PRE; ++q) {
            y_pre[q] = make_float4(0.f, 0.f, 0.f, 0.f);
            const int u = kp + q * ks;
            if (o.epi == EPI_RESID && owner_here && u < n_units) {
              const int c = u / RS, m = (u % RS) * 16 + e_row, n = sh.c0 + c * 32 + e_j * 4;
              if (m < p.M) y_pre[q] = *reinterpret_cast<const float4*>(static_cast<const float*>(o.ep.y) + static_cast<size_t>(m) * o.ep.ldy + n);
            }
          }
          int pos_row[4];  // EPI_QKV: cache slot of the row, -1 when the row is padding
#pragma unroll
          for (int q = 0; q < 4; ++q) {
            rs_row[q] = 1.f;
            pos_row[q] = -1;
            const int m = q * 16 + e_row;
            if (o.epi != EPI_RESID && owner_here && q < RS && m < p.M) {
              if (o.ep.ssq_in != nullptr) rs_row[q] = row_rstd(o.ep, m);
              if (o.epi == EPI_QKV) {
                const int b = m / p.rows_per_seq, r = m % p.rows_per_seq;
                if (r < p.n_valid[b]) {
                  const int pos = p.pos_base[b] + r;
                  if (pos < 0 || pos >= p.max_seq) atomicOr(p.error_word, ERRW_BAD_POSITION);
                  else pos_row[q] = pos;
                }
              }
            }
          }
          bool ok = mbar_wait(&acc_full[buf], acc_par, abort_flag, p.error_word);
          if (!epi_all(ok)) { alive = false; break; }
          tc_fence_after();
          if (warp_live) {
            TmemSource tsrc{lane_addr};
#pragma unroll 1
            for (int c = 0; c < n_chunks; ++c) {
              float v[32];
              tsrc.load(c * 32, v);
              const int u = c * RS + (row >> 4);
              const int owner = gbase + u % ks, slot = u / ks;
              const uint32_t dst = map_to_cta(recv_addr + static_cast<uint32_t>(((slot * ks + kp) * 16 + (row & 15)) * 128),
                                              static_cast<uint32_t>(owner));
#pragma unroll
              for (int q = 0; q < 8; ++q) st_cluster_f4(dst + q * 16, v[4 * q], v[4 * q + 1], v[4 * q + 2], v[4 * q + 3]);
            }
          }
          tc_fence_before();
          mbar_arrive(&acc_empty[buf]);
          epi_bar_sync();  // every pushing thread's stores are ordered before the arrivals below
          // the barrier counts CHAIN_C arrivals whatever ks is: each of the ks sources arrives CHAIN_C / ks times
          if (et < n_owners * (CHAIN_C / ks)) mbar_arrive_remote(ready_bar, static_cast<uint32_t>(gbase + et % n_owners));
          if (owner_here) {
            ok = mbar_wait_cluster(ready_bar, ready_par, abort_flag, p.error_word);
            if (!epi_all(ok)) { alive = false; break; }
            // RoPE + cache write on (row, 4 columns), four owned units at a time so that their table
            // loads are in flight together.  Packed rows of W inside a q or k head: 2i = dim i,
            // 2i + 1 = dim i + 64 (a RoPE pair); v heads keep their order; q heads, then k, then v.
            for (int slot0 = 0; o.epi == EPI_QKV && kp + slot0 * ks < n_units; slot0 += 4) {
              float2 co[4], si[4];
              int pos4[4];
#pragma unroll
              for (int q = 0; q < 4; ++q) {
                const int u = kp + (slot0 + q) * ks;
                pos4[q] = -1;
                co[q] = make_float2(1.f, 1.f);
                si[q] = make_float2(0.f, 0.f);
                if (u < n_units) {
#pragma unroll
                  for (int t = 0; t < 4; ++t)
                    if (t == u % RS) pos4[q] = pos_row[t];
                  const int n = sh.c0 + (u / RS) * 32 + e_j * 4;
                  if (pos4[q] >= 0 && n / 128 < p.n_q_heads + p.n_kv_heads) {
                    const int i0 = (n % 128) / 2;
                    co[q] = *reinterpret_cast<const float2*>(p.rope_cos + static_cast<size_t>(pos4[q]) * 64 + i0);
                    si[q] = *reinterpret_cast<const float2*>(p.rope_sin + static_cast<size_t>(pos4[q]) * 64 + i0);
                  }
                }
              }
#pragma unroll
              for (int q = 0; q < 4; ++q) {
                const int slot = slot0 + q, u = kp + slot * ks;
                if (u >= n_units || pos4[q] < 0) continue;
                const int m = (u % RS) * 16 + e_row, n = sh.c0 + (u / RS) * 32 + e_j * 4;
                float4 acc = make_float4(0.f, 0.f, 0.f, 0.f);
                const float4* src = reinterpret_cast<const float4*>(recv) + (static_cast<size_t>(slot) * ks * 16 + e_row) * 8 + e_j;
                for (int s2 = 0; s2 < ks; ++s2) {
                  const float4 w4 = src[static_cast<size_t>(s2) * 128];
                  acc.x += w4.x; acc.y += w4.y; acc.z += w4.z; acc.w += w4.w;
                }
                float rs = 1.f;
#pragma unroll
                for (int t = 0; t < 4; ++t)
                  if (t == u % RS) rs = rs_row[t];
                const float a0 = acc.x * rs, a1 = acc.y * rs, a2 = acc.z * rs, a3 = acc.w * rs;
                const int head = n / 128, off = n % 128, pos = pos4[q];
                const int b = m / p.rows_per_seq;
                if (head < p.n_q_heads + p.n_kv_heads) {
                  __nv_bfloat16* dst = head < p.n_q_heads
                      ? static_cast<__nv_bfloat16*>(o.ep.y) + static_cast<size_t>(m) * o.ep.ldy + head * 128
                      : p.k_cache + ((static_cast<size_t>(b) * p.n_kv_heads + (head - p.n_q_heads)) * p.max_seq + pos) * 128;
                  const int i0 = off / 2;  // pairs (i0, i0 + 64) and (i0 + 1, i0 + 65)
                  __nv_bfloat162 lo = __floats2bfloat162_rn(a0 * co[q].x - a1 * si[q].x, a2 * co[q].y - a3 * si[q].y);
                  __nv_bfloat162 hi = __floats2bfloat162_rn(a1 * co[q].x + a0 * si[q].x, a3 * co[q].y + a2 * si[q].y);
                  *reinterpret_cast<uint32_t*>(dst + i0) = *reinterpret_cast<uint32_t*>(&lo);
                  *reinterpret_cast<uint32_t*>(dst + 64 + i0) = *reinterpret_cast<uint32_t*>(&hi);
                } else if (head < p.n_q_heads + 2 * p.n_kv_heads) {
                  __nv_bfloat16* dst = p.v_cache +
                      ((static_cast<size_t>(b) * p.n_kv_heads + (head - p.n_q_heads - p.n_kv_heads)) * p.max_seq + pos) * 128 + off;
                  __nv_bfloat162 lo = __floats2bfloat162_rn(a0, a1), hi = __floats2bfloat162_rn(a2, a3);
                  *reinterpret_cast<uint2*>(dst) = make_uint2(*reinterpret_cast<uint32_t*>(&lo), *reinterpret_cast<uint32_t*>(&hi));
                }
              }
            }
            for (int slot = 0, u = kp; u < n_units && o.epi == EPI_RESID; ++slot, u += ks) {
              const int c = u / RS;
              const int m = (u % RS) * 16 + e_row, n = sh.c0 + c * 32 + e_j * 4;
              float4 acc = make_float4(0.f, 0.f, 0.f, 0.f);
              const float4* src = reinterpret_cast<const float4*>(recv) + (static_cast<size_t>(slot) * ks * 16 + e_row) * 8 + e_j;
              for (int s2 = 0; s2 < ks; ++s2) {
                const float4 w4 = src[static_cast<size_t>(s2) * 128];
                acc.x += w4.x; acc.y += w4.y; acc.z += w4.z; acc.w += w4.w;
              }
              const bool live = m < p.M;
              float* y = static_cast<float*>(o.ep.y) + static_cast<size_t>(m) * o.ep.ldy;
              float sq = 0.f;
              if (live) {
                float4 o0 = make_float4(0.f, 0.f, 0.f, 0.f);
                bool have = false;
#pragma unroll
                for (int q = 0; q < PRE; ++q)
                  if (q == slot) { o0 = y_pre[q]; have = true; }
                if (!have) o0 = *reinterpret_cast<const float4*>(y + n);
                const float4 o4 = make_float4(o0.x + acc.x, o0.y + acc.y, o0.z + acc.z, o0.w + acc.w);
                *reinterpret_cast<float4*>(y + n) = o4;
                sq = ((o4.x * o4.x + o4.y * o4.y) + o4.z * o4.z) + o4.w * o4.w;
                if (o.ep.yb != nullptr) {
                  __nv_bfloat162 lo = __floats2bfloat162_rn(o4.x, o4.y), hi = __floats2bfloat162_rn(o4.z, o4.w);
                  *reinterpret_cast<uint2*>(o.ep.yb + static_cast<size_t>(m) * o.ep.ldy + n) =
                      make_uint2(*reinterpret_cast<uint32_t*>(&lo), *reinterpret_cast<uint32_t*>(&hi));
                }
              }
              // the 8 threads of a row are 8 neighbouring lanes: chunk sum of squares in a fixed tree
              sq += __shfl_xor_sync(0xffffffffu, sq, 1);
              sq += __shfl_xor_sync(0xffffffffu, sq, 2);
              sq += __shfl_xor_sync(0xffffffffu, sq, 4);
              if (live && e_j == 0 && o.ep.ssq_out != nullptr)
                o.ep.ssq_out[static_cast<size_t>(m) * ((o.N + 31) / 32) + (sh.c0 + c * 32) / 32] = sq;
            }
          }
        }
      }
      // ---- border: this CTA's stores of matmul j are done
      if (j + 1 < p.n_ops) {
        epi_bar_sync();
        if (et == 0) {
          __threadfence();
          chain_arrive(p.sync + j);
        }
      }
    }
    tc_fence_before();
  }
  __syncthreads();
  if (warp == 1) {
    tc_fence_after();
    tmem_dealloc<TMEM_COLS>(tmem_base);
  }
}

}  // namespace tc
}  // namespace d3

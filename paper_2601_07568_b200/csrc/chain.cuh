// A skinny decode forward (up to 64 rows) runs as a chain: one persistent launch executes the
// operators of all layers one after the other -- QKV -> attention -> output projection -> gate/up ->
// down, layer after layer -- so that weights keep streaming from HBM across the borders between them.
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
//   * CHAIN_STRIP (gate/up: many columns): CTA i owns the column strip of units
//     [U i / n, U (i+1) / n) of 16 columns over the whole K range; the accumulator goes straight from
//     tensor memory to the epilogue (SwiGLU; RoPE + cache write is supported too).  No reduction.
//   * CHAIN_KSPLIT (O-proj, down: few columns, long K; QKV: so that a CTA does not re-read all of X
//     for a narrow strip): ks = 4 or 2 CTAs of a cluster share a strip of 32-column units and take a
//     ks-th of K each; the partial sums meet in distributed shared memory: a strip is cut into units of
//     16 rows x 32 columns, unit u belongs to the group's CTA u mod ks; every CTA leaves its partial in
//     its own shared memory and arrives on the owners' barriers; an owner reads its units from all ks
//     partials (remote loads by 128 threads at once: one warp pushing 16 KB through remote stores took
//     microseconds), adds them in rank order (fixed order: reproducible bits) with one (row, 4 columns)
//     element per thread and runs the epilogue (residual update, or RoPE + cache write).
// Weights come in the tiled form (contiguous pre-swizzled 128 x 64 blocks): a strip's rows are runs of
// whole 8-row swizzle groups inside the blocks it touches, copied with one bulk copy per block.
//
// Borders.  Matmul j+1 reads what matmul j wrote on other SMs, so each border is a grid-wide counter
// in global memory: a CTA adds one (release) after its last store of matmul j; the thread that loads
// activations and one epilogue thread wait for the count (acquire, bounded spin) before they touch
// matmul j+1's inputs.  Matmul 0 waits for the kernels before this launch (griddepcontrol.wait).
//
// Attention (CHAIN_ATTN) is an operator of the chain like the matmuls: cluster c takes the
// (sequence, kv head) pair c, its four CTAs a quarter of the keys each.  K/V tiles of 32 keys come in by
// TMA (the activation thread requests them), the four epilogue warps run the two small products on
// mma.sync with an online softmax (as attn_tc_kernel does), every warp leaves its unnormalised partial
// (O, m, l) in the CTA's staging buffer, and the CTA that owns a row (a quarter of the rows each) reads
// the row's partials from all four CTAs, merges them in source order and writes the row.  Meanwhile the weight
// thread fills the ring with the output projection's weights.
//
// The operators of a forward are described once, in global memory (the program); a launch runs a
// range of it.  Warp roles: 0 weights, 1 MMA issue + tensor-memory owner, 2-5 epilogue and attention,
// 6 activations and K/V tiles, 7 L2 prefetch of the weights ahead of the ring.
#pragma once
#include <cuda.h>

#include "attention.cuh"
#include "common.cuh"
#include "gemm_tc.cuh"
#include "ptx_sm100.cuh"

namespace d3 {
namespace tc {

constexpr int CHAIN_THREADS = 256;
constexpr int CHAIN_C = 4;
enum : int { CHAIN_STRIP = 0, CHAIN_KSPLIT = 1, CHAIN_ATTN = 2 };
constexpr int CHAIN_AKT = 32;      // keys per attention tile
constexpr int CHAIN_ASTAGES = 3;   // attention tile ring: 3 x 16 KB
constexpr uint32_t CHAIN_ASTAGE_BYTES = 4u * CHAIN_AKT * 128u;  // K lo, K hi, V lo, V hi slabs of [32][64] bf16
constexpr int CHAIN_ARECV_FLOATS = 64 * attn::PART_LD;           // attention's staging: 64 (key part, row) partial rows of (O, m, l)

struct ChainOp {
  int kind;   // CHAIN_STRIP / CHAIN_KSPLIT / CHAIN_ATTN
  int epi;    // CHAIN_STRIP: EPI_QKV or EPI_SWIGLU; CHAIN_KSPLIT: EPI_RESID or EPI_QKV
  int ks;     // CHAIN_KSPLIT: CTAs of a cluster that share a column strip and split K among them (1, 2 or 4);
              // the cluster then holds 4 / ks strips side by side
  int N, K;
  int x_map;  // which of the launch's activation tensor maps this matmul reads
  int layer;  // EPI_QKV and CHAIN_ATTN: the layer whose cache planes are written / read
  const __nv_bfloat16* w;  // tiled weights; CHAIN_ATTN: the query rows [M, n_q_heads * 128]
  EpiParams ep;            // CHAIN_ATTN: ep.y = output rows, same shape as the query rows
};

struct ChainParams {
  const ChainOp* prog;     // the forward's operators, in global memory
  int op_begin, op_end;    // this launch runs prog[op_begin, op_end)
  int M;
  int a_rows;              // rows of the X box: 32 or 64
  int stages;              // ring depth
  uint32_t w_stage_bytes;  // weight part of a stage: the widest strip of the program x 128 bytes
  int recv_bytes;          // staging region of the reductions (shared with the attention tile ring)
  int l2_ahead;            // weight slabs the L2 prefetch thread runs ahead of the weight thread (0: no prefetch)
  unsigned int* sync;      // [operators of the program] border counters, zero before the forward's first launch
  uint32_t* error_word;
  const int* skip_flag;
  // EPI_QKV and CHAIN_ATTN
  const float* rope_cos;
  const float* rope_sin;
  RowMap rm;
  int n_q_heads, n_kv_heads, max_seq;
  __nv_bfloat16* kv_base;        // cache [layer][K | V][max_batch][n_kv_heads][max_seq][128]
  long long kv_plane_rows;       // rows (of 128 elements) of one K or V plane
  float scale_log2;              // 1 / sqrt(d_head) * log2(e)
};

// This CTA's share of one matmul of the chain.
struct ChainShare {
  int c0, S;     // column strip [c0, c0 + S)
  int k0, n_k;   // K slabs [k0, k0 + n_k)
};
__device__ __forceinline__ ChainShare chain_share(const ChainOp& o, int cta, int n_cta, int cluster, int n_clusters, int rank) {
  ChainShare s;
  const int KC = (o.K + 63) / 64;
  if (o.kind == CHAIN_ATTN) {
    s.c0 = s.S = s.k0 = s.n_k = 0;  // no weights, no MMA of the tensor-memory pipeline
  } else if (o.kind == CHAIN_STRIP) {
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


// ---- attention inside the chain
// Geometry of one CHAIN_ATTN operator for this CTA (uniform over the CTA).
struct ChainAttn {
  bool work;        // this cluster has a (sequence, kv head) pair with live rows
  int b, g;         // sequence, kv head
  int n_valid, kv_len;
  int R;            // packed rows per kv head: query heads of the group x rows per sequence
  int BM;           // 32 or 64 packed rows
  int t0, n_my;     // this CTA's key tiles [t0, t0 + n_my) of CHAIN_AKT keys
  long long krow, vrow;  // first row of the pair's K / V in the cache tensor map
};
__device__ __forceinline__ ChainAttn chain_attn_geometry(const ChainParams& p, int layer, int cluster, int rank) {
  ChainAttn a;
  const int n_pairs = p.rm.bs * p.n_kv_heads;
  a.work = cluster < n_pairs;
  a.b = a.work ? cluster / p.n_kv_heads : 0;
  a.g = a.work ? cluster % p.n_kv_heads : 0;
  a.n_valid = a.work ? p.rm.n_valid[a.b] : 0;
  a.kv_len = a.work ? p.rm.kv_len[a.b] : 0;
  a.R = (p.n_q_heads / p.n_kv_heads) * p.rm.rows_per_seq;
  a.BM = a.R <= 32 ? 32 : 64;
  if (a.n_valid <= 0 || a.kv_len <= 0) a.work = false;
  const int n_tiles = a.work ? (a.kv_len + CHAIN_AKT - 1) / CHAIN_AKT : 0;
  const int tps = (n_tiles + CHAIN_C - 1) / CHAIN_C;
  a.t0 = rank * tps;
  const int t1 = a.t0 + tps < n_tiles ? a.t0 + tps : n_tiles;
  a.n_my = t1 > a.t0 ? t1 - a.t0 : 0;
  const long long plane = p.kv_plane_rows;
  a.krow = static_cast<long long>(2 * layer) * plane + (static_cast<long long>(a.b) * p.n_kv_heads + a.g) * p.max_seq;
  a.vrow = a.krow + plane;
  return a;
}

// The attention work of the four epilogue warps for one operator.  KQ = 1: 64 packed rows, warp w takes
// row group w and all keys of a tile; KQ = 2: 32 packed rows, warp w takes row group w % 2 and key part
// w / 2 (16 keys of every tile).  `tile_it` is the running count of attention tiles of this CTA (ring
// stage and phase).  Returns false when a wait gave up.
template <int KQ>
__device__ __forceinline__ bool chain_attention(const ChainParams& p, const ChainOp& o, const ChainAttn& a, int rank, int et,
                                                uint8_t* smem_kv, uint64_t* akv_full, uint64_t* akv_empty, float* recv,
                                                uint64_t* ready_bar, uint32_t ready_par, int& tile_it, volatile int* abort_flag) {
  using namespace attn;
  constexpr int NW = 4 / KQ;          // row groups of 16 packed rows
  constexpr int BM = NW * 16;
  constexpr int KPW = CHAIN_AKT / KQ;  // keys per warp and tile: 32 or 16
  constexpr int RPO = BM / CHAIN_C;    // rows per owner: 16 or 8
  constexpr int NS = CHAIN_C * KQ;     // sources per row: 4 or 8
  const int ew = et >> 5, lane = et & 31;
  const int rg = ew % NW, kq = ew / NW;
  const int g4 = lane >> 2, t4 = lane & 3;
  const int group = p.n_q_heads / p.n_kv_heads;
  const int rps = p.rm.rows_per_seq;
  const __nv_bfloat16* qbase = o.w;
  __nv_bfloat16* obase = static_cast<__nv_bfloat16*>(o.ep.y);

  float o_acc[16][4];
#pragma unroll
  for (int n = 0; n < 16; ++n)
#pragma unroll
    for (int e = 0; e < 4; ++e) o_acc[n][e] = 0.f;
  float m_lo = -INFINITY, m_hi = -INFINITY, l_lo = 0.f, l_hi = 0.f;
  bool alive = true;
  if (a.work) {
    // ---- Q fragments of this warp's 16 packed rows (rows g4 and g4 + 8), straight from global memory
    const int pr_lo = rg * 16 + g4, pr_hi = pr_lo + 8;
    auto row_ptr = [&](int pr, bool& ok) -> const __nv_bfloat16* {
      const int hg = pr / rps, r = pr % rps;
      ok = pr < a.R && r < a.n_valid;
      return qbase + (static_cast<size_t>(a.b) * rps + r) * p.n_q_heads * 128 + (a.g * group + hg) * 128;
    };
    bool ok_lo, ok_hi;
    const __nv_bfloat16* q_lo = row_ptr(pr_lo, ok_lo);
    const __nv_bfloat16* q_hi = row_ptr(pr_hi, ok_hi);
    uint32_t qa[8][4];
#pragma unroll
    for (int kk = 0; kk < 8; ++kk) {
      const int c = kk * 16 + t4 * 2;
      qa[kk][0] = ok_lo ? *reinterpret_cast<const uint32_t*>(q_lo + c) : 0u;
      qa[kk][1] = ok_hi ? *reinterpret_cast<const uint32_t*>(q_hi + c) : 0u;
      qa[kk][2] = ok_lo ? *reinterpret_cast<const uint32_t*>(q_lo + c + 8) : 0u;
      qa[kk][3] = ok_hi ? *reinterpret_cast<const uint32_t*>(q_hi + c + 8) : 0u;
    }
    // the 16 rows of a row group lie in one segment (segments are multiples of 16 rows): one key limit per warp
    const int kv_lim = row_kv_limit(p.rm, a.b, (rg * 16) % rps, a.kv_len);
    const int lm_row = lane & 7, lm_mat = lane >> 3;
    for (int i = 0; i < a.n_my && alive; ++i, ++tile_it) {
      const int s = tile_it % CHAIN_ASTAGES;
      const uint32_t ph = static_cast<uint32_t>(tile_it / CHAIN_ASTAGES) & 1u;
      alive = mbar_wait(&akv_full[s], ph, abort_flag, p.error_word);
      alive = __all_sync(0xffffffffu, alive);
      if (!alive) break;
      const uint32_t sb = smem_u32(smem_kv + s * CHAIN_ASTAGE_BYTES);
      const int j0 = (a.t0 + i) * CHAIN_AKT;
      // ---- S = Q K^T: key groups of 8, 8 k-steps of 16 over d_head
      float sc[KPW / 8][4];
#pragma unroll
      for (int n = 0; n < KPW / 8; ++n) {
        sc[n][0] = sc[n][1] = sc[n][2] = sc[n][3] = 0.f;
        const int key = kq * KPW + n * 8 + lm_row;
#pragma unroll
        for (int half = 0; half < 2; ++half) {
#pragma unroll
          for (int k2 = 0; k2 < 2; ++k2) {
            uint32_t b0, b1, b2, b3;
            ldmatrix_x4(sb + half * (CHAIN_AKT * 128) + swz(key, k2 * 4 + lm_mat), b0, b1, b2, b3);
            const int kk = half * 4 + k2 * 2;
            mma_bf16_16816(sc[n], qa[kk], b0, b1);
            mma_bf16_16816(sc[n], qa[kk + 1], b2, b3);
          }
        }
      }
      // ---- scale, mask keys beyond the row group's limit, online softmax (rows g4 and g4 + 8)
      float mx_lo = -INFINITY, mx_hi = -INFINITY;
#pragma unroll
      for (int n = 0; n < KPW / 8; ++n) {
        const int key = j0 + kq * KPW + n * 8 + t4 * 2;
        const bool v0 = key < kv_lim, v1 = key + 1 < kv_lim;
        sc[n][0] = v0 ? sc[n][0] * p.scale_log2 : -INFINITY;
        sc[n][1] = v1 ? sc[n][1] * p.scale_log2 : -INFINITY;
        sc[n][2] = v0 ? sc[n][2] * p.scale_log2 : -INFINITY;
        sc[n][3] = v1 ? sc[n][3] * p.scale_log2 : -INFINITY;
        mx_lo = fmaxf(mx_lo, fmaxf(sc[n][0], sc[n][1]));
        mx_hi = fmaxf(mx_hi, fmaxf(sc[n][2], sc[n][3]));
      }
      mx_lo = fmaxf(mx_lo, __shfl_xor_sync(0xffffffffu, mx_lo, 1));
      mx_lo = fmaxf(mx_lo, __shfl_xor_sync(0xffffffffu, mx_lo, 2));
      mx_hi = fmaxf(mx_hi, __shfl_xor_sync(0xffffffffu, mx_hi, 1));
      mx_hi = fmaxf(mx_hi, __shfl_xor_sync(0xffffffffu, mx_hi, 2));
      const float mn_lo = fmaxf(m_lo, mx_lo), mn_hi = fmaxf(m_hi, mx_hi);
      const float b_lo = mn_lo == -INFINITY ? 0.f : mn_lo, b_hi = mn_hi == -INFINITY ? 0.f : mn_hi;
      const float c_lo = exp2f(m_lo - b_lo), c_hi = exp2f(m_hi - b_hi);
      m_lo = mn_lo;
      m_hi = mn_hi;
      float s_lo = 0.f, s_hi = 0.f;
      uint32_t pa[KPW / 16][4];
#pragma unroll
      for (int n = 0; n < KPW / 8; ++n) {
        const float p0 = exp2f(sc[n][0] - b_lo), p1 = exp2f(sc[n][1] - b_lo);
        const float p2 = exp2f(sc[n][2] - b_hi), p3 = exp2f(sc[n][3] - b_hi);
        s_lo += p0 + p1;
        s_hi += p2 + p3;
        pa[n >> 1][(n & 1) * 2 + 0] = pack_bf16(p0, p1);
        pa[n >> 1][(n & 1) * 2 + 1] = pack_bf16(p2, p3);
      }
      l_lo = l_lo * c_lo + s_lo;
      l_hi = l_hi * c_hi + s_hi;
#pragma unroll
      for (int n = 0; n < 16; ++n) {
        o_acc[n][0] *= c_lo; o_acc[n][1] *= c_lo;
        o_acc[n][2] *= c_hi; o_acc[n][3] *= c_hi;
      }
      // ---- O += P V: k-steps of 16 keys, 16 output groups of 8 dims
#pragma unroll
      for (int kk = 0; kk < KPW / 16; ++kk) {
        const int key = kq * KPW + kk * 16 + (lm_mat & 1) * 8 + lm_row;
#pragma unroll
        for (int n2 = 0; n2 < 8; ++n2) {
          const int chunk = n2 * 2 + (lm_mat >> 1);
          uint32_t b0, b1, b2, b3;
          ldmatrix_x4_trans(sb + (2 + (chunk >> 3)) * (CHAIN_AKT * 128) + swz(key, chunk & 7), b0, b1, b2, b3);
          mma_bf16_16816(o_acc[n2 * 2], pa[kk], b0, b1);
          mma_bf16_16816(o_acc[n2 * 2 + 1], pa[kk], b2, b3);
        }
      }
      __syncwarp();
      if (lane == 0) mbar_arrive(&akv_empty[s]);  // the tile thread refills the stage once all four warps are through
    }
    // row sums over the quad
    l_lo += __shfl_xor_sync(0xffffffffu, l_lo, 1);
    l_lo += __shfl_xor_sync(0xffffffffu, l_lo, 2);
    l_hi += __shfl_xor_sync(0xffffffffu, l_hi, 1);
    l_hi += __shfl_xor_sync(0xffffffffu, l_hi, 2);
  }
  if (!epi_all(alive)) return false;
  if (!a.work) return true;  // uniform over the cluster: no pair, nothing to merge
  // ---- this warp's partial of its rows goes to the CTA's own staging buffer [key part][row][PART_LD]; the
  // owner of a row (a quarter of the rows each) then reads the row's partials from all four CTAs
  {
    float* r_lo = recv + (static_cast<size_t>(kq) * BM + rg * 16 + g4) * PART_LD;
    float* r_hi = r_lo + 8 * PART_LD;
#pragma unroll
    for (int n = 0; n < 16; ++n) {
      *reinterpret_cast<float2*>(r_lo + n * 8 + t4 * 2) = make_float2(o_acc[n][0], o_acc[n][1]);
      *reinterpret_cast<float2*>(r_hi + n * 8 + t4 * 2) = make_float2(o_acc[n][2], o_acc[n][3]);
    }
    if (t4 == 0) {
      r_lo[128] = m_lo; r_lo[129] = l_lo;  // a part without keys leaves m = -inf, l = 0
      r_hi[128] = m_hi; r_hi[129] = l_hi;
    }
  }
  epi_bar_sync();  // the whole partial is in place before the arrivals below
  if (et < CHAIN_C) mbar_arrive_remote(ready_bar, static_cast<uint32_t>(et));
  bool ok = mbar_wait_cluster(ready_bar, ready_par, abort_flag, p.error_word);
  if (!epi_all(ok)) return false;
  // ---- owner: merge the NS partials of its RPO rows in source order, one (row, 4 dims) item per thread and pass
  const uint32_t recv_addr = smem_u32(recv);
  for (int e = et; e < RPO * 32; e += 128) {
    const int local = e >> 5, c4 = (e & 31) * 4;
    const int pr = rank * RPO + local;
    const int hg = pr / rps, r = pr % rps;
    if (pr >= a.R || r >= a.n_valid) continue;
    float ms[NS], ls[NS];
    float4 vs[NS];
    float Mx = -INFINITY;
#pragma unroll
    for (int s2 = 0; s2 < NS; ++s2) {  // source s2: CTA s2 / KQ, key part s2 % KQ
      const uint32_t ra = map_to_cta(recv_addr + static_cast<uint32_t>(((s2 % KQ) * BM + pr) * PART_LD) * 4u, static_cast<uint32_t>(s2 / KQ));
      ms[s2] = ld_cluster_f(ra + 128 * 4);
      ls[s2] = ld_cluster_f(ra + 129 * 4);
      vs[s2] = ld_cluster_f4(ra + c4 * 4);
      Mx = fmaxf(Mx, ms[s2]);
    }
    float L = 0.f, a0 = 0.f, a1 = 0.f, a2 = 0.f, a3 = 0.f;
#pragma unroll
    for (int s2 = 0; s2 < NS; ++s2) {
      if (ls[s2] != 0.f) {
        const float w = exp2f(ms[s2] - Mx);
        L += w * ls[s2];
        a0 += w * vs[s2].x; a1 += w * vs[s2].y; a2 += w * vs[s2].z; a3 += w * vs[s2].w;
      }
    }
    const float inv = L > 0.f ? 1.0f / L : 0.f;
    __nv_bfloat16* out = obase + (static_cast<size_t>(a.b) * rps + r) * p.n_q_heads * 128 + (a.g * group + hg) * 128;
    *reinterpret_cast<uint2*>(out + c4) = make_uint2(pack_bf16(a0 * inv, a1 * inv), pack_bf16(a2 * inv, a3 * inv));
  }
  return true;
}

// Dynamic shared memory (1024-byte aligned inside the kernel):
//   [stages x a_rows x 128 B] X slabs, [stages x w_stage_bytes] W slabs (at least (128 - a_rows) * 128
//   bytes follow the last X slab: the MMA reads 128 rows of its A operand whatever a_rows is),
//   receive buffer [units per owner][4 sources][16 rows][32 columns] fp32, barriers.
inline size_t chain_recv_bytes(int a_rows, int max_ksplit_cols) {
  return static_cast<size_t>(a_rows) * max_ksplit_cols * 4;  // this CTA's fp32 partial of its widest K-split strip
}
// Everything but the ring: staging region (`recv` bytes: the largest of the matmuls' partial sums,
// attention's partial rows and the attention tile ring, which share it), barriers, alignment slack.
inline size_t chain_fixed_smem_bytes(size_t recv, int stages) {
  return 2048 + recv + (2 * stages + 2 * CHAIN_ASTAGES + 8) * 8 + 64 + 2 * sizeof(ChainOp) + 16;
}
inline size_t chain_smem_bytes(int a_rows, uint32_t w_stage_bytes, int stages, size_t recv) {
  size_t body = static_cast<size_t>(stages) * (static_cast<size_t>(a_rows) * 128 + w_stage_bytes);
  const size_t reach = static_cast<size_t>(stages - 1) * a_rows * 128 + 128 * 128;
  if (body < reach) body = reach;
  return body + chain_fixed_smem_bytes(recv, stages);
}

__global__ void __launch_bounds__(CHAIN_THREADS, 1)
chain_kernel(const __grid_constant__ CUtensorMap tmap_x0, const __grid_constant__ CUtensorMap tmap_x1,
             const __grid_constant__ CUtensorMap tmap_x2, const __grid_constant__ CUtensorMap tmap_kv, const ChainParams p) {
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
  // One region serves as the attention tile ring and as the staging buffer of the reductions (the
  // matmuls' partial sums, attention's partial rows): a CTA writes its staging buffer itself, after its own
  // tiles are consumed, and peers read a staging buffer only between two borders in which no tile arrives.
  uint8_t* smem_kv = smem + ((body + 1023) & ~size_t(1023));  // 1024-byte aligned slabs
  float* recv = reinterpret_cast<float*>(smem_kv);
  uint64_t* full_bar = reinterpret_cast<uint64_t*>(smem_kv + p.recv_bytes);
  uint64_t* empty_bar = full_bar + stages;
  uint64_t* acc_full = empty_bar + stages;   // [2]
  uint64_t* acc_empty = acc_full + 2;        // [2]
  uint64_t* ready_bar = acc_empty + 2;       // all four partials of this CTA's units have arrived
  uint64_t* akv_full = ready_bar + 1;        // [CHAIN_ASTAGES] attention tile ring
  uint64_t* akv_empty = akv_full + CHAIN_ASTAGES;
  uint32_t* tmem_slot = reinterpret_cast<uint32_t*>(akv_empty + CHAIN_ASTAGES);
  volatile int* abort_flag = reinterpret_cast<volatile int*>(tmem_slot + 1);
  // The epilogue warps read the operator they work on from shared memory: an acquire (border, cluster
  // barrier) drops the SM's cached copies of global memory, and every field read after it would cost
  // a trip to L2 in the middle of the epilogue.
  ChainOp* sops = reinterpret_cast<ChainOp*>(tmem_slot + 4);  // [2], 16-byte aligned
  volatile int* w_progress = reinterpret_cast<volatile int*>(tmem_slot + 2);  // weight slabs requested so far

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
    prefetch_tensormap(&tmap_kv);
    for (int s = 0; s < CHAIN_ASTAGES; ++s) {
      mbar_init(&akv_full[s], 1);
      mbar_init(&akv_empty[s], 4);  // one arrival per attention warp
    }
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
    *w_progress = 0;
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
      int s = 0, n_req = 0;
      uint32_t ph = 1;  // parity to wait for on the empty barrier (first lap: passes at once)
      bool ok = true;
      for (int j = p.op_begin; j < p.op_end && ok; ++j) {
        const ChainOp& o = p.prog[j];
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
          *w_progress = ++n_req;
          if (++s == stages) { s = 0; ph ^= 1u; }
        }
      }
    }
  } else if (warp == 7) {
    // ---------------- L2 prefetch: the same walk as the weight thread, p.l2_ahead slabs ahead of it.  While
    // the ring is full (a border's dependency resolves: epilogue, reduction, counter, activation load) HBM
    // would idle; these requests keep it busy, and the weight thread's later copies find their bytes in L2.
    if (p.l2_ahead > 0) {  // the whole warp: one 128-byte line per lane and request
      int n_pf = 0;
      bool ok = true;
      for (int j = p.op_begin; j < p.op_end && ok; ++j) {
        const ChainOp& o = p.prog[j];
        const ChainShare sh = chain_share(o, cta, n_cta, cluster, n_clusters, rank);
        if (sh.n_k == 0) continue;
        const int KC = (o.K + 63) / 64;
        const __nv_bfloat16* piece_src[3];
        uint32_t piece_bytes[3];
        {
          int row = sh.c0, left = sh.S;
#pragma unroll
          for (int q = 0; q < 3; ++q) {
            const int blk = row >> 7, r0 = row & 127;
            const int n = left < 128 - r0 ? left : 128 - r0;
            piece_src[q] = o.w + (static_cast<long long>(blk) * KC * 128 + r0) * 64;
            piece_bytes[q] = static_cast<uint32_t>(n) * 128u;
            row += n;
            left -= n;
          }
        }
        for (int i = 0; i < sh.n_k; ++i) {
          // stay within l2_ahead slabs of the weight thread (bounded wait: the weight thread always moves on or gives up)
          uint64_t t0 = 0;
          uint32_t it = 0;
          int wp = *w_progress;
          while (n_pf >= wp + p.l2_ahead) {
            __nanosleep(64);
            if ((++it & 0x3f) == 0) {
              if (*abort_flag) { ok = false; break; }
              const uint64_t now = global_ns();
              if (t0 == 0) t0 = now;
              else if (now - t0 > WAIT_LIMIT_NS) { ok = false; break; }
            }
            wp = *w_progress;
          }
          ok = __all_sync(0xffffffffu, ok);
          wp = __shfl_sync(0xffffffffu, wp, 0);
          if (!ok) break;
          if (n_pf >= wp) {  // (what the weight thread has already asked for needs no prefetch)
            const size_t slab = static_cast<size_t>(sh.k0 + i) * (128 * 64);
#pragma unroll
            for (int q = 0; q < 3; ++q)
              for (uint32_t b = static_cast<uint32_t>(lane) * 128u; b < piece_bytes[q]; b += 32u * 128u)
                prefetch_line_l2(reinterpret_cast<const uint8_t*>(piece_src[q] + slab) + b);
          }
          ++n_pf;
        }
      }
    }
  } else if (warp == 6) {
    // ---------------- activations: behind the border of each matmul
    if (lane == 0) {
      int s = 0;
      uint32_t ph = 1;
      int tile_it = 0;  // attention tiles requested so far
      bool ok = true;
      grid_dep_wait();
      for (int j = p.op_begin; j < p.op_end && ok; ++j) {
        // (read before the border's acquire, which drops the SM's cached copies of global memory)
        const ChainOp& o = p.prog[j];
        const int kind = o.kind;
        const ChainShare sh = chain_share(o, cta, n_cta, cluster, n_clusters, rank);
        const CUtensorMap* tm = x_map_of(o.x_map);
        ChainAttn at{};
        if (kind == CHAIN_ATTN) at = chain_attn_geometry(p, o.layer, cluster, rank);
        if (j > p.op_begin) {
          if (!chain_wait_count(p.sync + (j - 1), static_cast<unsigned int>(n_cta), abort_flag, p.error_word)) break;
          fence_proxy_async_all();  // the rows were written with ordinary stores; the loads below go through the async proxy
        }
        if (kind == CHAIN_ATTN) {
          // K/V tiles of this CTA's key range (the block's own rows were written by the QKV operator before the border)
          for (int i = 0; i < at.n_my; ++i, ++tile_it) {
            const int ks2 = tile_it % CHAIN_ASTAGES;
            const uint32_t kph = (static_cast<uint32_t>(tile_it / CHAIN_ASTAGES) & 1u) ^ 1u;
            if (!mbar_wait(&akv_empty[ks2], kph, abort_flag, p.error_word)) { ok = false; break; }
            uint8_t* st = smem_kv + ks2 * CHAIN_ASTAGE_BYTES;
            const int j0 = (at.t0 + i) * CHAIN_AKT;
            mbar_arrive_expect_tx(&akv_full[ks2], CHAIN_ASTAGE_BYTES);
            tma_load_2d(st, &tmap_kv, &akv_full[ks2], 0, static_cast<int>(at.krow + j0));
            tma_load_2d(st + CHAIN_AKT * 128, &tmap_kv, &akv_full[ks2], 64, static_cast<int>(at.krow + j0));
            tma_load_2d(st + 2 * CHAIN_AKT * 128, &tmap_kv, &akv_full[ks2], 0, static_cast<int>(at.vrow + j0));
            tma_load_2d(st + 3 * CHAIN_AKT * 128, &tmap_kv, &akv_full[ks2], 64, static_cast<int>(at.vrow + j0));
          }
          continue;
        }
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
      for (int j = p.op_begin; j < p.op_end && ok; ++j) {
        const ChainShare sh = chain_share(p.prog[j], cta, n_cta, cluster, n_clusters, rank);
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
    int n_acc = 0, n_ks = 0, attn_tiles = 0;
    bool alive = true;
    for (int j = p.op_begin; j < p.op_end && alive; ++j) {
      {  // the operator's description into shared memory (buffer j & 1: the previous one is still in use by no one,
         // every thread passed the barrier at the end of operator j - 1 after its last read of it)
        const uint32_t* src = reinterpret_cast<const uint32_t*>(p.prog + j);
        uint32_t* dst = reinterpret_cast<uint32_t*>(sops + (j & 1));
        for (int w = et; w < static_cast<int>(sizeof(ChainOp) / 4); w += 128) dst[w] = src[w];
        if (j == p.op_begin) epi_bar_sync();  // later operators: the border's barrier below orders the copy
      }
      const ChainOp& o = sops[j & 1];
      if (j > p.op_begin) {  // rows, chunk sums and residual values written by the operator before this one, on any SM
        bool ok = true;
        if (et == 0) ok = chain_wait_count(p.sync + (j - 1), static_cast<unsigned int>(n_cta), abort_flag, p.error_word);
        if (!epi_all(ok)) { alive = false; break; }
      }
      const ChainShare sh = chain_share(o, cta, n_cta, cluster, n_clusters, rank);
      if (o.kind == CHAIN_ATTN) {
        const ChainAttn at = chain_attn_geometry(p, o.layer, cluster, rank);
        const uint32_t ready_par = static_cast<uint32_t>(n_ks) & 1u;
        if (at.work) ++n_ks;  // every CTA of a cluster with a pair owns rows
        const bool ok = at.BM == 32
            ? chain_attention<2>(p, o, at, rank, et, smem_kv, akv_full, akv_empty, recv, ready_bar, ready_par, attn_tiles, abort_flag)
            : chain_attention<1>(p, o, at, rank, et, smem_kv, akv_full, akv_empty, recv, ready_bar, ready_par, attn_tiles, abort_flag);
        if (!ok) { alive = false; break; }
      } else if (sh.n_k > 0) {
        constexpr int buf = 0;
        const uint32_t acc_par = static_cast<uint32_t>(n_acc) & 1u;
        ++n_acc;
        // the matmul's parameters in the form the shared epilogue code reads
        GemmParams gp{};
        gp.M = p.M; gp.N = o.N; gp.K = o.K;
        gp.a_rows = p.a_rows;
        gp.error_word = p.error_word;
        gp.ep = o.ep;
        __nv_bfloat16* const k_cache = p.kv_base + static_cast<size_t>(2 * o.layer) * p.kv_plane_rows * 128;
        __nv_bfloat16* const v_cache = k_cache + static_cast<size_t>(p.kv_plane_rows) * 128;
        gp.rope_cos = p.rope_cos; gp.rope_sin = p.rope_sin; gp.pos_base = p.rm.pos_base; gp.n_valid = p.rm.n_valid;
        gp.rows_per_seq = p.rm.rows_per_seq; gp.n_q_heads = p.n_q_heads; gp.n_kv_heads = p.n_kv_heads; gp.max_seq = p.max_seq;
        gp.k_cache = k_cache; gp.v_cache = v_cache;
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
          // ---- K-split: every CTA of the group leaves its partial in its own shared memory and tells the
          // owners; an owner reads its units from all ks partials (remote loads, 128 threads at once)
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
                const int b = m / p.rm.rows_per_seq, r = m % p.rm.rows_per_seq;
                if (r < p.rm.n_valid[b]) {
                  const int pos = p.rm.pos_base[b] + r;
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
            // the accumulator goes to this CTA's own staging buffer: [chunk][row][8 groups of 4 columns], the
            // groups of a row rotated by the row so that neither these stores nor the owners' loads collide
            TmemSource tsrc{lane_addr};
#pragma unroll 1
            for (int c = 0; c < n_chunks; ++c) {
              float v[32];
              tsrc.load(c * 32, v);
              float4* dst = reinterpret_cast<float4*>(recv) + static_cast<size_t>(c * p.a_rows + row) * 8;
#pragma unroll
              for (int q = 0; q < 8; ++q) dst[q ^ (row & 7)] = make_float4(v[4 * q], v[4 * q + 1], v[4 * q + 2], v[4 * q + 3]);
            }
          }
          tc_fence_before();
          mbar_arrive(&acc_empty[buf]);
          epi_bar_sync();  // the whole partial is in place before the arrivals below
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
                {
                  const int srow = (u % RS) * 16 + e_row;
                  const uint32_t off = static_cast<uint32_t>((((u / RS) * p.a_rows + srow) * 8 + (e_j ^ (srow & 7))) * 16);
                  float4 part[CHAIN_C];
#pragma unroll
                  for (int s2 = 0; s2 < CHAIN_C; ++s2)
                    if (s2 < ks) part[s2] = ld_cluster_f4(map_to_cta(recv_addr + off, static_cast<uint32_t>(gbase + s2)));
#pragma unroll
                  for (int s2 = 0; s2 < CHAIN_C; ++s2)
                    if (s2 < ks) { acc.x += part[s2].x; acc.y += part[s2].y; acc.z += part[s2].z; acc.w += part[s2].w; }
                }
                float rs = 1.f;
#pragma unroll
                for (int t = 0; t < 4; ++t)
                  if (t == u % RS) rs = rs_row[t];
                const float a0 = acc.x * rs, a1 = acc.y * rs, a2 = acc.z * rs, a3 = acc.w * rs;
                const int head = n / 128, off = n % 128, pos = pos4[q];
                const int b = m / p.rm.rows_per_seq;
                if (head < p.n_q_heads + p.n_kv_heads) {
                  __nv_bfloat16* dst = head < p.n_q_heads
                      ? static_cast<__nv_bfloat16*>(o.ep.y) + static_cast<size_t>(m) * o.ep.ldy + head * 128
                      : k_cache + ((static_cast<size_t>(b) * p.n_kv_heads + (head - p.n_q_heads)) * p.max_seq + pos) * 128;
                  const int i0 = off / 2;  // pairs (i0, i0 + 64) and (i0 + 1, i0 + 65)
                  __nv_bfloat162 lo = __floats2bfloat162_rn(a0 * co[q].x - a1 * si[q].x, a2 * co[q].y - a3 * si[q].y);
                  __nv_bfloat162 hi = __floats2bfloat162_rn(a1 * co[q].x + a0 * si[q].x, a3 * co[q].y + a2 * si[q].y);
                  *reinterpret_cast<uint32_t*>(dst + i0) = *reinterpret_cast<uint32_t*>(&lo);
                  *reinterpret_cast<uint32_t*>(dst + 64 + i0) = *reinterpret_cast<uint32_t*>(&hi);
                } else if (head < p.n_q_heads + 2 * p.n_kv_heads) {
                  __nv_bfloat16* dst = v_cache +
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
              {
                const uint32_t off = static_cast<uint32_t>(((c * p.a_rows + m) * 8 + (e_j ^ (m & 7))) * 16);
                float4 part[CHAIN_C];
#pragma unroll
                for (int s2 = 0; s2 < CHAIN_C; ++s2)
                  if (s2 < ks) part[s2] = ld_cluster_f4(map_to_cta(recv_addr + off, static_cast<uint32_t>(gbase + s2)));
#pragma unroll
                for (int s2 = 0; s2 < CHAIN_C; ++s2)
                  if (s2 < ks) { acc.x += part[s2].x; acc.y += part[s2].y; acc.z += part[s2].z; acc.w += part[s2].w; }
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
      if (j + 1 < p.op_end) {
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
  cluster_sync_all();  // no CTA leaves while a peer may still read its staging buffer
}

}  // namespace tc
}  // namespace d3

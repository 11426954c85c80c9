// Block-bidirectional attention over the KV cache: every live row of sequence b attends to cache
// slots [0, kv_len[b]) of its kv head (prefix and the block's own rows, written just before), with
// no causal mask.  Online softmax in fp32.
#pragma once
#include "common.cuh"
#include "small_kernels.cuh"

namespace d3 {
namespace attn {

// ----------------------------------------------------------------------------- SIMT kernel (any T)
// grid (ceil(rows_per_seq / QT), hq, bs), 128 threads.  Keys are staged 32 at a time in shared
// memory as fp32; lane j scores key j, then lanes own output dims (lane + 32 i).
constexpr int QT = 8, KC = 32, THREADS = 128;

template <typename T, int DH>
__global__ void __launch_bounds__(THREADS) attn_simt_kernel(const T* __restrict__ q, const T* __restrict__ k_cache,
                                                            const T* __restrict__ v_cache, T* __restrict__ out,
                                                            RowMap rm, int hq, int hkv, int max_seq, float scale) {
  __shared__ float Ks[KC][DH + 1];
  __shared__ float Vs[KC][DH + 1];
  __shared__ float Qs[QT][DH];
  const int b = blockIdx.z, h = blockIdx.y, r0 = blockIdx.x * QT;
  const int n_valid = rm.n_valid[b];
  if (r0 >= n_valid) return;
  const int kv_len = rm.kv_len[b];
  const int g = h / (hq / hkv);
  const T* kb = k_cache + (static_cast<size_t>(b) * hkv + g) * max_seq * DH;
  const T* vb = v_cache + (static_cast<size_t>(b) * hkv + g) * max_seq * DH;
  const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
  constexpr int RPW = QT / (THREADS / 32);  // rows per warp
  constexpr int DPL = DH / 32;              // dims per lane

  for (int e = threadIdx.x; e < QT * DH; e += THREADS) {
    int r = e / DH, d = e % DH;
    int row = r0 + r;
    Qs[r][d] = (row < n_valid)
                   ? TypeOps<T>::to_f(q[(static_cast<size_t>(b) * rm.rows_per_seq + row) * hq * DH + h * DH + d]) * scale
                   : 0.f;
  }
  float m_run[RPW], l_run[RPW], acc[RPW][DPL];
#pragma unroll
  for (int i = 0; i < RPW; ++i) {
    m_run[i] = -INFINITY;
    l_run[i] = 0.f;
#pragma unroll
    for (int d = 0; d < DPL; ++d) acc[i][d] = 0.f;
  }
  for (int j0 = 0; j0 < kv_len; j0 += KC) {
    __syncthreads();
    for (int e = threadIdx.x; e < KC * DH; e += THREADS) {
      int j = e / DH, d = e % DH;
      bool in = (j0 + j) < kv_len;
      Ks[j][d] = in ? TypeOps<T>::to_f(kb[static_cast<size_t>(j0 + j) * DH + d]) : 0.f;
      Vs[j][d] = in ? TypeOps<T>::to_f(vb[static_cast<size_t>(j0 + j) * DH + d]) : 0.f;
    }
    __syncthreads();
#pragma unroll
    for (int i = 0; i < RPW; ++i) {
      const int r = warp * RPW + i;
      if (r0 + r >= n_valid) continue;  // warp-uniform
      float s = 0.f;
#pragma unroll 8
      for (int d = 0; d < DH; ++d) s = fmaf(Qs[r][d], Ks[lane][d], s);
      if (j0 + lane >= row_kv_limit(rm, b, r0 + r, kv_len)) s = -INFINITY;  // keys of later segments stay unseen
      float mx = s;
#pragma unroll
      for (int o = 16; o > 0; o >>= 1) mx = fmaxf(mx, __shfl_xor_sync(0xffffffffu, mx, o));
      const float m_new = fmaxf(m_run[i], mx);
      const float p = __expf(s - m_new);  // -inf -> 0
      const float corr = __expf(m_run[i] - m_new);
      l_run[i] = l_run[i] * corr + warp_sum(p);
      m_run[i] = m_new;
#pragma unroll
      for (int d = 0; d < DPL; ++d) acc[i][d] *= corr;
      for (int j = 0; j < KC; ++j) {
        const float pj = __shfl_sync(0xffffffffu, p, j);
#pragma unroll
        for (int d = 0; d < DPL; ++d) acc[i][d] = fmaf(pj, Vs[j][lane + 32 * d], acc[i][d]);
      }
    }
  }
#pragma unroll
  for (int i = 0; i < RPW; ++i) {
    const int row = r0 + warp * RPW + i;
    if (row >= n_valid) continue;
    const float inv = 1.0f / l_run[i];
    T* o = out + (static_cast<size_t>(b) * rm.rows_per_seq + row) * hq * DH + h * DH;
#pragma unroll
    for (int d = 0; d < DPL; ++d) o[lane + 32 * d] = TypeOps<T>::from_f(acc[i][d] * inv);
  }
}

}  // namespace attn
}  // namespace d3

// ----------------------------------------------------------------------------- tensor-core kernel
// bf16, d_head = 128.  The work is bound by reading K and V once from HBM (at 32 query rows per
// kv head the arithmetic intensity is 32 flop/byte), so the design goal is bytes in flight, not
// tensor throughput: K/V tiles of 64 keys are staged by TMA (128-byte swizzle) in a 3-deep ring,
// the two small products per tile run on mma.sync m16n8k16 with fragments read by ldmatrix, and the
// softmax stays in registers.  One CTA = one (sequence, kv head, query tile, key split); a query
// tile packs the rows of all query heads that share the kv head (GQA): packed row pr = head_in_group
// * rows_per_seq + r.  With several key splits (at most 8) the CTAs of one query tile form a
// thread-block cluster: each leaves its unnormalised partial (O, m, l) in its own shared memory,
// and after a cluster barrier every CTA merges a slice of the rows, reading its peers' partials
// through distributed shared memory in split order; nothing goes through global memory.
#include "ptx_sm100.cuh"

namespace d3 {
namespace attn {

constexpr int KT = 64;        // keys per tile
constexpr int TC_STAGES = 3;  // ring depth: 3 x 32 KB
constexpr int PART_LD = 132;  // floats per partial row: 128 outputs, m, l, 2 pad
constexpr uint32_t STAGE_BYTES = 4u * KT * 128u;  // K lo, K hi, V lo, V hi slabs of [KT][64] bf16

struct AttnTcParams {
  const __nv_bfloat16* q;  // [bs * rows_per_seq, hq * 128]
  __nv_bfloat16* out;      // same shape
  RowMap rm;
  int hq, hkv, max_seq;
  long long k_row0, v_row0;  // first row of this layer's K / V plane in the cache tensor map
  int n_splits;      // = gridDim.z = cluster size along z (1..8)
  float scale_log2;  // 1/sqrt(d_head) * log2(e)
  uint32_t* error_word;
};

__device__ __forceinline__ void ldmatrix_x4(uint32_t addr, uint32_t& r0, uint32_t& r1, uint32_t& r2, uint32_t& r3) {
  asm volatile("ldmatrix.sync.aligned.m8n8.x4.shared.b16 {%0, %1, %2, %3}, [%4];"
               : "=r"(r0), "=r"(r1), "=r"(r2), "=r"(r3) : "r"(addr));
}
__device__ __forceinline__ void ldmatrix_x4_trans(uint32_t addr, uint32_t& r0, uint32_t& r1, uint32_t& r2, uint32_t& r3) {
  asm volatile("ldmatrix.sync.aligned.m8n8.x4.trans.shared.b16 {%0, %1, %2, %3}, [%4];"
               : "=r"(r0), "=r"(r1), "=r"(r2), "=r"(r3) : "r"(addr));
}
__device__ __forceinline__ void mma_bf16_16816(float (&c)[4], const uint32_t (&a)[4], uint32_t b0, uint32_t b1) {
  asm volatile("mma.sync.aligned.m16n8k16.row.col.f32.bf16.bf16.f32 {%0, %1, %2, %3}, {%4, %5, %6, %7}, {%8, %9}, {%0, %1, %2, %3};"
               : "+f"(c[0]), "+f"(c[1]), "+f"(c[2]), "+f"(c[3])
               : "r"(a[0]), "r"(a[1]), "r"(a[2]), "r"(a[3]), "r"(b0), "r"(b1));
}
__device__ __forceinline__ uint32_t pack_bf16(float lo, float hi) {
  __nv_bfloat162 t = __floats2bfloat162_rn(lo, hi);
  return *reinterpret_cast<uint32_t*>(&t);
}
// Byte offset of 16-byte chunk `c` (0..7) of row `r` inside a [rows][64] bf16 slab written by TMA
// with the 128-byte swizzle (slab base 1024-byte aligned).
__device__ __forceinline__ uint32_t swz(int r, int c) { return static_cast<uint32_t>(r * 128 + ((c ^ (r & 7)) << 4)); }

// grid (q_tiles, bs * hkv, n_splits); NW groups of 16 packed rows, each worked on by KQ warps that
// take KT / KQ keys of every tile (a decode-sized CTA would otherwise keep two of the SM's four
// tensor-core partitions idle and walk through its tiles four times as long).  Warp w: row group
// w % NW, key part w / NW.  Every warp keeps its own running softmax state; the key parts are
// merged through shared memory after the last tile, then the key splits across the cluster.
// Registers: two CTAs per SM (128 registers a thread) cost the 8-row-group variant a few hundred bytes
// of spills and still pay (GQA decode: 38 -> 34 us per launch); the 4-row-group variant was slower that
// way at long prefixes (102 -> 109 us) and keeps its 174 registers and one CTA per SM.
template <int NW, int KQ>
__global__ void __launch_bounds__(NW * KQ * 32, NW == 4 ? 1 : 2) attn_tc_kernel(const __grid_constant__ CUtensorMap tmap_kv,
                                                               const AttnTcParams p) {
  constexpr int BM = NW * 16;
  constexpr int KPW = KT / KQ;  // keys per warp and tile: 64, 32 or 16
  constexpr int NTHREADS = NW * KQ * 32;
  static_assert(KPW % 16 == 0, "a warp takes whole 16-key MMA steps");
  extern __shared__ uint8_t smem_raw[];
  uint8_t* smem = reinterpret_cast<uint8_t*>((reinterpret_cast<uintptr_t>(smem_raw) + 1023) & ~uintptr_t(1023));
  uint64_t* full_bar = reinterpret_cast<uint64_t*>(smem + TC_STAGES * STAGE_BYTES);
  uint64_t* empty_bar = full_bar + TC_STAGES;
  volatile int* abort_flag = reinterpret_cast<volatile int*>(empty_bar + TC_STAGES);

  const int warp_id = threadIdx.x >> 5, lane = threadIdx.x & 31;
  const int warp = warp_id % NW;  // row group
  const int kq = warp_id / NW;    // key part
  const int g4 = lane >> 2, t4 = lane & 3;
  const int qt = blockIdx.x, pair = blockIdx.y, split = blockIdx.z;
  const int b = pair / p.hkv, g = pair % p.hkv;
  const int group = p.hq / p.hkv;
  const int rps = p.rm.rows_per_seq;

  if (threadIdx.x == 0) {
    ptx::prefetch_tensormap(&tmap_kv);
    for (int s = 0; s < TC_STAGES; ++s) {
      ptx::mbar_init(&full_bar[s], 1);
      ptx::mbar_init(&empty_bar[s], NW * KQ);
    }
    *abort_flag = 0;
    ptx::fence_barrier_init();
  }
  __syncthreads();
  ptx::grid_dep_launch();
  // The row map was written by a kernel that completed before this forward's first kernel started, and
  // cache rows below pos_base are not touched by this forward: both may be read before the
  // dependency wait.  Q and the rows the QKV kernel of this layer writes may not.
  const int n_valid = p.rm.n_valid[b];
  const int kv_len = p.rm.kv_len[b];
  const int stable_keys = p.rm.pos_base[b];  // keys [0, pos_base) come from earlier forwards
  const int R = group * rps;
  bool work = !(qt * BM >= R || n_valid <= 0 || kv_len <= 0);  // rows of this tile that exist at all (uniform over the CTA)
  if (work) {  // a tile whose rows are all beyond n_valid has nothing to do (rows of one head are contiguous)
    bool any = false;
    for (int pr = qt * BM; pr < min(R, (qt + 1) * BM) && !any; pr += 1) any = (pr % rps) < n_valid;
    work = any;
  }
  if (!work) {
    ptx::grid_dep_wait();
    return;
  }
  const int n_tiles = (kv_len + KT - 1) / KT;
  const int tps = (n_tiles + p.n_splits - 1) / p.n_splits;
  const int t0 = split * tps, t1 = min(n_tiles, t0 + tps);
  const int n_my = max(t1 - t0, 0);

  const long long krow = p.k_row0 + (static_cast<long long>(b) * p.hkv + g) * p.max_seq;
  const long long vrow = p.v_row0 + (static_cast<long long>(b) * p.hkv + g) * p.max_seq;
  auto issue = [&](int i) {  // tile t0 + i into stage i % TC_STAGES
    const int s = i % TC_STAGES;
    uint8_t* st = smem + s * STAGE_BYTES;
    const int j0 = (t0 + i) * KT;
    ptx::mbar_arrive_expect_tx(&full_bar[s], STAGE_BYTES);
    ptx::tma_load_2d(st, &tmap_kv, &full_bar[s], 0, static_cast<int>(krow + j0));
    ptx::tma_load_2d(st + KT * 128, &tmap_kv, &full_bar[s], 64, static_cast<int>(krow + j0));
    ptx::tma_load_2d(st + 2 * KT * 128, &tmap_kv, &full_bar[s], 0, static_cast<int>(vrow + j0));
    ptx::tma_load_2d(st + 3 * KT * 128, &tmap_kv, &full_bar[s], 64, static_cast<int>(vrow + j0));
  };
  // first lap of the ring: tiles that lie wholly in the stable prefix are requested while the kernel
  // before this one still runs, the others after the dependency wait
  auto stable = [&](int i) { return (t0 + i + 1) * KT <= stable_keys; };
  if (threadIdx.x == 0)
    for (int i = 0; i < min(n_my, TC_STAGES); ++i)
      if (stable(i)) issue(i);
  ptx::grid_dep_wait();  // everything below reads what earlier kernels of the stream wrote
  if (threadIdx.x == 0)
    for (int i = 0; i < min(n_my, TC_STAGES); ++i)
      if (!stable(i)) issue(i);

  // ---- Q fragments of this warp's 16 packed rows (rows g4 and g4 + 8), straight from global memory
  const int pr_lo = qt * BM + warp * 16 + g4, pr_hi = pr_lo + 8;
  auto row_ptr = [&](int pr, bool& ok) -> const __nv_bfloat16* {
    const int hg = pr / rps, r = pr % rps;
    ok = pr < R && r < n_valid;
    return p.q + (static_cast<size_t>(b) * rps + r) * p.hq * 128 + (g * group + hg) * 128;
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

  float o_acc[16][4];
#pragma unroll
  for (int n = 0; n < 16; ++n)
#pragma unroll
    for (int e = 0; e < 4; ++e) o_acc[n][e] = 0.f;
  float m_lo = -INFINITY, m_hi = -INFINITY, l_lo = 0.f, l_hi = 0.f;

  // the 16 rows of a row group lie in one segment (segments are multiples of 16 rows): one key limit per warp
  const int kv_lim = row_kv_limit(p.rm, b, (qt * BM + warp * 16) % rps, kv_len);
  // ldmatrix lane roles: lanes 0-7 address matrix 0, 8-15 matrix 1, 16-23 matrix 2, 24-31 matrix 3
  const int lm_row = lane & 7, lm_mat = lane >> 3;
  bool alive = true;
  for (int i = 0; i < n_my && alive; ++i) {
    const int s = i % TC_STAGES;
    const uint32_t ph = static_cast<uint32_t>(i / TC_STAGES) & 1u;
    alive = ptx::mbar_wait(&full_bar[s], ph, abort_flag, p.error_word);
    alive = __all_sync(0xffffffffu, alive);
    if (!alive) break;
    const uint32_t sb = ptx::smem_u32(smem + s * STAGE_BYTES);
    const int j0 = (t0 + i) * KT;

    // ---- S = Q K^T for 64 keys: 8 key groups of 8, 8 k-steps of 16 over d_head
    float sc[KPW / 8][4];
#pragma unroll
    for (int n = 0; n < KPW / 8; ++n) {
      sc[n][0] = sc[n][1] = sc[n][2] = sc[n][3] = 0.f;
      const int key = kq * KPW + n * 8 + lm_row;
#pragma unroll
      for (int half = 0; half < 2; ++half) {      // K lo slab (dims 0-63), K hi slab (dims 64-127)
#pragma unroll
        for (int k2 = 0; k2 < 2; ++k2) {          // 32 dims per ldmatrix.x4 = two k-steps
          uint32_t b0, b1, b2, b3;
          ldmatrix_x4(sb + half * (KT * 128) + swz(key, k2 * 4 + lm_mat), b0, b1, b2, b3);
          const int kk = half * 4 + k2 * 2;
          mma_bf16_16816(sc[n], qa[kk], b0, b1);
          mma_bf16_16816(sc[n], qa[kk + 1], b2, b3);
        }
      }
    }
    // ---- scale, mask keys beyond kv_len, online softmax (rows g4 and g4 + 8)
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
    // a key part of the last tile may lie wholly beyond kv_len: the maximum then stays -inf, and the
    // exponentials are taken against 0 so that they come out as 0 instead of NaN
    const float mn_lo = fmaxf(m_lo, mx_lo), mn_hi = fmaxf(m_hi, mx_hi);
    const float b_lo = mn_lo == -INFINITY ? 0.f : mn_lo, b_hi = mn_hi == -INFINITY ? 0.f : mn_hi;
    const float c_lo = exp2f(m_lo - b_lo), c_hi = exp2f(m_hi - b_hi);
    m_lo = mn_lo;
    m_hi = mn_hi;
    float s_lo = 0.f, s_hi = 0.f;
    uint32_t pa[KPW / 16][4];  // P as A fragments: k-steps of 16 keys
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
    // ---- O += P V: 4 k-steps of 16 keys, 16 output groups of 8 dims
#pragma unroll
    for (int kk = 0; kk < KPW / 16; ++kk) {
      // matrices of one ldmatrix.x4.trans: (keys 0-7, dims d..d+7), (keys 8-15, same dims),
      // (keys 0-7, dims d+8..), (keys 8-15, dims d+8..)
      const int key = kq * KPW + kk * 16 + (lm_mat & 1) * 8 + lm_row;
#pragma unroll
      for (int n2 = 0; n2 < 8; ++n2) {  // 16 dims per ldmatrix
        const int chunk = n2 * 2 + (lm_mat >> 1);  // 16-byte chunk 0..15 over 128 dims
        uint32_t b0, b1, b2, b3;
        ldmatrix_x4_trans(sb + (2 + (chunk >> 3)) * (KT * 128) + swz(key, chunk & 7), b0, b1, b2, b3);
        mma_bf16_16816(o_acc[n2 * 2], pa[kk], b0, b1);
        mma_bf16_16816(o_acc[n2 * 2 + 1], pa[kk], b2, b3);
      }
    }
    // ---- release the stage; the producer thread refills it with tile i + TC_STAGES
    __syncwarp();
    if (lane == 0) ptx::mbar_arrive(&empty_bar[s]);
    if (threadIdx.x == 0 && i + TC_STAGES < n_my) {
      if (ptx::mbar_wait(&empty_bar[s], ph, abort_flag, p.error_word)) issue(i + TC_STAGES);
    }
  }
  // row sums over the quad
  l_lo += __shfl_xor_sync(0xffffffffu, l_lo, 1);
  l_lo += __shfl_xor_sync(0xffffffffu, l_lo, 2);
  l_hi += __shfl_xor_sync(0xffffffffu, l_hi, 1);
  l_hi += __shfl_xor_sync(0xffffffffu, l_hi, 2);

  auto out_ptr = [&](int pr) -> __nv_bfloat16* {
    const int hg = pr / rps, r = pr % rps;
    return p.out + (static_cast<size_t>(b) * rps + r) * p.hq * 128 + (g * group + hg) * 128;
  };
  float* red = reinterpret_cast<float*>(smem);  // [KQ][BM][PART_LD]: partial of every key part; part 0 becomes the CTA's
  if constexpr (KQ == 1) {
    if (p.n_splits == 1) {
      if (!alive) return;
      const float i_lo = 1.0f / l_lo, i_hi = 1.0f / l_hi;
      if (ok_lo) {
        __nv_bfloat16* o = out_ptr(pr_lo);
#pragma unroll
        for (int n = 0; n < 16; ++n)
          *reinterpret_cast<uint32_t*>(o + n * 8 + t4 * 2) = pack_bf16(o_acc[n][0] * i_lo, o_acc[n][1] * i_lo);
      }
      if (ok_hi) {
        __nv_bfloat16* o = out_ptr(pr_hi);
#pragma unroll
        for (int n = 0; n < 16; ++n)
          *reinterpret_cast<uint32_t*>(o + n * 8 + t4 * 2) = pack_bf16(o_acc[n][2] * i_hi, o_acc[n][3] * i_hi);
      }
      return;
    }
  }
  // ---- partials go to shared memory: merged over the key parts here, over the key splits across the cluster
  __syncthreads();  // every warp is done with the K/V stages: their memory now holds the partials
  {
    float* r_lo = red + (static_cast<size_t>(kq) * BM + warp * 16 + g4) * PART_LD;
    float* r_hi = r_lo + 8 * PART_LD;
#pragma unroll
    for (int n = 0; n < 16; ++n) {
      *reinterpret_cast<float2*>(r_lo + n * 8 + t4 * 2) = make_float2(o_acc[n][0], o_acc[n][1]);
      *reinterpret_cast<float2*>(r_hi + n * 8 + t4 * 2) = make_float2(o_acc[n][2], o_acc[n][3]);
    }
    if (t4 == 0) {
      r_lo[128] = m_lo; r_lo[129] = l_lo;  // a part or split without keys leaves m = -inf, l = 0
      r_hi[128] = m_hi; r_hi[129] = l_hi;
    }
  }
  if constexpr (KQ > 1) {
    __syncthreads();
    // one thread per (row, 4 output dims); everything is read before anything of part 0 is overwritten
    constexpr int EPT = (BM * 32 + NTHREADS - 1) / NTHREADS;
    float4 acc[EPT];
    float Ms[EPT], Ls[EPT];
#pragma unroll
    for (int j = 0; j < EPT; ++j) {
      const int e = threadIdx.x + j * NTHREADS;
      acc[j] = make_float4(0.f, 0.f, 0.f, 0.f);
      Ms[j] = -INFINITY;
      Ls[j] = 0.f;
      if (e < BM * 32) {
        const int row = e >> 5, c4 = (e & 31) * 4;
        float mq[KQ], lq[KQ];
#pragma unroll
        for (int q2 = 0; q2 < KQ; ++q2) {
          const float* r = red + (static_cast<size_t>(q2) * BM + row) * PART_LD;
          mq[q2] = r[128];
          lq[q2] = r[129];
          Ms[j] = fmaxf(Ms[j], mq[q2]);
        }
#pragma unroll
        for (int q2 = 0; q2 < KQ; ++q2) {  // key parts in index order: fixed order of the sums
          if (lq[q2] != 0.f) {
            const float w = exp2f(mq[q2] - Ms[j]);
            const float4 v = *reinterpret_cast<const float4*>(red + (static_cast<size_t>(q2) * BM + row) * PART_LD + c4);
            Ls[j] += w * lq[q2];
            acc[j].x += w * v.x; acc[j].y += w * v.y; acc[j].z += w * v.z; acc[j].w += w * v.w;
          }
        }
      }
    }
    if (p.n_splits == 1) {
      if (!alive) return;
#pragma unroll
      for (int j = 0; j < EPT; ++j) {
        const int e = threadIdx.x + j * NTHREADS;
        if (e >= BM * 32) continue;
        const int row = e >> 5, c4 = (e & 31) * 4;
        const int pr = qt * BM + row;
        if (pr >= R || (pr % rps) >= n_valid) continue;
        const float inv = 1.0f / Ls[j];
        *reinterpret_cast<uint2*>(out_ptr(pr) + c4) =
            make_uint2(pack_bf16(acc[j].x * inv, acc[j].y * inv), pack_bf16(acc[j].z * inv, acc[j].w * inv));
      }
      return;
    }
    __syncthreads();
#pragma unroll
    for (int j = 0; j < EPT; ++j) {
      const int e = threadIdx.x + j * NTHREADS;
      if (e >= BM * 32) continue;
      const int row = e >> 5, c4 = (e & 31) * 4;
      float* r = red + static_cast<size_t>(row) * PART_LD;
      *reinterpret_cast<float4*>(r + c4) = acc[j];
      if (c4 == 0) { r[128] = Ms[j]; r[129] = Ls[j]; }
    }
  }
  ptx::cluster_sync_all();
  {
    const int S = p.n_splits;
    const int rank = static_cast<int>(ptx::cluster_ctarank());
    const int rpr = (BM + S - 1) / S;  // rows per CTA of the cluster
    const int row0 = rank * rpr, row1 = min(BM, row0 + rpr);
    const uint32_t red_addr = ptx::smem_u32(red);
    for (int e = threadIdx.x; e < (row1 - row0) * 32; e += NTHREADS) {  // one thread per (row, 4 output dims)
      const int row = row0 + (e >> 5), c4 = (e & 31) * 4;
      const int pr = qt * BM + row;
      if (pr >= R || (pr % rps) >= n_valid) continue;
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
      float L = 0.f, a0 = 0.f, a1 = 0.f, a2 = 0.f, a3 = 0.f;
#pragma unroll
      for (int s2 = 0; s2 < 8; ++s2) {
        if (s2 < S && ls[s2] != 0.f) {
          const float w = exp2f(ms[s2] - M);
          L += w * ls[s2];
          a0 += w * vs[s2].x; a1 += w * vs[s2].y; a2 += w * vs[s2].z; a3 += w * vs[s2].w;
        }
      }
      const float inv = 1.0f / L;
      uint2 o2 = make_uint2(pack_bf16(a0 * inv, a1 * inv), pack_bf16(a2 * inv, a3 * inv));
      *reinterpret_cast<uint2*>(out_ptr(pr) + c4) = o2;
    }
  }
  ptx::cluster_sync_all();  // no CTA may leave while a peer still reads its partial
}

inline size_t attn_tc_smem_bytes() { return 1024 + TC_STAGES * STAGE_BYTES + 2 * TC_STAGES * 8 + 64; }

}  // namespace attn
}  // namespace d3

// bf16 matmul Y[M,N] = X[M,K] . W[N,K]^T on the sm_100a tensor cores.
//
//   * operands are staged in shared memory by TMA (128-byte swizzle, 64-element K slabs),
//   * one elected thread issues tcgen05.mma (128 x BLOCK_N x 16) into a TMEM accumulator,
//   * four epilogue warps read the accumulator back with tcgen05.ld; TMEM lane = row of X, so every
//     epilogue (residual add, SwiGLU, RoPE + cache write, softmax statistics) is thread-local.
//
// Scheduling.  The work is the list of units (output tile, 64-wide K slab), tile-major.  The grid is
// at most one CTA per SM and CTA i owns the contiguous unit range [U*i/n, U*(i+1)/n): every SM
// streams the same number of weight bytes whatever the shape.  A range is cut into segments at tile
// borders.  A segment that spans a whole tile goes straight from TMEM to its epilogue; otherwise the
// CTA writes an fp32 partial tile and bumps the tile's arrival counter, and the CTA that arrives last
// (nobody waits) sums the partials in K order and runs the epilogue, so results do not depend on
// timing.  Two TMEM accumulators alternate between segments: the epilogue of one segment overlaps the
// MMAs of the next.
//
// Dependent launch.  Weights do not depend on the previous kernel of the stream, so the producer
// fills the whole shared-memory ring with weight slabs before it executes griddepcontrol.wait, and
// only then loads the matching activation slabs; with at most ~100 KB of shared memory per CTA the
// next matmul's CTAs become resident and stream weights while the current kernel drains.
//
// Skinny case (M <= 64 rows, the batch-1 denoise step): the X box is only a_rows high, and the
// stage stride of X in shared memory shrinks with it, so that almost all of shared memory holds
// weight slabs in flight; rows a_rows..127 of the MMA's A operand then alias neighbouring stages
// and produce garbage in TMEM lanes that no one reads.
#pragma once
#include <cuda.h>

#include "common.cuh"
#include "ptx_sm100.cuh"

namespace d3 {
namespace tc {

constexpr int BLOCK_M = 128;
constexpr int BLOCK_K = 64;  // 64 bf16 = 128 bytes = one swizzle row
constexpr int UMMA_K = 16;
constexpr int NUM_THREADS = 224;  // warps 0 and 6: TMA, warp 1: MMA + TMEM owner, warps 2-5: epilogue
constexpr int MAX_CTAS = 512;     // upper bound of the grid (segment list of a tile lives in shared memory)

struct GemmParams {
  int M, N, K;
  int a_rows;       // rows of the X box: 32, 64, 96 or 128 (one row tile per unit), 256 (two)
  int stages;       // pipeline depth
  int m_tiles, n_tiles, k_chunks;
  long long total_units;  // m_tiles * n_tiles * k_chunks
  float* partial;   // partial tiles [2 * grid][row tiles per unit][BLOCK_N][128] fp32: slot 2i = CTA i's first segment, 2i+1 = its last
  int* tile_count;  // arrival counters [tiles], zero on entry and on exit
  uint32_t* error_word;
  const int* skip_flag;  // optional: non-zero -> the whole launch is a no-op
  uint32_t wait_limit_us;  // unit-range kernel: limit of every wait in microseconds (0: the default of ptx::mbar_wait)
  int stall;               // unit-range kernel, give-up path probe: the producers issue no loads at all
  int n_producers;       // 1 or 2 TMA-issuing warps
  int rr;                // 1: whole tiles dealt round-robin in a rasterised order (wide matmuls), 0: contiguous unit ranges
  int gm;                // round-robin mode: row tiles per band
  const __nv_bfloat16* w_packed;  // tiled weights (w_tiled = 1)
  long long w_blocks;             // number of 128 x 64 blocks in w_packed
  int w_tiled;           // 0: W row-major [N, K]; 1: W stored as contiguous [128 x 64] blocks, block (n_tile, kc) at
                         // row (n_tile * k_chunks + kc) * 128 of a [rows, 64] array (see pack_tiled_kernel)
  // pair kernel, optional: rows are laid out as sequences of live_rps rows (a multiple of 256) of which the first
  // live_n_valid[sequence] are in use; a 256-row tile without a live row is not computed
  const int* live_n_valid;
  int live_rps;
  EpiParams ep;
  // EPI_QKV only
  const float* rope_cos;  // [max_seq][64]
  const float* rope_sin;
  const int* pos_base;    // [bs]
  const int* n_valid;     // [bs]
  int rows_per_seq;
  int n_q_heads, n_kv_heads, max_seq;
  __nv_bfloat16* k_cache;  // this layer: [bs][n_kv_heads][max_seq][128]
  __nv_bfloat16* v_cache;
};

using namespace ptx;

// K-major operand tile in shared memory, 128-byte swizzle: rows of 128 bytes, 8-row groups 1024 bytes
// apart.  Field layout of the 64-bit matrix descriptor: start address >> 4 in bits [0,14), leading
// byte offset >> 4 in [16,30) (1 for swizzled K-major), stride byte offset >> 4 in [32,46) (1024 >> 4),
// descriptor version 1 in [46,48), swizzle mode in [61,64) (2 = 128 bytes).
__device__ __forceinline__ uint64_t make_smem_desc(uint32_t smem_addr) {
  uint64_t d = 0;
  d |= static_cast<uint64_t>((smem_addr & 0x3FFFF) >> 4);
  d |= static_cast<uint64_t>(1) << 16;
  d |= static_cast<uint64_t>(1024 >> 4) << 32;
  d |= static_cast<uint64_t>(1) << 46;
  d |= static_cast<uint64_t>(2) << 61;
  return d;
}
// Instruction descriptor for kind::f16: D fp32 (bits [4,6) = 1), A and B bf16 ([7,10) = [10,13) = 1),
// both K-major (bits 15, 16 = 0), N >> 3 in [17,23), M >> 4 in [24,29).
__host__ __device__ constexpr uint32_t make_idesc(int m, int n) {
  return (1u << 4) | (1u << 7) | (1u << 10) | (static_cast<uint32_t>(n >> 3) << 17) |
         (static_cast<uint32_t>(m >> 4) << 24);
}

__device__ __forceinline__ void epi_bar_sync() { asm volatile("bar.sync 1, 128;" ::: "memory"); }

// ----------------------------------------------------------------------------- epilogue helpers
// Source of one 32-column chunk of this thread's accumulator row: TMEM, or the sum of split-K partials.
struct TmemSource {
  uint32_t taddr_row;  // tmem base + (lane group << 16)
  __device__ __forceinline__ void load(int c, float (&v)[32]) const {
    tmem_ld_32x32(taddr_row + static_cast<uint32_t>(c), v);
    tmem_ld_wait();
  }
};
template <int SLOT_COLS>
struct PartialSource {
  const float* partial;   // workspace base; one slot = SLOT_COLS columns x 128 rows
  const int* slots;       // shared memory: partial slots of this tile's segments in K order
  int n_seg, row;
  int col0;               // first column of this row tile inside the slot
  __device__ __forceinline__ void load(int c, float (&v)[32]) const {
#pragma unroll
    for (int j = 0; j < 32; ++j) v[j] = 0.f;
    int s = 0;
    for (; s + 1 < n_seg; s += 2) {  // two segments' loads in flight; the sums stay in K order
      const float* p0 = partial + (static_cast<size_t>(slots[s]) * SLOT_COLS + col0 + c) * 128 + row;
      const float* p1 = partial + (static_cast<size_t>(slots[s + 1]) * SLOT_COLS + col0 + c) * 128 + row;
      float t0[32], t1[32];
#pragma unroll
      for (int j = 0; j < 32; ++j) t0[j] = __ldcg(p0 + j * 128);
#pragma unroll
      for (int j = 0; j < 32; ++j) t1[j] = __ldcg(p1 + j * 128);
#pragma unroll
      for (int j = 0; j < 32; ++j) v[j] = (v[j] + t0[j]) + t1[j];
    }
    if (s < n_seg) {
      const float* p0 = partial + (static_cast<size_t>(slots[s]) * SLOT_COLS + col0 + c) * 128 + row;
#pragma unroll
      for (int j = 0; j < 32; ++j) v[j] += __ldcg(p0 + j * 128);
    }
  }
};

// SiLU with the approximate division (the exact one is a long dependent sequence, and a skinny
// matmul's epilogue is one warp deep): error of a few ulp, far below the bf16 rounding of the output.
__device__ __forceinline__ float silu_fast(float g) { return __fdividef(g, 1.0f + __expf(-g)); }

// All 32 threads of a warp must call this together (the TMEM loads are warp-wide); `live` only
// predicates this thread's stores.
// Chunks (32 columns each) c_first, c_first + c_stride, ... of the tile are handled; the TMEM path
// takes them all (0, 1), the partial-sum path spreads them over the threads that share a row.
// `n_end` >= 0 ends the tile before column n_end (a column strip narrower than BLOCK_N; a multiple of
// 16, so the last chunk may be half a chunk); otherwise the tile ends with the matrix.
// `rs` multiplies the accumulator row first (the RMSNorm factor of row m when the operand was the
// un-normalised residual copy, see EpiParams; 1 otherwise).
template <int EPI, int BLOCK_N, typename Source>
__device__ __forceinline__ void run_epilogue(const Source& src, const GemmParams& p, int m, int n0, bool live,
                                             int c_first = 0, int c_stride = 1, int n_end = -1, float rs = 1.f) {
  const int N = n_end >= 0 ? n_end : p.N;
  if constexpr (EPI == EPI_F32 || EPI == EPI_RESID) {
    float* y = static_cast<float*>(p.ep.y) + static_cast<size_t>(m) * p.ep.ldy;
    for (int c = 32 * c_first; c < BLOCK_N; c += 32 * c_stride) {
      if (n0 + c >= N) break;
      float v[32];
      src.load(c, v);
      const bool vec = (n0 + c + 32 <= N) && ((p.ep.ldy & 7) == 0);
      if (!live) continue;
      const float sc = p.ep.scale * rs;
      float sq = 0.f;  // EPI_RESID: sum of squares of this chunk of the updated row
      if (vec) {
        float4* y4 = reinterpret_cast<float4*>(y + n0 + c);
        if constexpr (EPI == EPI_RESID) {
          float4 o[8];
#pragma unroll
          for (int j = 0; j < 8; ++j) o[j] = y4[j];  // all eight loads in flight
#pragma unroll
          for (int j = 0; j < 8; ++j) {
            o[j].x += v[4 * j]; o[j].y += v[4 * j + 1]; o[j].z += v[4 * j + 2]; o[j].w += v[4 * j + 3];
            y4[j] = o[j];
            sq += o[j].x * o[j].x; sq += o[j].y * o[j].y; sq += o[j].z * o[j].z; sq += o[j].w * o[j].w;
          }
          if (p.ep.yb != nullptr) {
            uint4* b4 = reinterpret_cast<uint4*>(p.ep.yb + static_cast<size_t>(m) * p.ep.ldy + n0 + c);
#pragma unroll
            for (int j = 0; j < 4; ++j) {
              __nv_bfloat162 a = __floats2bfloat162_rn(o[2 * j].x, o[2 * j].y), b = __floats2bfloat162_rn(o[2 * j].z, o[2 * j].w);
              __nv_bfloat162 cc = __floats2bfloat162_rn(o[2 * j + 1].x, o[2 * j + 1].y), d = __floats2bfloat162_rn(o[2 * j + 1].z, o[2 * j + 1].w);
              b4[j] = make_uint4(*reinterpret_cast<uint32_t*>(&a), *reinterpret_cast<uint32_t*>(&b),
                                 *reinterpret_cast<uint32_t*>(&cc), *reinterpret_cast<uint32_t*>(&d));
            }
          }
        } else {
#pragma unroll
          for (int j = 0; j < 8; ++j)
            y4[j] = make_float4(v[4 * j] * sc, v[4 * j + 1] * sc, v[4 * j + 2] * sc, v[4 * j + 3] * sc);
        }
      } else {
#pragma unroll
        for (int j = 0; j < 32; ++j) {
          int n = n0 + c + j;
          if (n < N) {
            if constexpr (EPI == EPI_RESID) {
              const float o = y[n] + v[j];
              y[n] = o;
              sq += o * o;
              if (p.ep.yb != nullptr) p.ep.yb[static_cast<size_t>(m) * p.ep.ldy + n] = __float2bfloat16_rn(o);
            } else {
              y[n] = v[j] * sc;
            }
          }
        }
      }
      if constexpr (EPI == EPI_RESID) {
        if (p.ep.ssq_out != nullptr) p.ep.ssq_out[static_cast<size_t>(m) * ((p.N + 31) / 32) + (n0 + c) / 32] = sq;
      }
    }
  } else if constexpr (EPI == EPI_T) {
    __nv_bfloat16* y = static_cast<__nv_bfloat16*>(p.ep.y) + static_cast<size_t>(m) * p.ep.ldy;
    for (int c = 32 * c_first; c < BLOCK_N; c += 32 * c_stride) {
      if (n0 + c >= N) break;
      float v[32];
      src.load(c, v);
      if (!live) continue;
#pragma unroll
      for (int j = 0; j < 32; ++j) v[j] *= rs;
      if ((n0 + c + 32 <= N) && ((p.ep.ldy & 7) == 0)) {
        uint4* y4 = reinterpret_cast<uint4*>(y + n0 + c);
#pragma unroll
        for (int j = 0; j < 4; ++j) {
          __nv_bfloat162 a = __floats2bfloat162_rn(v[8 * j], v[8 * j + 1]);
          __nv_bfloat162 b = __floats2bfloat162_rn(v[8 * j + 2], v[8 * j + 3]);
          __nv_bfloat162 cc = __floats2bfloat162_rn(v[8 * j + 4], v[8 * j + 5]);
          __nv_bfloat162 d = __floats2bfloat162_rn(v[8 * j + 6], v[8 * j + 7]);
          uint4 o;
          o.x = *reinterpret_cast<uint32_t*>(&a); o.y = *reinterpret_cast<uint32_t*>(&b);
          o.z = *reinterpret_cast<uint32_t*>(&cc); o.w = *reinterpret_cast<uint32_t*>(&d);
          y4[j] = o;
        }
      } else {
#pragma unroll
        for (int j = 0; j < 32; ++j)
          if (n0 + c + j < N) y[n0 + c + j] = __float2bfloat16_rn(v[j]);
      }
    }
  } else if constexpr (EPI == EPI_SWIGLU) {
    // packed rows of W: 2j = gate row of hidden unit j, 2j+1 = its up row; a 32-column chunk gives 16 outputs
    __nv_bfloat16* y = static_cast<__nv_bfloat16*>(p.ep.y) + static_cast<size_t>(m) * p.ep.ldy;
    const int F = N / 2;
    for (int c = 32 * c_first; c < BLOCK_N; c += 32 * c_stride) {
      if (n0 + c >= N) break;
      float v[32];
      src.load(c, v);
      if (!live) continue;
#pragma unroll
      for (int j = 0; j < 32; ++j) v[j] *= rs;
      const int h0 = (n0 + c) / 2;
      if (h0 + 16 <= F && (p.ep.ldy & 7) == 0) {
        uint32_t w[8];
#pragma unroll
        for (int q = 0; q < 8; ++q) {
          __nv_bfloat162 t = __floats2bfloat162_rn(silu_fast(v[4 * q]) * v[4 * q + 1], silu_fast(v[4 * q + 2]) * v[4 * q + 3]);
          w[q] = *reinterpret_cast<uint32_t*>(&t);
        }
        uint4* y4 = reinterpret_cast<uint4*>(y + h0);
        y4[0] = make_uint4(w[0], w[1], w[2], w[3]);
        y4[1] = make_uint4(w[4], w[5], w[6], w[7]);
      } else if (h0 + 8 == F && (p.ep.ldy & 7) == 0) {  // half a chunk: 8 outputs
        uint32_t w[4];
#pragma unroll
        for (int q = 0; q < 4; ++q) {
          __nv_bfloat162 t = __floats2bfloat162_rn(silu_fast(v[4 * q]) * v[4 * q + 1], silu_fast(v[4 * q + 2]) * v[4 * q + 3]);
          w[q] = *reinterpret_cast<uint32_t*>(&t);
        }
        *reinterpret_cast<uint4*>(y + h0) = make_uint4(w[0], w[1], w[2], w[3]);
      } else {
#pragma unroll
        for (int j = 0; j < 16; ++j)
          if (h0 + j < F) y[h0 + j] = __float2bfloat16_rn(silu_fast(v[2 * j]) * v[2 * j + 1]);
      }
    }
  } else if constexpr (EPI == EPI_STATS) {
    // one partial per 128-column tile so that the merge kernel sees the same tiling for any BLOCK_N
    static_assert(BLOCK_N % 128 == 0, "statistics epilogue works on 128-column tiles");
    for (int g = 0; g < BLOCK_N; g += 128) {
      SoftStat st = stat_empty();
      for (int c = 0; c < 128; c += 32) {
        if (n0 + g + c >= N) break;
        float v[32];
        src.load(g + c, v);
#pragma unroll
        for (int j = 0; j < 32; ++j) {
          int n = n0 + g + c + j;
          if (n < N && n != p.ep.mask_id) stat_add(st, v[j] * (p.ep.scale * rs), n);
        }
      }
      int t = (n0 + g) / 128;
      if (live && t < p.ep.n_tiles)
        p.ep.stat_part[static_cast<size_t>(m) * p.ep.n_tiles + t] = make_float4(st.m, st.z, st.s, __int_as_float(st.a));
      if (p.ep.sample_part != nullptr) {
        // temperature sampling: a second pass over the tile for the largest l + T * g; one Philox
        // call per four consecutive columns (the chunks start at multiples of 32)
        SampleStat sp = sample_empty();
        const SampleRow sr = live ? sample_row(p.ep, m) : SampleRow{0u, 0u, 0u};
        for (int c = 0; c < 128; c += 32) {
          if (n0 + g + c >= N) break;
          float v[32];
          src.load(g + c, v);
#pragma unroll
          for (int q = 0; q < 8; ++q) {
            const int nq = n0 + g + c + 4 * q;
            const uint4 bits = philox4x32_10(make_uint4(static_cast<uint32_t>(nq >> 2), sr.pos, sr.step, sr.seq), p.ep.seed_lo, p.ep.seed_hi);
            const uint32_t w[4] = {bits.x, bits.y, bits.z, bits.w};
#pragma unroll
            for (int j = 0; j < 4; ++j) {
              const int n = nq + j;
              const float l = v[4 * q + j] * (p.ep.scale * rs);
              if (n < N && n != p.ep.mask_id) sample_add(sp, __fadd_rn(l, __fmul_rn(p.ep.temperature, gumbel_from_bits(w[j]))), l, n);  // no contraction: product and sum rounded separately
            }
          }
        }
        if (live && t < p.ep.n_tiles)
          p.ep.sample_part[static_cast<size_t>(m) * p.ep.n_tiles + t] = make_float4(sp.pm, sp.la, __int_as_float(sp.pa), 0.f);
      }
    }
  } else if constexpr (EPI == EPI_QKV) {
    // d_head = 128.  Packed rows of W inside a q or k head: 2i = dim i, 2i+1 = dim i+64 (a RoPE pair);
    // v heads keep their order.  q heads first, then k heads, then v heads.
    int pos = 0, b = 0;
    if (live) {
      b = m / p.rows_per_seq;
      const int r = m % p.rows_per_seq;
      pos = p.pos_base[b] + r;
      if (r >= p.n_valid[b]) live = false;
      else if (pos < 0 || pos >= p.max_seq) {
        atomicOr(p.error_word, ERRW_BAD_POSITION);
        live = false;
      }
      if (!live) pos = 0;
    }
    const float* cs = p.rope_cos + static_cast<size_t>(pos) * 64;
    const float* sn = p.rope_sin + static_cast<size_t>(pos) * 64;
    for (int c = 32 * c_first; c < BLOCK_N; c += 32 * c_stride) {
      const int n = n0 + c;
      if (n >= N) break;
      float v[32];
      src.load(c, v);
      if (!live) continue;
#pragma unroll
      for (int j = 0; j < 32; ++j) v[j] *= rs;
      // two halves of 16 columns: a chunk that starts 16 columns before a head border spans two heads
#pragma unroll
      for (int h = 0; h < 2; ++h) {
        const int nh = n + 16 * h;
        if (nh >= N) break;
        const int head = nh / 128, off = nh % 128;
        if (head < p.n_q_heads + p.n_kv_heads) {
          __nv_bfloat16* dst;
          if (head < p.n_q_heads) {
            dst = static_cast<__nv_bfloat16*>(p.ep.y) + static_cast<size_t>(m) * p.ep.ldy + head * 128;
          } else {
            dst = p.k_cache + ((static_cast<size_t>(b) * p.n_kv_heads + (head - p.n_q_heads)) * p.max_seq + pos) * 128;
          }
          const int i0 = off / 2;  // pair index of column 0 of this half: 8 pairs, dims i0.. and 64+i0..
          // the 8 cosines and sines of this row and half in four 16-byte loads (a lane reads its own
          // table row: scalar loads would cost a cache line each)
          const float4 ca = *reinterpret_cast<const float4*>(cs + i0), cb = *reinterpret_cast<const float4*>(cs + i0 + 4);
          const float4 sa = *reinterpret_cast<const float4*>(sn + i0), sb = *reinterpret_cast<const float4*>(sn + i0 + 4);
          const float cs8[8] = {ca.x, ca.y, ca.z, ca.w, cb.x, cb.y, cb.z, cb.w};
          const float sn8[8] = {sa.x, sa.y, sa.z, sa.w, sb.x, sb.y, sb.z, sb.w};
          uint32_t lo[4], hi[4];
#pragma unroll
          for (int q = 0; q < 4; ++q) {
            float l2[2], h2[2];
#pragma unroll
            for (int e = 0; e < 2; ++e) {
              const int j = 2 * q + e;
              const float co = cs8[j], si = sn8[j];
              const float a = v[16 * h + 2 * j], bb = v[16 * h + 2 * j + 1];
              l2[e] = a * co - bb * si;
              h2[e] = bb * co + a * si;
            }
            __nv_bfloat162 tl = __floats2bfloat162_rn(l2[0], l2[1]);
            __nv_bfloat162 th = __floats2bfloat162_rn(h2[0], h2[1]);
            lo[q] = *reinterpret_cast<uint32_t*>(&tl);
            hi[q] = *reinterpret_cast<uint32_t*>(&th);
          }
          *reinterpret_cast<uint4*>(dst + i0) = make_uint4(lo[0], lo[1], lo[2], lo[3]);
          *reinterpret_cast<uint4*>(dst + 64 + i0) = make_uint4(hi[0], hi[1], hi[2], hi[3]);
        } else if (head < p.n_q_heads + 2 * p.n_kv_heads) {
          __nv_bfloat16* dst = p.v_cache +
              ((static_cast<size_t>(b) * p.n_kv_heads + (head - p.n_q_heads - p.n_kv_heads)) * p.max_seq + pos) * 128 + off;
          uint32_t w[8];
#pragma unroll
          for (int q = 0; q < 8; ++q) {
            __nv_bfloat162 t = __floats2bfloat162_rn(v[16 * h + 2 * q], v[16 * h + 2 * q + 1]);
            w[q] = *reinterpret_cast<uint32_t*>(&t);
          }
          uint4* d4 = reinterpret_cast<uint4*>(dst);
          d4[0] = make_uint4(w[0], w[1], w[2], w[3]);
          d4[1] = make_uint4(w[4], w[5], w[6], w[7]);
        }
      }
    }
  }
}

// ----------------------------------------------------------------------------- kernel
__device__ __forceinline__ long long unit_begin(long long U, int i, int n) {
  // 64-bit division is emulated (hundreds of cycles) and sits on the critical tail of split tiles
  if (U * n < 0x7fffffffll) return static_cast<long long>(static_cast<unsigned int>(U) * static_cast<unsigned int>(i) / static_cast<unsigned int>(n));
  return U * i / n;
}
// The CTA whose unit range contains unit x (ranges of CTAs without units are skipped by construction).
__device__ __forceinline__ int cta_of_unit(long long x, long long U, int n) {
  int i = (U * n < 0x7fffffffll) ? static_cast<int>(static_cast<unsigned int>(x) * static_cast<unsigned int>(n) / static_cast<unsigned int>(U))
                                 : static_cast<int>(x * n / U);
  if (i > n - 1) i = n - 1;
  while (i + 1 < n && unit_begin(U, i + 1, n) <= x) ++i;
  while (i > 0 && unit_begin(U, i, n) > x) --i;
  return i;
}

// grid = (n_ctas); dynamic shared memory (1024-byte aligned inside the kernel):
//   [stages x a_rows x 128 B]  X slabs      (stage stride a_rows*128)
//   [stages x BLOCK_N x 128 B] W slabs
//   barriers: full[stages], empty[stages], acc_full[2], acc_empty[2]; tmem address; flags; segment list
// MT = 1: one 128-row tile per unit.  MT = 2 (129..511 rows): a unit covers two row tiles that share
// the weight slab (X box of 256 rows, two MMAs per K step into two accumulators), so weights cross
// L2 and shared memory once for both; p.m_tiles then counts groups of 256 rows and p.a_rows is 256.
template <int EPI, int BLOCK_N, int MT>
__global__ void __launch_bounds__(NUM_THREADS, 2)
gemm_tc_kernel(const __grid_constant__ CUtensorMap tmap_x, const __grid_constant__ CUtensorMap tmap_w,
               const GemmParams p) {
  if (p.skip_flag != nullptr && *p.skip_flag != 0) return;  // written at least one whole graph launch earlier
  grid_dep_launch();
  extern __shared__ uint8_t smem_raw[];
  uint8_t* smem = reinterpret_cast<uint8_t*>((reinterpret_cast<uintptr_t>(smem_raw) + 1023) & ~uintptr_t(1023));
  const int stages = p.stages;
  const uint32_t a_stage_bytes = static_cast<uint32_t>(p.a_rows) * 128u;
  constexpr uint32_t b_stage_bytes = BLOCK_N * 128u;
  uint8_t* smem_a = smem;
  uint8_t* smem_b = smem + static_cast<size_t>(stages) * a_stage_bytes;
  uint64_t* full_bar = reinterpret_cast<uint64_t*>(smem_b + static_cast<size_t>(stages) * b_stage_bytes);
  uint64_t* empty_bar = full_bar + stages;
  uint64_t* acc_full = empty_bar + stages;
  uint64_t* acc_empty = acc_full + 2;
  uint32_t* tmem_slot = reinterpret_cast<uint32_t*>(acc_empty + 2);
  volatile int* abort_flag = reinterpret_cast<volatile int*>(tmem_slot + 1);
  int* last_flag = const_cast<int*>(abort_flag) + 1;  // 0: not last, else number of segments of the tile
  int* list_len = last_flag + 1;                       // number of segments of the tile being finished
  int* seg_slots = last_flag + 2;                      // [MAX_CTAS]

  const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
  const int cta = blockIdx.x, n_cta = gridDim.x;
  const uint64_t wait_ns = p.wait_limit_us != 0 ? static_cast<uint64_t>(p.wait_limit_us) * 1000ull : WAIT_LIMIT_NS;
  const long long U = p.total_units;
  const int KC = p.k_chunks;
  // Unit range of this CTA.  Round-robin mode (wide matmuls): the CTA owns whole tiles cta, cta + n,
  // cta + 2n, ... of a rasterised tile order, numbered here 0, 1, 2, ... (see tile_mn below).
  const int n_tiles_all = p.m_tiles * p.n_tiles;
  const int my_tiles = p.rr ? (cta < n_tiles_all ? (n_tiles_all - cta + n_cta - 1) / n_cta : 0) : 0;
  const long long u0 = p.rr ? 0 : unit_begin(U, cta, n_cta);
  const long long u1 = p.rr ? static_cast<long long>(my_tiles) * KC : unit_begin(U, cta + 1, n_cta);
  // Row tile (group) and column tile of a tile index.  Contiguous mode: row tiles fastest.  Round-robin
  // mode: the CTAs running at the same time work on neighbouring tiles of bands of p.gm row tiles, so
  // a weight tile is fetched from HBM once and shared through L2 by the CTAs of its band column, and
  // an activation tile by the CTAs of its band row.
  auto tile_mn = [&](int t, int& m_t, int& n_t) {
    if (p.rr) {
      const int q = cta + t * n_cta;
      const int band_sz = p.gm * p.n_tiles;
      const int band = q / band_sz, r = q - band * band_sz;
      const int rows_here = (p.m_tiles - band * p.gm) < p.gm ? (p.m_tiles - band * p.gm) : p.gm;
      n_t = r / rows_here;
      m_t = band * p.gm + r % rows_here;
    } else {
      m_t = t % p.m_tiles;
      n_t = t / p.m_tiles;
    }
  };
  constexpr uint32_t TMEM_COLS = 2 * MT * BLOCK_N;  // 256 or 512: a power of two >= 32
  static_assert(TMEM_COLS <= 512, "two accumulators of MT row tiles must fit tensor memory");

  if (threadIdx.x == 0) {
    prefetch_tensormap(&tmap_x);
    prefetch_tensormap(&tmap_w);
    for (int s = 0; s < stages; ++s) {
      mbar_init(&full_bar[s], 1);
      mbar_init(&empty_bar[s], 1);
    }
    for (int b = 0; b < 2; ++b) {
      mbar_init(&acc_full[b], 1);
      mbar_init(&acc_empty[b], 128);
    }
    *abort_flag = 0;
    *last_flag = 0;
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

  if (warp == 0 || warp == 6) {
    // ---------------- TMA producers: warp 0 alone, or warps 0 and 6 taking alternate units
    const int n_prod = p.n_producers, pi = warp == 0 ? 0 : 1;
    if (lane == 0 && pi < n_prod && !p.stall) {
      const uint32_t tx = a_stage_bytes + b_stage_bytes;
      const long long n_total = u1 - u0;
      // Arms the stage's barrier with the bytes that will arrive and issues the weight loads.
      auto load_w = [&](int s, int n_tile, int kc) {
        uint8_t* dst = smem_b + static_cast<size_t>(s) * b_stage_bytes;
        if (p.w_tiled) {
          // one contiguous, pre-swizzled 16 KB block per 128 weight rows; a 256-wide tile at the
          // ragged end of N may have only its first block (the other half of the stage keeps stale
          // data, which lands in output columns >= N that nobody stores)
          const long long blk0 = static_cast<long long>(n_tile * (BLOCK_N / 128)) * KC + kc;
          int nb = 0;
#pragma unroll
          for (int h = 0; h < BLOCK_N / 128; ++h)
            if (blk0 + static_cast<long long>(h) * KC < p.w_blocks) ++nb;
          mbar_arrive_expect_tx(&full_bar[s], a_stage_bytes + static_cast<uint32_t>(nb) * 128u * 128u);
#pragma unroll
          for (int h = 0; h < BLOCK_N / 128; ++h)
            if (h < nb)
              bulk_load_1d(dst + h * 128 * 128, p.w_packed + (blk0 + static_cast<long long>(h) * KC) * (128 * 64),
                           128 * 128, &full_bar[s]);
        } else {
          mbar_arrive_expect_tx(&full_bar[s], tx);
          tma_load_2d(dst, &tmap_w, &full_bar[s], kc * BLOCK_K, n_tile * BLOCK_N);
        }
      };
      const int pre = static_cast<int>(n_total < stages ? n_total : stages);
      // These loops run once per K slab in a single thread and pace the CTA: (tile, K slab) and
      // (stage, parity) are running counters, no division per slab.
      const int tile0 = static_cast<int>(u0 / KC);
      const int kc_first = static_cast<int>(u0 - static_cast<long long>(tile0) * KC);
      // weights first: they do not depend on the kernels before this one
      int m_t = 0, n_t = 0, mn_of = -1;  // row and column tile of tile `mn_of`
      {
        int tile = tile0, kc = kc_first + pi;
        while (kc >= KC) { kc -= KC; ++tile; }
        for (int i = pi; i < pre; i += n_prod) {
          if (tile != mn_of) { tile_mn(tile, m_t, n_t); mn_of = tile; }
          load_w(i, n_t, kc);
          kc += n_prod;
          while (kc >= KC) { kc -= KC; ++tile; }
        }
      }
      grid_dep_wait();
      int tile = tile0, kc = kc_first + pi;
      while (kc >= KC) { kc -= KC; ++tile; }
      for (int i = pi; i < pre; i += n_prod) {
        if (tile != mn_of) { tile_mn(tile, m_t, n_t); mn_of = tile; }
        tma_load_2d(smem_a + static_cast<size_t>(i) * a_stage_bytes, &tmap_x, &full_bar[i], kc * BLOCK_K, m_t * (MT * BLOCK_M));
        kc += n_prod;
        while (kc >= KC) { kc -= KC; ++tile; }
      }
      // (tile, kc) now name unit `first`, the first one past the prefetched ring that is this producer's
      long long i = pre;
      while (i % n_prod != pi) ++i;
      int s = static_cast<int>(i % stages);
      uint32_t ph = (static_cast<uint32_t>(i / stages) & 1u) ^ 1u;  // parity to wait for on the empty barrier
      for (; i < n_total; i += n_prod) {
        if (!mbar_wait(&empty_bar[s], ph, abort_flag, p.error_word, wait_ns)) break;
        if (tile != mn_of) { tile_mn(tile, m_t, n_t); mn_of = tile; }
        load_w(s, n_t, kc);
        tma_load_2d(smem_a + static_cast<size_t>(s) * a_stage_bytes, &tmap_x, &full_bar[s], kc * BLOCK_K, m_t * (MT * BLOCK_M));
        kc += n_prod;
        while (kc >= KC) { kc -= KC; ++tile; }
        s += n_prod;
        if (s >= stages) { s -= stages; ph ^= 1u; }
      }
    } else if (lane == 0) {
      grid_dep_wait();
    }
  } else if (warp == 1) {
    // ---------------- MMA issuer
    if (lane == 0) {
      constexpr uint32_t idesc = make_idesc(BLOCK_M, BLOCK_N);
      const uint64_t adesc0 = make_smem_desc(smem_u32(smem_a)), bdesc0 = make_smem_desc(smem_u32(smem_b));
      const uint64_t a_step = a_stage_bytes >> 4, b_step = b_stage_bytes >> 4;  // stage strides in descriptor units
      uint64_t adesc = adesc0, bdesc = bdesc0;
      int s = 0;
      uint32_t ph = 0;
      int seg = 0;
      bool ok = true;
      int tile = static_cast<int>(u0 / KC);
      int kc0 = static_cast<int>(u0 - static_cast<long long>(tile) * KC);
      for (long long u = u0; u < u1 && ok; ++seg) {
        const long long left = u1 - u;
        const int n_k = static_cast<int>(left < KC - kc0 ? left : KC - kc0);
        const int buf = seg & 1;
        // the epilogue must have drained this accumulator (two segments ago)
        if (!mbar_wait(&acc_empty[buf], (static_cast<uint32_t>(seg >> 1) & 1u) ^ 1u, abort_flag, p.error_word, wait_ns)) break;
        tc_fence_after();
        const uint32_t tmem_d = tmem_base + static_cast<uint32_t>(buf * MT * BLOCK_N);
        for (int j = 0; j < n_k; ++j) {
          if (!mbar_wait(&full_bar[s], ph, abort_flag, p.error_word, wait_ns)) { ok = false; break; }
          tc_fence_after();
#pragma unroll
          for (int kk = 0; kk < BLOCK_K / UMMA_K; ++kk) {
            // advancing K by 16 bf16 = 32 bytes inside the swizzled row: +2 in the (>>4) address field
#pragma unroll
            for (int mt = 0; mt < MT; ++mt)  // row tile mt: 128 rows = 16 KB further down the X stage
              umma_bf16(tmem_d + static_cast<uint32_t>(mt * BLOCK_N), adesc + static_cast<uint64_t>(2 * kk + mt * 1024),
                        bdesc + static_cast<uint64_t>(2 * kk), idesc, (j > 0 || kk > 0) ? 1u : 0u);
          }
          umma_commit(&empty_bar[s]);  // frees the stage once these MMAs have read it
          adesc += a_step;
          bdesc += b_step;
          if (++s == stages) { s = 0; ph ^= 1u; adesc = adesc0; bdesc = bdesc0; }
        }
        if (ok) umma_commit(&acc_full[buf]);  // this segment's accumulator is complete
        u += n_k;
        ++tile;  // a segment ends at a tile border or at the end of the range
        kc0 = 0;
      }
    }
  } else {
    // ---------------- epilogue warps: TMEM lane group = warp % 4
    grid_dep_wait();  // residual rows, positions and counters come from earlier kernels
    const int lg = warp & 3;
    const int row = lg * 32 + lane;
    const int et = threadIdx.x - 64;  // 0..127
    int seg = 0;
    for (long long u = u0; u < u1; ++seg) {
      const int tile = static_cast<int>(u / KC);
      const int kc0 = static_cast<int>(u - static_cast<long long>(tile) * KC);
      const long long left = u1 - u;
      const int n_k = static_cast<int>(left < KC - kc0 ? left : KC - kc0);
      u += n_k;
      const int buf = seg & 1;
      int m_group, n_tile;
      tile_mn(tile, m_group, n_tile);
      const int n0 = n_tile * BLOCK_N;
      if (n_k != KC && et == 0) {
        // split tile: its segments in K order (the CTAs whose ranges meet [tile*KC, (tile+1)*KC)),
        // worked out while the MMAs of this segment still run
        const long long t_lo = static_cast<long long>(tile) * KC, t_hi = t_lo + KC;
        const int i_lo = cta_of_unit(t_lo, U, n_cta), i_hi = cta_of_unit(t_hi - 1, U, n_cta);
        int n_list = 0;
        for (int i = i_lo; i <= i_hi; ++i) {
          const long long a = unit_begin(U, i, n_cta), b = unit_begin(U, i + 1, n_cta);
          const long long lo = a > t_lo ? a : t_lo, hi = b < t_hi ? b : t_hi;
          if (lo < hi) seg_slots[n_list++] = 2 * i + (lo == t_lo ? 1 : 0);
        }
        *list_len = n_list;
      }
      const int rows_pad = p.a_rows < 128 ? p.a_rows : 128;  // rows of one row tile that can be live
      // Row factors (folded RMSNorm) of the rows this thread may finish, fetched while the MMAs of the
      // segment still run: its TMEM lane's row for a whole tile, row et % rows_pad when the partial
      // sums of a split tile are spread over the threads.
      float rs_tmem[MT], rs_part[MT];
#pragma unroll
      for (int mt = 0; mt < MT; ++mt) {
        rs_tmem[mt] = 1.f;
        rs_part[mt] = 1.f;
        if (p.ep.ssq_in != nullptr) {
          const int m_tile = m_group * MT + mt;
          if (n_k == KC || EPI == EPI_STATS) {
            const int m = m_tile * BLOCK_M + row;
            if (lg * 32 < rows_pad && m < p.M) rs_tmem[mt] = row_rstd(p.ep, m);
          } else {
            const int m2 = m_tile * BLOCK_M + et % rows_pad;
            if (et / rows_pad < 128 / rows_pad && m2 < p.M) rs_part[mt] = row_rstd(p.ep, m2);
          }
        }
      }
      bool ok = mbar_wait(&acc_full[buf], static_cast<uint32_t>(seg >> 1) & 1u, abort_flag, p.error_word, wait_ns);
      ok = __all_sync(0xffffffffu, ok);
      if (!ok) break;
      tc_fence_after();
      const uint32_t tmem_seg = tmem_base + static_cast<uint32_t>(buf * MT * BLOCK_N) + (static_cast<uint32_t>(lg * 32) << 16);
      if (n_k == KC) {
#pragma unroll
        for (int mt = 0; mt < MT; ++mt) {
          const int m_tile = m_group * MT + mt;
          const int m = m_tile * BLOCK_M + row;
          // warp-uniform: does this lane group hold any row of X at all?
          const bool warp_live = (lg * 32 < rows_pad) && (m_tile * BLOCK_M + lg * 32 < p.M);
          TmemSource tsrc{tmem_seg + static_cast<uint32_t>(mt * BLOCK_N)};
          if (warp_live) run_epilogue<EPI, BLOCK_N>(tsrc, p, m, n0, m < p.M, 0, 1, -1, rs_tmem[mt]);
        }
        tc_fence_before();
        mbar_arrive(&acc_empty[buf]);
        continue;
      }
      // partial tile: park it, then let the last arrival finish the tile
      const int my_slot = 2 * cta + (kc0 == 0 ? 1 : 0);  // a segment starting at K = 0 is this CTA's last one
#pragma unroll
      for (int mt = 0; mt < MT; ++mt) {
        const int m_tile = m_group * MT + mt;
        const bool warp_live = (lg * 32 < rows_pad) && (m_tile * BLOCK_M + lg * 32 < p.M);
        if (warp_live) {
          TmemSource tsrc{tmem_seg + static_cast<uint32_t>(mt * BLOCK_N)};
          float* mine = p.partial + (static_cast<size_t>(my_slot) * MT + mt) * BLOCK_N * 128 + row;
          for (int c = 0; c < BLOCK_N; c += 32) {
            float v[32];
            tsrc.load(c, v);
#pragma unroll
            for (int j = 0; j < 32; ++j) mine[static_cast<size_t>(c + j) * 128] = v[j];
          }
        }
      }
      tc_fence_before();
      mbar_arrive(&acc_empty[buf]);
      epi_bar_sync();  // every thread's partial stores are ordered before thread 0's release below
      if (et == 0) {
        const int n_list = *list_len;
        int old;  // release: the partial is visible to whoever sees the count; acquire: so are the others'
        asm volatile("atom.add.acq_rel.gpu.global.s32 %0, [%1], 1;" : "=r"(old) : "l"(&p.tile_count[tile]) : "memory");
        const int last = (old == n_list - 1) ? n_list : 0;
        if (last) p.tile_count[tile] = 0;  // ready for the next launch
        *last_flag = last;
      }
      epi_bar_sync();
      const int n_seg = *last_flag;
      if (n_seg > 0) {
#pragma unroll
        for (int mt = 0; mt < MT; ++mt) {
          const int m_tile = m_group * MT + mt;
          if (m_tile * BLOCK_M >= p.M) break;
          if constexpr (EPI == EPI_STATS) {  // one statistic per (row, 128 columns): a row stays with one thread
            const bool warp_live = (lg * 32 < rows_pad) && (m_tile * BLOCK_M + lg * 32 < p.M);
            if (warp_live) {
              const int m = m_tile * BLOCK_M + row;
              PartialSource<MT * BLOCK_N> psrc{p.partial, seg_slots, n_seg, row, mt * BLOCK_N};
              run_epilogue<EPI, BLOCK_N>(psrc, p, m, n0, m < p.M, 0, 1, -1, rs_tmem[mt]);
            }
          } else {
            // the sums come from memory, not from TMEM lanes: spread (row, 32-column chunk) pairs over
            // all 128 threads so that a 32-row matmul does not leave the reduction to one warp
            const int tpr = 128 / rows_pad;  // threads per row: 4, 2, 1, 1 for 32, 64, 96, 128 rows
            const int prow = et % rows_pad, part = et / rows_pad;
            if (part < tpr) {
              const int m2 = m_tile * BLOCK_M + prow;
              PartialSource<MT * BLOCK_N> psrc{p.partial, seg_slots, n_seg, prow, mt * BLOCK_N};
              run_epilogue<EPI, BLOCK_N>(psrc, p, m2, n0, m2 < p.M, part, tpr, -1, rs_part[mt]);
            }
          }
        }
      }
      epi_bar_sync();  // seg_slots and last_flag are reused by the next segment
    }
    tc_fence_before();
  }
  __syncthreads();
  if (warp == 1) {
    tc_fence_after();
    tmem_dealloc<TMEM_COLS>(tmem_base);
  }
}

// ----------------------------------------------------------------------------- cluster K-split kernel
// Matmuls of up to 256 rows (one or two row tiles of a_rows <= 128 rows, 128-column tiles) with an
// elementwise epilogue (fp32, bf16 or residual output).  The grid is made of clusters of C CTAs (C = 1..8).  A cluster owns whole output
// tiles; inside it every CTA takes one C-th of the K range of each tile, so all C partial
// accumulators of a tile are complete at about the same time.  They meet in distributed shared
// memory: a tile is cut into units of 16 rows x 32 columns, unit u belongs to CTA u mod C, and every
// CTA pushes its partial of each unit into the owner's shared memory (remote stores), then arrives
// on the owner's barrier (release at cluster scope).  An owner waits for its C arrivals, adds the
// partials in rank order (fixed order: reproducible bits) with one (row, 4 columns) element per
// thread, and runs the epilogue.  Nobody reads another CTA's memory, so a CTA leaves as soon as it
// has pushed its partials and finished its own units; no global workspace, no atomics.
struct ClusterSplit {
  int C;           // CTAs per cluster
  int n_clusters;  // clusters that have tiles
};

// grid = (n_clusters * C), cluster dims (C, 1, 1).  Dynamic shared memory as in gemm_tc_kernel, plus
// the receive buffer [units per owner][C sources][16 rows][32 columns] fp32 and the two cluster barriers.
template <int EPI>
__global__ void __launch_bounds__(NUM_THREADS, 2)
gemm_ck_kernel(const __grid_constant__ CUtensorMap tmap_x, const __grid_constant__ CUtensorMap tmap_w,
               const GemmParams p, const ClusterSplit cs) {
  constexpr int BLOCK_N = 128;
  if (p.skip_flag != nullptr && *p.skip_flag != 0) return;
  grid_dep_launch();
  extern __shared__ uint8_t smem_raw[];
  uint8_t* smem = reinterpret_cast<uint8_t*>((reinterpret_cast<uintptr_t>(smem_raw) + 1023) & ~uintptr_t(1023));
  const int stages = p.stages;
  const uint32_t a_stage_bytes = static_cast<uint32_t>(p.a_rows) * 128u;
  constexpr uint32_t b_stage_bytes = BLOCK_N * 128u;
  uint8_t* smem_a = smem;
  uint8_t* smem_b = smem + static_cast<size_t>(stages) * a_stage_bytes;
  float* recv = reinterpret_cast<float*>(smem_b + static_cast<size_t>(stages) * b_stage_bytes);
  const int n_units = 4 * (p.a_rows / 16);             // 16-row x 32-column units of a tile
  const int units_per_owner = (n_units + cs.C - 1) / cs.C;
  uint64_t* full_bar = reinterpret_cast<uint64_t*>(recv + static_cast<size_t>(units_per_owner) * cs.C * 512);
  uint64_t* empty_bar = full_bar + stages;
  uint64_t* acc_full = empty_bar + stages;
  uint64_t* acc_empty = acc_full + 2;
  uint64_t* ready_bar = acc_empty + 2;  // all C partials of this CTA's units of the current tile have arrived
  uint64_t* free_bar = ready_bar + 1;   // every owner has added up the previous tile: its buffers may be overwritten
  uint32_t* tmem_slot = reinterpret_cast<uint32_t*>(free_bar + 1);
  volatile int* abort_flag = reinterpret_cast<volatile int*>(tmem_slot + 1);

  const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
  const int C = cs.C;
  const int rank = static_cast<int>(cluster_ctarank());
  const int cluster = blockIdx.x / C;
  const int T = p.m_tiles * p.n_tiles;  // tile t: row tile t % m_tiles, column tile t / m_tiles (the row tiles of a
                                        // column tile run side by side and share its weights through L2)
  const int KC = p.k_chunks;
  const int t0 = static_cast<int>(static_cast<long long>(T) * cluster / cs.n_clusters);
  const int t1 = static_cast<int>(static_cast<long long>(T) * (cluster + 1) / cs.n_clusters);
  const int kc0 = KC * rank / C, kc1 = KC * (rank + 1) / C;  // C <= KC: never empty
  const int n_k = kc1 - kc0;
  const long long n_total = static_cast<long long>(t1 - t0) * n_k;
  constexpr uint32_t TMEM_COLS = 2 * BLOCK_N;

  if (threadIdx.x == 0) {
    prefetch_tensormap(&tmap_x);
    if (!p.w_tiled) prefetch_tensormap(&tmap_w);
    for (int s = 0; s < stages; ++s) {
      mbar_init(&full_bar[s], 1);
      mbar_init(&empty_bar[s], 1);
    }
    for (int b = 0; b < 2; ++b) {
      mbar_init(&acc_full[b], 1);
      mbar_init(&acc_empty[b], 128);
    }
    mbar_init(ready_bar, static_cast<uint32_t>(C));
    mbar_init(free_bar, static_cast<uint32_t>(n_units < C ? n_units : C));  // one arrival per owner
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

  if (warp == 0 || warp == 6) {
    // ---------------- TMA producers: alternate units
    const int pi = warp == 0 ? 0 : 1;
    if (lane == 0) {
      const uint32_t tx = a_stage_bytes + b_stage_bytes;
      // unit i of this CTA = (tile t0 + i / n_k, slab kc0 + i % n_k), kept as running counters (no
      // division per slab: these single-thread loops pace the CTA)
      auto advance = [&](int& n_tile, int& k, int by) {
        k += by;
        while (k >= n_k) { k -= n_k; ++n_tile; }
      };
      auto load_w = [&](int s, int n_tile, int kc) {
        uint8_t* dst = smem_b + static_cast<size_t>(s) * b_stage_bytes;
        mbar_arrive_expect_tx(&full_bar[s], tx);
        if (p.w_tiled) bulk_load_1d(dst, p.w_packed + (static_cast<long long>(n_tile) * KC + kc) * (128 * 64), 128 * 128, &full_bar[s]);
        else tma_load_2d(dst, &tmap_w, &full_bar[s], kc * BLOCK_K, n_tile * BLOCK_N);
      };
      const int pre = static_cast<int>(n_total < stages ? n_total : stages);
      const int MTL = p.m_tiles;
      {
        int n_tile = t0, k = 0;
        advance(n_tile, k, pi);
        for (int i = pi; i < pre; i += 2) {  // weights first: they do not depend on the kernels before this one
          load_w(i, n_tile / MTL, kc0 + k);
          advance(n_tile, k, 2);
        }
      }
      grid_dep_wait();
      int n_tile = t0, k = 0;
      advance(n_tile, k, pi);
      for (int i = pi; i < pre; i += 2) {
        tma_load_2d(smem_a + static_cast<size_t>(i) * a_stage_bytes, &tmap_x, &full_bar[i], (kc0 + k) * BLOCK_K, (n_tile % MTL) * BLOCK_M);
        advance(n_tile, k, 2);
      }
      long long i = pre;
      if ((i & 1) != pi) ++i;
      int s = static_cast<int>(i % stages);
      uint32_t ph = (static_cast<uint32_t>(i / stages) & 1u) ^ 1u;  // parity to wait for on the empty barrier
      for (; i < n_total; i += 2) {
        if (!mbar_wait(&empty_bar[s], ph, abort_flag, p.error_word)) break;
        load_w(s, n_tile / MTL, kc0 + k);
        tma_load_2d(smem_a + static_cast<size_t>(s) * a_stage_bytes, &tmap_x, &full_bar[s], (kc0 + k) * BLOCK_K, (n_tile % MTL) * BLOCK_M);
        advance(n_tile, k, 2);
        s += 2;
        if (s >= stages) { s -= stages; ph ^= 1u; }
      }
    }
  } else if (warp == 1) {
    // ---------------- MMA issuer: one accumulator per tile, alternating TMEM halves
    if (lane == 0) {
      constexpr uint32_t idesc = make_idesc(BLOCK_M, BLOCK_N);
      const uint64_t adesc0 = make_smem_desc(smem_u32(smem_a)), bdesc0 = make_smem_desc(smem_u32(smem_b));
      const uint64_t a_step = a_stage_bytes >> 4, b_step = b_stage_bytes >> 4;
      uint64_t adesc = adesc0, bdesc = bdesc0;
      int s = 0;
      uint32_t ph = 0;
      bool ok = true;
      for (int t = t0; t < t1 && ok; ++t) {
        const int seg = t - t0, buf = seg & 1;
        if (!mbar_wait(&acc_empty[buf], (static_cast<uint32_t>(seg >> 1) & 1u) ^ 1u, abort_flag, p.error_word)) break;
        tc_fence_after();
        const uint32_t tmem_d = tmem_base + static_cast<uint32_t>(buf * BLOCK_N);
        for (int k = 0; k < n_k; ++k) {
          if (!mbar_wait(&full_bar[s], ph, abort_flag, p.error_word)) { ok = false; break; }
          tc_fence_after();
#pragma unroll
          for (int kk = 0; kk < BLOCK_K / UMMA_K; ++kk)
            umma_bf16(tmem_d, adesc + static_cast<uint64_t>(2 * kk), bdesc + static_cast<uint64_t>(2 * kk), idesc,
                      (k > 0 || kk > 0) ? 1u : 0u);
          umma_commit(&empty_bar[s]);
          adesc += a_step;
          bdesc += b_step;
          if (++s == stages) { s = 0; ph ^= 1u; adesc = adesc0; bdesc = bdesc0; }
        }
        if (ok) umma_commit(&acc_full[buf]);
      }
    }
  } else {
    // ---------------- epilogue warps
    grid_dep_wait();
    const int lg = warp & 3;
    const int row = lg * 32 + lane;
    const int et = threadIdx.x - 64;  // 0..127
    const bool warp_live = lg * 32 < p.a_rows;  // this warp's TMEM lanes hold rows of X (zero rows beyond M)
    const uint32_t recv_addr = smem_u32(recv);
    const int RS = p.a_rows / 16;     // row slices of a tile
    const int n_owners = n_units < C ? n_units : C;
    const int n_tiles_mine = t1 - t0;
    // as an owner: element (row e_row of the unit, columns 4 * e_j ..) of every unit of this CTA
    const int e_j = et & 7, e_row = et >> 3;
    bool alive = true;
    int seg = 0;
    for (int t = t0; t < t1; ++t, ++seg) {
      const int buf = seg & 1;
      const int n0 = (t / p.m_tiles) * BLOCK_N;
      const int m0 = (t % p.m_tiles) * BLOCK_M;  // first row of this row tile
      // the residual values this thread will update (first unit): in flight while the MMAs still run
      float4 y_pre = make_float4(0.f, 0.f, 0.f, 0.f);
      bool y_pre_ok = false;
      if constexpr (EPI == EPI_RESID) {
        if (rank < n_units) {
          const int c = rank / RS, m = m0 + (rank % RS) * 16 + e_row, n = n0 + c * 32 + e_j * 4;
          if (m < p.M && n + 4 <= p.N && (p.ep.ldy & 3) == 0) {
            y_pre = *reinterpret_cast<const float4*>(static_cast<const float*>(p.ep.y) + static_cast<size_t>(m) * p.ep.ldy + n);
            y_pre_ok = true;
          }
        }
      }
      float rs = 1.f;  // row factor (folded RMSNorm) of this thread's row of its first unit; others are fetched later
      if (EPI != EPI_RESID && p.ep.ssq_in != nullptr && rank < n_units) {
        const int m = m0 + (rank % RS) * 16 + e_row;
        if (m < p.M) rs = row_rstd(p.ep, m);
      }
      bool ok = mbar_wait(&acc_full[buf], static_cast<uint32_t>(seg >> 1) & 1u, abort_flag, p.error_word);
      // the owners must have added up the previous tile before their buffers are overwritten
      if (ok && seg > 0) ok = mbar_wait_cluster(free_bar, static_cast<uint32_t>(seg - 1) & 1u, abort_flag, p.error_word);
      ok = __all_sync(0xffffffffu, ok);
      if (!ok) { alive = false; break; }
      tc_fence_after();
      if (warp_live) {
        // push this lane's row of every 32-column chunk to the chunk's owner:
        // receive buffer [slot][source rank][16 rows][8 groups of 4 columns]
        TmemSource tsrc{tmem_base + static_cast<uint32_t>(buf * BLOCK_N) + (static_cast<uint32_t>(lg * 32) << 16)};
#pragma unroll 1
        for (int c = 0; c < 4; ++c) {
          float v[32];
          tsrc.load(c * 32, v);
          const int u = c * RS + (row >> 4);
          const int owner = u % C, slot = u / C;
          const uint32_t dst = map_to_cta(recv_addr + static_cast<uint32_t>(((slot * C + rank) * 16 + (row & 15)) * 128), static_cast<uint32_t>(owner));
#pragma unroll
          for (int j = 0; j < 8; ++j) st_cluster_f4(dst + j * 16, v[4 * j], v[4 * j + 1], v[4 * j + 2], v[4 * j + 3]);
        }
      }
      tc_fence_before();
      mbar_arrive(&acc_empty[buf]);
      epi_bar_sync();  // every pushing thread's stores are ordered before the arrivals below
      if (et < n_owners) mbar_arrive_remote(ready_bar, static_cast<uint32_t>(et));
      if (rank < n_units) {
        // ---- owner: wait for the C partials of its units, add them in rank order, epilogue
        ok = mbar_wait_cluster(ready_bar, static_cast<uint32_t>(seg) & 1u, abort_flag, p.error_word);
        ok = __all_sync(0xffffffffu, ok);
        if (!ok) { alive = false; break; }
        for (int slot = 0, u = rank; u < n_units; ++slot, u += C) {
          const int c = u / RS;
          const int m = m0 + (u % RS) * 16 + e_row, n = n0 + c * 32 + e_j * 4;
          float4 acc = make_float4(0.f, 0.f, 0.f, 0.f);
          const float4* src = reinterpret_cast<const float4*>(recv) + (static_cast<size_t>(slot) * C * 16 + e_row) * 8 + e_j;
          for (int s2 = 0; s2 < C; ++s2) {
            const float4 w = src[static_cast<size_t>(s2) * 128];
            acc.x += w.x; acc.y += w.y; acc.z += w.z; acc.w += w.w;
          }
          const bool live = m < p.M;
          const bool vec = n + 4 <= p.N && (p.ep.ldy & 3) == 0;
          if constexpr (EPI == EPI_RESID) {
            float* y = static_cast<float*>(p.ep.y) + static_cast<size_t>(m) * p.ep.ldy;
            float sq = 0.f;
            if (live) {
              if (vec) {
                const float4 o0 = (slot == 0 && y_pre_ok) ? y_pre : *reinterpret_cast<const float4*>(y + n);
                const float4 o = make_float4(o0.x + acc.x, o0.y + acc.y, o0.z + acc.z, o0.w + acc.w);
                *reinterpret_cast<float4*>(y + n) = o;
                sq = ((o.x * o.x + o.y * o.y) + o.z * o.z) + o.w * o.w;
                if (p.ep.yb != nullptr) {
                  __nv_bfloat162 lo = __floats2bfloat162_rn(o.x, o.y), hi = __floats2bfloat162_rn(o.z, o.w);
                  *reinterpret_cast<uint2*>(p.ep.yb + static_cast<size_t>(m) * p.ep.ldy + n) =
                      make_uint2(*reinterpret_cast<uint32_t*>(&lo), *reinterpret_cast<uint32_t*>(&hi));
                }
              } else {
                const float a4[4] = {acc.x, acc.y, acc.z, acc.w};
#pragma unroll
                for (int q = 0; q < 4; ++q) {
                  if (n + q < p.N) {
                    const float o = y[n + q] + a4[q];
                    y[n + q] = o;
                    sq += o * o;
                    if (p.ep.yb != nullptr) p.ep.yb[static_cast<size_t>(m) * p.ep.ldy + n + q] = __float2bfloat16_rn(o);
                  }
                }
              }
            }
            // the 8 threads of a row are 8 neighbouring lanes: chunk sum of squares in a fixed tree
            sq += __shfl_xor_sync(0xffffffffu, sq, 1);
            sq += __shfl_xor_sync(0xffffffffu, sq, 2);
            sq += __shfl_xor_sync(0xffffffffu, sq, 4);
            if (live && e_j == 0 && p.ep.ssq_out != nullptr && n0 + c * 32 < p.N)
              p.ep.ssq_out[static_cast<size_t>(m) * ((p.N + 31) / 32) + (n0 + c * 32) / 32] = sq;
          } else {
            if (slot > 0 && p.ep.ssq_in != nullptr && live) rs = row_rstd(p.ep, m);
            const float sc = (EPI == EPI_F32 ? p.ep.scale : 1.f) * rs;
            const float a4[4] = {acc.x * sc, acc.y * sc, acc.z * sc, acc.w * sc};
            if (live) {
              if constexpr (EPI == EPI_F32) {
                float* y = static_cast<float*>(p.ep.y) + static_cast<size_t>(m) * p.ep.ldy;
                if (vec) *reinterpret_cast<float4*>(y + n) = make_float4(a4[0], a4[1], a4[2], a4[3]);
                else
#pragma unroll
                  for (int q = 0; q < 4; ++q) if (n + q < p.N) y[n + q] = a4[q];
              } else {
                __nv_bfloat16* y = static_cast<__nv_bfloat16*>(p.ep.y) + static_cast<size_t>(m) * p.ep.ldy;
                if (vec) {
                  __nv_bfloat162 lo = __floats2bfloat162_rn(a4[0], a4[1]), hi = __floats2bfloat162_rn(a4[2], a4[3]);
                  *reinterpret_cast<uint2*>(y + n) = make_uint2(*reinterpret_cast<uint32_t*>(&lo), *reinterpret_cast<uint32_t*>(&hi));
                } else {
#pragma unroll
                  for (int q = 0; q < 4; ++q) if (n + q < p.N) y[n + q] = __float2bfloat16_rn(a4[q]);
                }
              }
            }
          }
        }
        if (seg + 1 < n_tiles_mine) {  // more tiles: tell every CTA of the cluster that this owner's buffers are free
          epi_bar_sync();
          if (et < C) mbar_arrive_remote(free_bar, static_cast<uint32_t>(et));
        }
      }
    }
    (void)alive;
    tc_fence_before();
  }
  __syncthreads();
  if (warp == 1) {
    tc_fence_after();
    tmem_dealloc<TMEM_COLS>(tmem_base);
  }
}

inline size_t gemm_ck_recv_bytes(int a_rows, int C) {
  const int n_units = 4 * (a_rows / 16);
  return static_cast<size_t>((n_units + C - 1) / C) * C * 2048;
}
inline size_t gemm_ck_smem_bytes(int a_rows, int stages, int C) {
  size_t body = static_cast<size_t>(stages) * (a_rows * 128 + 128 * 128) + gemm_ck_recv_bytes(a_rows, C);
  size_t need = static_cast<size_t>(stages) * a_rows * 128 + static_cast<size_t>(128 - a_rows) * 128 + 128 * 128;
  if (body < need) body = need;
  return 1024 + body + (2 * stages + 6) * 8 + 64;
}

// ----------------------------------------------------------------------------- column-strip kernel
// Skinny matmuls with many output columns (QKV, gate/up at up to 64 rows).  CTA b owns the column
// strip [b*S, (b+1)*S) over the whole K range (S a multiple of 16 that divides N, S <= 256): every
// output is produced by one CTA, so there are no partial tiles, no arrival counters and no fix-up
// after the last weight byte has arrived; all CTAs stream the same number of weight bytes.  The price
// is that every CTA reads all of X (from L2), which the host accepts while S >= rows of X.
// Weights must be in the tiled form: strip rows are a run of whole 8-row swizzle groups inside the
// 128-row blocks, copied with one bulk copy per block touched.
//
// A CTA moves a K slab every few hundred cycles, and what paces it is the latency of the dependent
// instructions one thread executes per slab (barrier wait, copy or MMA issue, commit), not bandwidth.
// So the slabs are dealt to p.n_producers (1 or 2) independent pipelines, slab i to pipeline
// i mod n: each has a producer thread (weights, then after the dependency wait X slabs), an
// MMA-issuing thread and its own TMEM accumulator; they share the stage ring, and the epilogue
// adds the accumulators (pipeline 0 first: fixed order).  Producer / MMA warps: 0 / 1 and 6 / 7;
// warps 2-5 run the epilogue.  Shared memory: [stages x a_rows x 128 B] X, [stages x S x 128 B] W,
// barriers.
constexpr int STRIP_THREADS = 256;

// The sum of two accumulators, pipeline 0 first.
struct TmemPairSource {
  uint32_t taddr_row0, taddr_row1;
  bool two;
  __device__ __forceinline__ void load(int c, float (&v)[32]) const {
    tmem_ld_32x32(taddr_row0 + static_cast<uint32_t>(c), v);
    if (two) {
      float w[32];
      tmem_ld_32x32(taddr_row1 + static_cast<uint32_t>(c), w);  // both loads in flight
      tmem_ld_wait();
#pragma unroll
      for (int j = 0; j < 32; ++j) v[j] += w[j];
    } else {
      tmem_ld_wait();
    }
  }
};

template <int EPI, int TCOLS>
__global__ void __launch_bounds__(STRIP_THREADS, 2)
gemm_strip_kernel(const __grid_constant__ CUtensorMap tmap_x, const GemmParams p, const int S) {
  if (p.skip_flag != nullptr && *p.skip_flag != 0) return;
  grid_dep_launch();
  extern __shared__ uint8_t smem_raw[];
  uint8_t* smem = reinterpret_cast<uint8_t*>((reinterpret_cast<uintptr_t>(smem_raw) + 1023) & ~uintptr_t(1023));
  const int stages = p.stages;
  const uint32_t a_stage_bytes = static_cast<uint32_t>(p.a_rows) * 128u;
  const uint32_t b_stage_bytes = static_cast<uint32_t>(S) * 128u;
  uint8_t* smem_a = smem;
  uint8_t* smem_b = smem + static_cast<size_t>(stages) * a_stage_bytes;
  // the MMA reads 128 rows of X whatever a_rows is: the barriers start after that reach
  size_t body = static_cast<size_t>(stages) * (a_stage_bytes + b_stage_bytes);
  const size_t reach = static_cast<size_t>(stages - 1) * a_stage_bytes + 128 * 128;
  if (body < reach) body = reach;
  uint64_t* full_bar = reinterpret_cast<uint64_t*>(smem + ((body + 7) & ~size_t(7)));
  uint64_t* empty_bar = full_bar + stages;
  uint64_t* acc_full = empty_bar + stages;
  uint32_t* tmem_slot = reinterpret_cast<uint32_t*>(acc_full + 1);
  volatile int* abort_flag = reinterpret_cast<volatile int*>(tmem_slot + 1);

  const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
  const int KC = p.k_chunks;
  const int n_pipe = p.n_producers;                  // 1 or 2; the host gives 2 only when 2 * S <= TCOLS and KC >= 2
  const int c0 = static_cast<int>(blockIdx.x) * S;  // first column of the strip
  // CTA b walks K from slab (b * p.gm) mod KC and wraps around, so that the CTAs of a moment do not
  // all read the same X slab (the same few L2 lines); the order of a strip's fp32 sums is fixed by b.
  const int k_off = static_cast<int>((static_cast<long long>(blockIdx.x) * p.gm) % KC);

  if (threadIdx.x == 0) {
    prefetch_tensormap(&tmap_x);
    for (int s = 0; s < stages; ++s) {
      mbar_init(&full_bar[s], 1);
      mbar_init(&empty_bar[s], 1);
    }
    mbar_init(acc_full, static_cast<uint32_t>(n_pipe));  // one commit per pipeline
    *abort_flag = 0;
    fence_barrier_init();
  }
  if (warp == 1) {
    tmem_alloc<TCOLS>(tmem_slot);
    tmem_relinquish();
  }
  tc_fence_before();
  __syncthreads();
  tc_fence_after();
  const uint32_t tmem_base = *tmem_slot;

  // The single-thread loops below carry running counters instead of dividing by `stages` or KC, and
  // all address arithmetic that does not change with the slab is done up front.
  const int pipe = (warp == 0 || warp == 1) ? 0 : 1;
  if ((warp == 0 || warp == 6) && pipe < n_pipe) {
    // ---------------- producer of pipeline `pipe`: slabs pipe, pipe + n_pipe, ...
    if (lane == 0) {
      // the strip's rows inside the 128-row blocks it touches: up to three runs of whole 8-row groups
      const __nv_bfloat16* piece_src[3];
      uint32_t piece_bytes[3], piece_dst[3];
      {
        int row = c0, left = S;
        uint32_t off = 0;
#pragma unroll
        for (int j = 0; j < 3; ++j) {  // S <= 256: at most three blocks
          const int blk = row >> 7, r0 = row & 127;
          const int n = left < 128 - r0 ? left : 128 - r0;  // 0 once the strip is covered
          piece_src[j] = p.w_packed + (static_cast<long long>(blk) * KC * 128 + r0) * 64;
          piece_bytes[j] = static_cast<uint32_t>(n) * 128u;
          piece_dst[j] = off;
          off += static_cast<uint32_t>(n) * 128u;
          row += n;
          left -= n;
        }
      }
      auto load_w = [&](int s, int kc) {  // arms the stage with all the bytes that will arrive, then the weights
        mbar_arrive_expect_tx(&full_bar[s], a_stage_bytes + b_stage_bytes);
        uint8_t* dst = smem_b + static_cast<uint32_t>(s) * b_stage_bytes;
        const size_t slab = static_cast<size_t>(kc) * (128 * 64);
#pragma unroll
        for (int j = 0; j < 3; ++j)
          if (piece_bytes[j] != 0) bulk_load_1d(dst + piece_dst[j], piece_src[j] + slab, piece_bytes[j], &full_bar[s]);
      };
      auto load_x = [&](int s, int kc) {
        tma_load_2d(smem_a + static_cast<uint32_t>(s) * a_stage_bytes, &tmap_x, &full_bar[s], kc * BLOCK_K, 0);
      };
      auto wrap_kc = [&](int kc) { return kc >= KC ? kc - KC : kc; };
      const int pre = KC < stages ? KC : stages;  // slabs of the first lap: their stages are free
      // weights of the first lap: they do not depend on the kernels before this one
      int kc = wrap_kc(k_off + pipe);
      for (int i = pipe; i < pre; i += n_pipe) {
        load_w(i, kc);
        kc = wrap_kc(kc + n_pipe);
      }
      grid_dep_wait();
      kc = wrap_kc(k_off + pipe);
      int i = pipe;
      for (; i < pre; i += n_pipe) {
        load_x(i, kc);
        kc = wrap_kc(kc + n_pipe);
      }
      int s = i - stages;          // slab i >= stages lives in stage i mod stages (i < stages + n_pipe here)
      uint32_t ph = 0;             // parity of the empty barrier's completed phase to wait for
      for (; i < KC; i += n_pipe) {
        if (!mbar_wait(&empty_bar[s], ph, abort_flag, p.error_word)) break;
        load_w(s, kc);
        load_x(s, kc);
        kc = wrap_kc(kc + n_pipe);
        s += n_pipe;
        if (s >= stages) { s -= stages; ph ^= 1u; }
      }
    }
  } else if ((warp == 1 || warp == 7) && pipe < n_pipe) {
    // ---------------- MMA issuer of pipeline `pipe`
    if (lane == 0) {
      const uint32_t idesc = make_idesc(BLOCK_M, S);
      const uint64_t adesc0 = make_smem_desc(smem_u32(smem_a)), bdesc0 = make_smem_desc(smem_u32(smem_b));
      const uint64_t a_step = a_stage_bytes >> 4, b_step = b_stage_bytes >> 4;  // stage strides in descriptor units
      const uint32_t tmem_d = tmem_base + static_cast<uint32_t>(pipe * (TCOLS / 2));
      int s = pipe;
      uint32_t ph = 0;
      bool ok = true;
      for (int i = pipe; i < KC; i += n_pipe) {
        if (!mbar_wait(&full_bar[s], ph, abort_flag, p.error_word)) { ok = false; break; }
        tc_fence_after();
        const uint64_t adesc = adesc0 + a_step * static_cast<uint64_t>(s), bdesc = bdesc0 + b_step * static_cast<uint64_t>(s);
#pragma unroll
        for (int kk = 0; kk < BLOCK_K / UMMA_K; ++kk)
          umma_bf16(tmem_d, adesc + static_cast<uint64_t>(2 * kk), bdesc + static_cast<uint64_t>(2 * kk), idesc,
                    (i > pipe || kk > 0) ? 1u : 0u);
        umma_commit(&empty_bar[s]);
        s += n_pipe;
        if (s >= stages) { s -= stages; ph ^= 1u; }
      }
      if (ok) umma_commit(acc_full);
    }
  }
  // ---------------- epilogue: warps 2-5, TMEM lane group = warp % 4.  With at most 32 rows only lane
  // group 0 holds anything, and one warp alone would take microseconds over a wide strip: warp 0
  // (same lane group; its producer thread is done by then) takes every other 32-column chunk.
  const bool helper = warp == 0 && p.a_rows <= 32 && S > 32;
  if (warp == 0) __syncwarp();  // lanes 1-31 wait here for the producer thread instead of polling beside it
  if ((warp >= 2 && warp <= 5) || helper) {
    grid_dep_wait();
    const int lg = warp & 3;
    const int row = lg * 32 + lane;
    const bool warp_live = lg * 32 < p.a_rows && lg * 32 < p.M;
    const bool shared_chunks = p.a_rows <= 32 && S > 32;  // lane group 0 is worked on by warps 4 and 0
    const int c_first = helper ? 1 : 0, c_stride = shared_chunks ? 2 : 1;
    // row factor (folded RMSNorm): fetched while the accumulators are still being built
    const float rs = (warp_live && row < p.M && p.ep.ssq_in != nullptr) ? row_rstd(p.ep, row) : 1.f;
    bool ok = mbar_wait(acc_full, 0u, abort_flag, p.error_word);
    ok = __all_sync(0xffffffffu, ok);
    if (ok) {
      tc_fence_after();
      if (warp_live) {
        const uint32_t lane_addr = tmem_base + (static_cast<uint32_t>(lg * 32) << 16);
        TmemPairSource tsrc{lane_addr, lane_addr + static_cast<uint32_t>(TCOLS / 2), n_pipe == 2};
        run_epilogue<EPI, 256>(tsrc, p, row, c0, row < p.M, c_first, c_stride, c0 + S, rs);
      }
    }
    tc_fence_before();
  }
  __syncthreads();
  if (warp == 1) {
    tc_fence_after();
    tmem_dealloc<TCOLS>(tmem_base);
  }
}

inline size_t gemm_strip_smem_bytes(int a_rows, int S, int stages) {
  size_t body = static_cast<size_t>(stages) * (a_rows * 128 + S * 128);
  const size_t reach = static_cast<size_t>(stages - 1) * a_rows * 128 + 128 * 128;
  if (body < reach) body = reach;
  return 1024 + body + 8 + (2 * stages + 1) * 8 + 64;
}

inline size_t gemm_tc_smem_bytes(int a_rows, int block_n, int stages) {
  // The MMA reads 128 rows of the X operand whatever a_rows is: the last X stage must be followed by
  // at least (128 - a_rows) * 128 bytes of allocated shared memory (the W stages, plus padding).
  size_t body = static_cast<size_t>(stages) * (a_rows * 128 + block_n * 128);
  size_t need = static_cast<size_t>(stages) * a_rows * 128 + static_cast<size_t>(a_rows < 128 ? 128 - a_rows : 0) * 128 + 128 * 128;
  if (body < need) body = need;
  return 1024 + body + (2 * stages + 4) * 8 + 64 + MAX_CTAS * 4;
}

}  // namespace tc
}  // namespace d3

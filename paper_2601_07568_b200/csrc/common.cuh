// Shared declarations of the d3 CUDA library: element types, epilogue codes, device error word.
#pragma once
#include <cuda_bf16.h>
#include <cuda_runtime.h>
#include <stdint.h>

namespace d3 {

// ---- device error word bits (read back through d3_get_error_word)
enum : uint32_t {
  ERRW_MBAR_TIMEOUT = 1u << 0,   // a bounded mbarrier wait gave up
  ERRW_BAD_TOKEN_ID = 1u << 1,   // a token id outside [0, vocab)
  ERRW_BAD_POSITION = 1u << 2,   // a cache slot outside [0, max_seq)
  ERRW_TMEM_ALLOC = 1u << 3,     // tensor-memory allocation returned an unexpected address
  ERRW_BAD_STATISTIC = 1u << 4,  // every masked row of a block had an unusable (NaN) statistic: lowest row forced
};

// ---- matmul epilogues
enum : int {
  EPI_F32 = 0,     // y fp32 [m, n] = acc * scale
  EPI_T = 1,       // y T [m, n] = acc
  EPI_RESID = 2,   // y fp32 [m, n] += acc
  EPI_SWIGLU = 3,  // y T [m, n/2]: columns come in groups of 128 = 64 gate then 64 up
  EPI_STATS = 4,   // per (row, 128-column tile): (max, sum exp, sum exp*(l-max), argmax) of scale*acc
  EPI_QKV = 5,     // RoPE on q and k heads (d_head = 128 = one tile), q -> y T, k/v -> cache
};

struct EpiParams {
  void* y = nullptr;          // output (meaning depends on the epilogue)
  int ldy = 0;                // leading dimension of y in elements
  float scale = 1.0f;         // EPI_F32 / EPI_STATS
  int mask_id = -1;           // EPI_STATS: excluded column
  float4* stat_part = nullptr;  // EPI_STATS: [m][n_tiles]
  int n_tiles = 0;
  // RMSNorm folded into the tensor-core matmuls.  A residual epilogue also leaves a bf16 copy of the
  // updated rows (the next matmul's operand) and the sum of squares of every 32-column chunk of them;
  // a matmul fed with that un-normalised copy multiplies accumulator row m by
  // rsqrt(sum(ssq_in[m][0 .. ssq_chunks)) * inv_k + rms_eps) (the norm's gains sit in the weight columns).
  __nv_bfloat16* yb = nullptr;   // EPI_RESID: [m][ldy] bf16 copy of y after the update
  float* ssq_out = nullptr;      // EPI_RESID: [m][ceil(n / 32)]
  const float* ssq_in = nullptr; // any epilogue but EPI_RESID: chunk sums of the operand rows
  int ssq_chunks = 0;
  float inv_k = 0.f, rms_eps = 0.f;
  // EPI_STATS with temperature sampling (sample_part != nullptr): per (row, 128-column tile) also the
  // largest perturbed logit l + temperature * g (g standard Gumbel noise), the index attaining it
  // (lowest on ties) and the unperturbed logit there.  The noise of row m is keyed by
  // (seed; sequence m / rows_per_seq, position pos_base[sequence] + m % rows_per_seq, step).
  float4* sample_part = nullptr;  // [m][n_tiles]: (perturbed max, logit at it, index bits, unused)
  float temperature = 0.f;
  uint32_t seed_lo = 0, seed_hi = 0;
  const int* pos_base = nullptr;    // [sequences]
  int rows_per_seq = 1;
  const int* draw_step = nullptr;   // [sequences] step counter of each sequence (null: draw_step_add alone)
  int draw_step_add = 0;
};

// Row factor of a matmul whose operand rows were left un-normalised; chunk sums added in index
// order (the same bits whichever thread or kernel asks).
__device__ __forceinline__ float row_rstd(const EpiParams& ep, int m) {
  const float* r = ep.ssq_in + static_cast<size_t>(m) * ep.ssq_chunks;
  float tot = 0.f;
  int i = 0;
  if ((ep.ssq_chunks & 3) == 0) {
    const float4* r4 = reinterpret_cast<const float4*>(r);
    for (; i + 16 <= ep.ssq_chunks; i += 16) {  // four independent 16-byte loads in flight
      const float4 a = __ldcg(r4 + i / 4), b = __ldcg(r4 + i / 4 + 1), c = __ldcg(r4 + i / 4 + 2), d = __ldcg(r4 + i / 4 + 3);
      tot += a.x; tot += a.y; tot += a.z; tot += a.w;
      tot += b.x; tot += b.y; tot += b.z; tot += b.w;
      tot += c.x; tot += c.y; tot += c.z; tot += c.w;
      tot += d.x; tot += d.y; tot += d.z; tot += d.w;
    }
  }
  for (; i < ep.ssq_chunks; ++i) tot += __ldcg(r + i);
  return rsqrtf(tot * ep.inv_k + ep.rms_eps);
}

// Philox-4x32 with 10 rounds (Salmon et al., SC'11): a counter-based generator, four 32-bit words
// per call, no state.
__device__ __forceinline__ uint4 philox4x32_10(uint4 c, uint32_t k0, uint32_t k1) {
#pragma unroll
  for (int r = 0; r < 10; ++r) {
    const uint32_t hi0 = __umulhi(0xD2511F53u, c.x), lo0 = 0xD2511F53u * c.x;
    const uint32_t hi1 = __umulhi(0xCD9E8D57u, c.z), lo1 = 0xCD9E8D57u * c.z;
    c = make_uint4(hi1 ^ c.y ^ k0, lo1, hi0 ^ c.w ^ k1, lo0);
    k0 += 0x9E3779B9u;
    k1 += 0xBB67AE85u;
  }
  return c;
}
// Standard Gumbel noise from a 32-bit word: u = (top 23 bits + 1/2) * 2^-23 in (0, 1), g = -ln(-ln u).
__device__ __forceinline__ float gumbel_from_bits(uint32_t x) {
  const float u = (static_cast<float>(x >> 9) + 0.5f) * 1.1920928955078125e-07f;
  return -logf(-logf(u));
}
// Sampling nonce of matmul row m: counter words 1..3 = (position, step, sequence).
struct SampleRow {
  uint32_t pos, step, seq;
};
__device__ __forceinline__ SampleRow sample_row(const EpiParams& ep, int m) {
  const int b = m / ep.rows_per_seq;
  SampleRow r;
  r.seq = static_cast<uint32_t>(b);
  r.pos = static_cast<uint32_t>((ep.pos_base ? ep.pos_base[b] : 0) + m % ep.rows_per_seq);
  r.step = static_cast<uint32_t>((ep.draw_step ? ep.draw_step[b] : 0) + ep.draw_step_add);
  return r;
}
// Running maximum of the perturbed logits: pm = max, la = logit at it, pa = lowest index attaining it.
struct SampleStat {
  float pm, la;
  int pa;
};
__device__ __forceinline__ SampleStat sample_empty() { return SampleStat{-INFINITY, 0.f, 0x7fffffff}; }
__device__ __forceinline__ void sample_add(SampleStat& st, float pert, float l, int idx) {
  if (pert > st.pm || (pert == st.pm && idx < st.pa)) {
    st.pm = pert;
    st.la = l;
    st.pa = idx;
  }
}
__device__ __forceinline__ SampleStat sample_merge(const SampleStat& a, const SampleStat& b) {
  return (b.pm > a.pm || (b.pm == a.pm && b.pa < a.pa)) ? b : a;
}

template <typename T> struct TypeOps;
template <> struct TypeOps<float> {
  static __device__ __forceinline__ float to_f(float v) { return v; }
  static __device__ __forceinline__ float from_f(float v) { return v; }
};
template <> struct TypeOps<__nv_bfloat16> {
  static __device__ __forceinline__ float to_f(__nv_bfloat16 v) { return __bfloat162float(v); }
  static __device__ __forceinline__ __nv_bfloat16 from_f(float v) { return __float2bfloat16_rn(v); }
};

__device__ __forceinline__ float silu_f(float g) { return g / (1.0f + __expf(-g)); }

// Running softmax statistics of a set of logits: m = max, z = sum e^(l-m), s = sum e^(l-m)(l-m),
// a = lowest index attaining m.  Empty set: m = -inf, z = s = 0, a = INT_MAX.
struct SoftStat {
  float m, z, s;
  int a;
};
__device__ __forceinline__ SoftStat stat_empty() { return SoftStat{-INFINITY, 0.f, 0.f, 0x7fffffff}; }
// Merge b into a.  Associative up to rounding; ties on the maximum keep the lower index.
__device__ __forceinline__ SoftStat stat_merge(const SoftStat& a, const SoftStat& b) {
  if (b.z == 0.f) return a;
  if (a.z == 0.f) return b;
  SoftStat r;
  r.m = fmaxf(a.m, b.m);
  float da = a.m - r.m, db = b.m - r.m;  // <= 0
  float ea = __expf(da), eb = __expf(db);
  r.z = ea * a.z + eb * b.z;
  r.s = ea * (a.s + da * a.z) + eb * (b.s + db * b.z);
  r.a = (a.m > b.m) ? a.a : (b.m > a.m) ? b.a : min(a.a, b.a);
  return r;
}
__device__ __forceinline__ void stat_add(SoftStat& st, float l, int idx) {
  if (l > st.m) {
    float d = st.m - l;  // < 0 (or -inf when empty)
    float e = (st.z == 0.f) ? 0.f : __expf(d);
    st.s = (st.z == 0.f) ? 0.f : e * (st.s + d * st.z);
    st.z = e * st.z + 1.0f;
    st.m = l;
    st.a = idx;
  } else {
    float d = l - st.m;  // <= 0
    float e = __expf(d);
    st.z += e;
    st.s += e * d;
    // equal maxima: indices are visited in ascending order, so the first one stays
  }
}

}  // namespace d3

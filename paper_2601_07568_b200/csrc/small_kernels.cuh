// Row-wise and per-sequence kernels around the matmuls: embedding gather, RMSNorm, RoPE + cache
// write, softmax-statistics merge, the threshold unmask decision and the generate-loop bookkeeping.
#pragma once
#include "common.cuh"
#include "ptx_sm100.cuh"

namespace d3 {

// Per-sequence row map of one forward: row m belongs to sequence b = m / rows_per_seq at offset
// r = m % rows_per_seq; it is live when r < n_valid[b] and sits at absolute position pos_base[b] + r;
// its attention reads cache slots [0, kv_len[b]).
// `seg` > 0 cuts the rows of a sequence into segments of `seg` rows (consecutive blocks in one
// forward): row r then sees slots [0, pos_base[b] + (r / seg + 1) * seg) only - the prefix, the earlier
// segments and its own, never a later one.  seg = 0: every row sees [0, kv_len[b]).
struct RowMap {
  const int* pos_base;
  const int* n_valid;
  const int* kv_len;
  int rows_per_seq;
  int bs;
  int seg;
};
__device__ __forceinline__ int row_kv_limit(const RowMap& rm, int b, int r, int kv_len) {
  if (rm.seg <= 0) return kv_len;
  const int lim = rm.pos_base[b] + (r / rm.seg + 1) * rm.seg;
  return lim < kv_len ? lim : kv_len;
}

__device__ __forceinline__ float warp_sum(float v) {
#pragma unroll
  for (int o = 16; o > 0; o >>= 1) v += __shfl_xor_sync(0xffffffffu, v, o);
  return v;
}

// ----------------------------------------------------------------------------- embedding
template <typename T>
__global__ void embed_kernel(const int* __restrict__ ids, const T* __restrict__ emb, float* __restrict__ x, int d,
                             int vocab, uint32_t* error_word) {
  ptx::grid_dep_wait();
  ptx::grid_dep_launch();
  const int m = blockIdx.x;
  int id = ids[m];
  if (id < 0 || id >= vocab) {
    if (threadIdx.x == 0) atomicOr(error_word, ERRW_BAD_TOKEN_ID);
    id = 0;
  }
  const T* src = emb + static_cast<size_t>(id) * d;
  float* dst = x + static_cast<size_t>(m) * d;
  for (int i = threadIdx.x; i < d; i += blockDim.x) dst[i] = TypeOps<T>::to_f(src[i]);
}

// ----------------------------------------------------------------------------- folded RMSNorm helpers
// What a residual epilogue leaves behind for the next matmul (see EpiParams), for rows that no matmul
// has written yet (the embeddings): bf16 copy of x and the sum of squares of every 32-column chunk.
// One block per row; thread t takes chunks t, t + blockDim.x, ...
__global__ void row_prep_kernel(const float* __restrict__ x, __nv_bfloat16* __restrict__ xb, float* __restrict__ ssq, int d) {
  ptx::grid_dep_wait();
  ptx::grid_dep_launch();
  const int m = blockIdx.x;
  const int n_chunks = (d + 31) / 32;
  const float* row = x + static_cast<size_t>(m) * d;
  __nv_bfloat16* out = xb + static_cast<size_t>(m) * d;
  for (int ch = threadIdx.x; ch < n_chunks; ch += blockDim.x) {
    float sq = 0.f;
    const int e1 = min(d, ch * 32 + 32);
    for (int e = ch * 32; e < e1; ++e) {  // same element order as the matmul epilogue's chunk sum
      const float v = row[e];
      sq += v * v;
      out[e] = __float2bfloat16_rn(v);
    }
    ssq[static_cast<size_t>(m) * n_chunks + ch] = sq;
  }
}

// w[n, k] *= gain[k] (rounded to bf16 once): the gains of the RMSNorm in front of a matmul, moved
// into its weight columns when the weights are loaded.
// grid (ceil(k / 256), rows): one thread per element, the column index needs no division.
__global__ void scale_columns_kernel(__nv_bfloat16* __restrict__ w, const float* __restrict__ gain, int k) {
  const int col = blockIdx.x * blockDim.x + threadIdx.x;
  if (col >= k) return;
  __nv_bfloat16* e = w + static_cast<size_t>(blockIdx.y) * k + col;
  *e = __float2bfloat16_rn(__bfloat162float(*e) * gain[col]);
}

// ----------------------------------------------------------------------------- RMSNorm
// xn[m, :] = T(x[m, :] * rsqrt(mean(x^2) + eps) * gain); fp32 arithmetic, fixed reduction order.
// One 256-thread block per row; d % 4 == 0.  The row is read once as float4 and the first 4096
// elements stay in registers between the two passes.
__device__ __forceinline__ void store4(float* dst, float a, float b, float c, float d) {
  *reinterpret_cast<float4*>(dst) = make_float4(a, b, c, d);
}
__device__ __forceinline__ void store4(__nv_bfloat16* dst, float a, float b, float c, float d) {
  __nv_bfloat162 lo = __floats2bfloat162_rn(a, b), hi = __floats2bfloat162_rn(c, d);
  *reinterpret_cast<uint2*>(dst) = make_uint2(*reinterpret_cast<uint32_t*>(&lo), *reinterpret_cast<uint32_t*>(&hi));
}
template <typename T>
__global__ void __launch_bounds__(256) rmsnorm_kernel(const float* __restrict__ x, const float* __restrict__ gain,
                                                      T* __restrict__ xn, int d, float eps) {
  ptx::grid_dep_wait();
  ptx::grid_dep_launch();
  const int m = blockIdx.x;
  const float4* row = reinterpret_cast<const float4*>(x + static_cast<size_t>(m) * d);
  const float4* g4 = reinterpret_cast<const float4*>(gain);
  const int n4 = d >> 2;
  float4 v[4];
  float ss = 0.f;
#pragma unroll
  for (int i = 0; i < 4; ++i) {
    const int idx = threadIdx.x + i * 256;
    v[i] = idx < n4 ? row[idx] : make_float4(0.f, 0.f, 0.f, 0.f);
    ss += v[i].x * v[i].x + v[i].y * v[i].y + v[i].z * v[i].z + v[i].w * v[i].w;
  }
  for (int idx = threadIdx.x + 1024; idx < n4; idx += 256) {
    const float4 t = row[idx];
    ss += t.x * t.x + t.y * t.y + t.z * t.z + t.w * t.w;
  }
  __shared__ float red[8];
  ss = warp_sum(ss);
  if ((threadIdx.x & 31) == 0) red[threadIdx.x >> 5] = ss;
  __syncthreads();
  float tot = 0.f;
#pragma unroll
  for (int w = 0; w < 8; ++w) tot += red[w];  // same order in every thread
  const float rstd = rsqrtf(tot / static_cast<float>(d) + eps);
  T* out = xn + static_cast<size_t>(m) * d;
#pragma unroll
  for (int i = 0; i < 4; ++i) {
    const int idx = threadIdx.x + i * 256;
    if (idx < n4) {
      const float4 g = g4[idx];
      store4(out + 4 * idx, v[i].x * rstd * g.x, v[i].y * rstd * g.y, v[i].z * rstd * g.z, v[i].w * rstd * g.w);
    }
  }
  for (int idx = threadIdx.x + 1024; idx < n4; idx += 256) {
    const float4 t = row[idx], g = g4[idx];
    store4(out + 4 * idx, t.x * rstd * g.x, t.y * rstd * g.y, t.z * rstd * g.z, t.w * rstd * g.w);
  }
}

// ----------------------------------------------------------------------------- RoPE + cache write
// qkv: fp32 [M, (hq + 2 hkv) * dh] straight from the projection, whose q and k rows are packed so
// that columns (2k, 2k+1) of a head hold dims (k, k + dh/2).  q heads are rotated and stored as
// T [M, hq*dh] in natural dim order; k heads are rotated and stored in the cache, v heads stored as
// they are.
template <typename T>
__global__ void rope_kv_kernel(const float* __restrict__ qkv, T* __restrict__ q_out, T* __restrict__ k_cache,
                               T* __restrict__ v_cache, const float* __restrict__ rope_cos,
                               const float* __restrict__ rope_sin, RowMap rm, int hq, int hkv, int dh, int max_seq,
                               uint32_t* error_word) {
  const int m = blockIdx.x;
  const int b = m / rm.rows_per_seq, r = m % rm.rows_per_seq;
  if (r >= rm.n_valid[b]) return;
  const int pos = rm.pos_base[b] + r;
  if (pos < 0 || pos >= max_seq) {
    if (threadIdx.x == 0) atomicOr(error_word, ERRW_BAD_POSITION);
    return;
  }
  const int half = dh / 2;
  const int nq = hq * dh, nkv = hkv * dh;
  const float* row = qkv + static_cast<size_t>(m) * (nq + 2 * nkv);
  const float* cs = rope_cos + static_cast<size_t>(pos) * half;
  const float* sn = rope_sin + static_cast<size_t>(pos) * half;
  // rotated pairs of q and k
  const int n_pairs = (hq + hkv) * half;
  for (int i = threadIdx.x; i < n_pairs; i += blockDim.x) {
    const int head = i / half, k = i % half;
    const float a = row[head * dh + 2 * k], bb = row[head * dh + 2 * k + 1];
    const float lo = a * cs[k] - bb * sn[k];
    const float hi = bb * cs[k] + a * sn[k];
    if (head < hq) {
      T* dst = q_out + static_cast<size_t>(m) * nq + head * dh;
      dst[k] = TypeOps<T>::from_f(lo);
      dst[k + half] = TypeOps<T>::from_f(hi);
    } else {
      T* dst = k_cache + ((static_cast<size_t>(b) * hkv + (head - hq)) * max_seq + pos) * dh;
      dst[k] = TypeOps<T>::from_f(lo);
      dst[k + half] = TypeOps<T>::from_f(hi);
    }
  }
  for (int i = threadIdx.x; i < nkv; i += blockDim.x) {
    const int head = i / dh, k = i % dh;
    v_cache[((static_cast<size_t>(b) * hkv + head) * max_seq + pos) * dh + k] =
        TypeOps<T>::from_f(row[nq + nkv + i]);
  }
}

// ----------------------------------------------------------------------------- statistics merge
// One warp per row merges the per-tile partial statistics in ascending tile order (fixed tree) and
// writes confidence = 1/Z, entropy = ln Z - S/Z (nats) and the arg max.
__global__ void stats_merge_kernel(const float4* __restrict__ part, int n_tiles, int M, float* __restrict__ conf,
                                   float* __restrict__ entropy, int* __restrict__ argmax) {
  ptx::grid_dep_wait();
  ptx::grid_dep_launch();
  const int m = blockIdx.x * (blockDim.x >> 5) + (threadIdx.x >> 5);
  const int lane = threadIdx.x & 31;
  if (m >= M) return;
  SoftStat st = stat_empty();
  for (int t = lane; t < n_tiles; t += 32) {
    float4 v = part[static_cast<size_t>(m) * n_tiles + t];
    SoftStat o{v.x, v.y, v.z, __float_as_int(v.w)};
    st = stat_merge(st, o);
  }
#pragma unroll
  for (int o = 16; o > 0; o >>= 1) {
    SoftStat other;
    other.m = __shfl_xor_sync(0xffffffffu, st.m, o);
    other.z = __shfl_xor_sync(0xffffffffu, st.z, o);
    other.s = __shfl_xor_sync(0xffffffffu, st.s, o);
    other.a = __shfl_xor_sync(0xffffffffu, st.a, o);
    // keep the operand order fixed (lower lane first) so every lane computes the same bits
    st = (lane & o) ? stat_merge(other, st) : stat_merge(st, other);
  }
  if (lane == 0) {
    if (st.z > 0.f) {
      conf[m] = 1.0f / st.z;
      entropy[m] = fmaxf(logf(st.z) - st.s / st.z, 0.f);
      argmax[m] = st.a;
    } else {
      conf[m] = 0.f;
      entropy[m] = 0.f;
      argmax[m] = 0;
    }
  }
}

// The same with temperature sampling: the token is the index of the largest perturbed logit over all
// tiles (lowest index on ties) and the confidence its probability e^(l - m) / Z under the unperturbed
// softmax; the entropy is unchanged.
__global__ void stats_merge_sample_kernel(const float4* __restrict__ part, const float4* __restrict__ sample_part, int n_tiles,
                                          int M, float* __restrict__ conf, float* __restrict__ entropy, int* __restrict__ argmax) {
  ptx::grid_dep_wait();
  ptx::grid_dep_launch();
  const int m = blockIdx.x * (blockDim.x >> 5) + (threadIdx.x >> 5);
  const int lane = threadIdx.x & 31;
  if (m >= M) return;
  SoftStat st = stat_empty();
  SampleStat sp = sample_empty();
  for (int t = lane; t < n_tiles; t += 32) {
    const float4 v = part[static_cast<size_t>(m) * n_tiles + t];
    st = stat_merge(st, SoftStat{v.x, v.y, v.z, __float_as_int(v.w)});
    const float4 w = sample_part[static_cast<size_t>(m) * n_tiles + t];
    sp = sample_merge(sp, SampleStat{w.x, w.y, __float_as_int(w.z)});
  }
#pragma unroll
  for (int o = 16; o > 0; o >>= 1) {
    SoftStat other;
    other.m = __shfl_xor_sync(0xffffffffu, st.m, o);
    other.z = __shfl_xor_sync(0xffffffffu, st.z, o);
    other.s = __shfl_xor_sync(0xffffffffu, st.s, o);
    other.a = __shfl_xor_sync(0xffffffffu, st.a, o);
    st = (lane & o) ? stat_merge(other, st) : stat_merge(st, other);
    SampleStat so;
    so.pm = __shfl_xor_sync(0xffffffffu, sp.pm, o);
    so.la = __shfl_xor_sync(0xffffffffu, sp.la, o);
    so.pa = __shfl_xor_sync(0xffffffffu, sp.pa, o);
    sp = sample_merge(sp, so);
  }
  if (lane == 0) {
    if (st.z > 0.f && sp.pa != 0x7fffffff) {
      conf[m] = fminf(expf(sp.la - st.m) / st.z, 1.0f);
      entropy[m] = fmaxf(logf(st.z) - st.s / st.z, 0.f);
      argmax[m] = sp.pa;
    } else {
      conf[m] = 0.f;
      entropy[m] = 0.f;
      argmax[m] = 0;
    }
  }
}

// Statistics straight from fp32 logits rows (SIMT path and tests): one block per row.
__global__ void stats_from_logits_kernel(const float* __restrict__ logits, int V, int mask_id, float4* __restrict__ part,
                                         int n_tiles) {
  // one warp per (row, 128-column tile); lanes stride the tile, then a fixed shuffle tree
  const int m = blockIdx.y;
  const int t = blockIdx.x * (blockDim.x >> 5) + (threadIdx.x >> 5);
  const int lane = threadIdx.x & 31;
  if (t >= n_tiles) return;
  const float* row = logits + static_cast<size_t>(m) * V;
  SoftStat st = stat_empty();
  for (int j = lane; j < 128; j += 32) {
    int n = t * 128 + j;
    if (n < V && n != mask_id) stat_add(st, row[n], n);
  }
#pragma unroll
  for (int o = 16; o > 0; o >>= 1) {
    SoftStat other;
    other.m = __shfl_xor_sync(0xffffffffu, st.m, o);
    other.z = __shfl_xor_sync(0xffffffffu, st.z, o);
    other.s = __shfl_xor_sync(0xffffffffu, st.s, o);
    other.a = __shfl_xor_sync(0xffffffffu, st.a, o);
    st = (lane & o) ? stat_merge(other, st) : stat_merge(st, other);
  }
  if (lane == 0) part[static_cast<size_t>(m) * n_tiles + t] = make_float4(st.m, st.z, st.s, __int_as_float(st.a));
}

// ----------------------------------------------------------------------------- decision
// One warp per sequence.  Commits every masked position clearing the threshold and always the most
// confident masked one (lowest index on ties); writes ids, clears mask bytes, emits (pos, id) in
// ascending position order.  Returns through the out arrays; `remaining` (optional) gets the number of
// masks left.  B <= 128.
struct UnmaskOut {
  int committed;
  int forced;     // 1 when the forced position did not clear the threshold
  int remaining;
};
__device__ __forceinline__ UnmaskOut unmask_block(const float* conf, const float* ent, const int* argmax, int* ids,
                                                  uint8_t* mask, int B, float tau, int mode, int* out_pos,
                                                  int* out_ids, int* commit_step, int step, bool force = true,
                                                  uint32_t* error_word = nullptr) {
  const int lane = threadIdx.x & 31;
  // pass 1: best masked position
  float best = -INFINITY;
  int best_r = 0x7fffffff;
  for (int r = lane; r < B; r += 32) {
    if (mask[r]) {
      float s = (mode == 0) ? conf[r] : -ent[r];
      if (s > best || (s == best && r < best_r)) {
        best = s;
        best_r = r;
      }
    }
  }
#pragma unroll
  for (int o = 16; o > 0; o >>= 1) {
    float ob = __shfl_xor_sync(0xffffffffu, best, o);
    int orr = __shfl_xor_sync(0xffffffffu, best_r, o);
    if (orr != 0x7fffffff && (best_r == 0x7fffffff || ob > best || (ob == best && orr < best_r))) {
      best = ob;
      best_r = orr;
    }
  }
  UnmaskOut res{0, 0, 0};
  if (best_r == 0x7fffffff) {
    // no masked row compared greater than -inf: either nothing is masked, or every masked row's
    // statistic is unusable (NaN compares false).  The block must still lose a mask per forward
    // (Sec. 3.2, at-least-one rule), so the lowest masked row is forced and the error word is raised.
    int first = 0x7fffffff;
    for (int r = lane; r < B; r += 32)
      if (mask[r] && r < first) first = r;
#pragma unroll
    for (int o = 16; o > 0; o >>= 1) first = min(first, __shfl_xor_sync(0xffffffffu, first, o));
    if (first == 0x7fffffff) return res;  // nothing masked
    best_r = first;
    if (lane == 0 && error_word != nullptr) atomicOr(error_word, ERRW_BAD_STATISTIC);
  }
  int base = 0;
  for (int r0 = 0; r0 < B; r0 += 32) {
    const int r = r0 + lane;
    bool masked = (r < B) && mask[r];
    bool clears = masked && ((mode == 0) ? (conf[r] > tau) : (ent[r] < tau));
    bool commit = clears || (force && masked && r == best_r);  // without `force`: only what clears the threshold
    if (force && masked && r == best_r && !clears) res.forced = 1;
    unsigned bal = __ballot_sync(0xffffffffu, commit);
    if (commit) {
      int slot = base + __popc(bal & ((1u << lane) - 1u));
      int tok = argmax[r];
      ids[r] = tok;
      mask[r] = 0;
      if (out_pos) out_pos[slot] = r;
      if (out_ids) out_ids[slot] = tok;
      if (commit_step) commit_step[r] = step;
    }
    base += __popc(bal);
    res.remaining += __popc(__ballot_sync(0xffffffffu, masked && !commit));
  }
  res.forced = __any_sync(0xffffffffu, res.forced) ? 1 : 0;
  res.committed = base;
  return res;
}

__global__ void unmask_kernel(const float* __restrict__ conf, const float* __restrict__ ent,
                              const int* __restrict__ argmax, int* ids, uint8_t* mask, int B, float tau, int mode,
                              int* out_pos, int* out_ids, int* out_count, uint32_t* error_word) {
  const int b = blockIdx.x;
  UnmaskOut r = unmask_block(conf + b * B, ent + b * B, argmax + b * B, ids + b * B, mask + b * B, B, tau, mode,
                             out_pos ? out_pos + b * B : nullptr, out_ids ? out_ids + b * B : nullptr, nullptr, 0, true,
                             error_word);
  if (threadIdx.x == 0 && out_count) out_count[b] = r.committed;
}

// ----------------------------------------------------------------------------- generate bookkeeping
// A sequence denoises its current block until no mask is left, then the block needs one more forward
// on its final tokens so that the cached K/V are theirs (finalize).  That forward is independent of
// the first denoise step of the next block except that the latter reads the former's K/V, which the
// same forward writes before its attention runs: with `fuse` the two run as one forward of 2B rows
// (segment 0 = the finished block, segment 1 = the new, fully masked block; segment 0 never sees
// segment 1).  The last block of a request, and every block when fuse is off, is finalized alone.
enum : int { SEQ_DENOISE = 0, SEQ_FINALIZE = 1, SEQ_DONE = 2, SEQ_FUSED = 3 };
struct GenState {
  int* mode;        // [bs] SEQ_*
  int* block_idx;   // [bs] block being denoised
  int* step;        // [bs] denoise steps taken in the current block
  int* prefix_len;  // [bs] cached prefix: prompt + finalized blocks
  int* ids;         // [bs, B] current block
  uint8_t* mask;    // [bs, B]
  int* prev;        // [bs, B] finished block waiting for its finalize forward (SEQ_FUSED)
  int* fwd_ids;     // [bs, 2B] ids of the next forward, rows_per_seq = B or 2B
  int* out_ids;     // [bs, gen_len]
  int* commit_step; // [bs, gen_len] or null
  long long* counters;  // [0] denoise fwd, [1] finalize fwd, [2] tokens, [3] forced, [4] seqs not done, [5] seqs in SEQ_FUSED,
                        // [6] sequences stopped early on the end-of-sequence id, [7] sequences waiting for a KV-refresh
  int* hist;            // [bs, max_seq] ids of the stored prefix (prompt and stored blocks)
  int* refresh_flag;    // [bs] 1: the stored prefix of this sequence is to be recomputed before the next forward
  unsigned long long* commit_hist;  // [COMMIT_HIST_BINS] decisions that committed k tokens (k = bin index)
  uint32_t* error_word;
};
constexpr int COMMIT_HIST_BINS = 129;  // a block has at most 128 positions

// Row map and input ids of the next decode forward (rows_per_seq = R, B or 2B) from the generate
// state.  One block per sequence.
__global__ void gen_rowmap_kernel(GenState g, int bs, int B, int R, int mask_id, int* pos_base, int* n_valid, int* kv_len) {
  const int b = blockIdx.x;
  const int mode = g.mode[b];
  const int rows = mode == SEQ_DONE ? 0 : (mode == SEQ_FUSED ? 2 * B : B);
  if (threadIdx.x == 0) {
    pos_base[b] = g.prefix_len[b];
    n_valid[b] = rows;
    kv_len[b] = rows > 0 ? g.prefix_len[b] + rows : 0;
  }
  for (int r = threadIdx.x; r < R; r += blockDim.x) {
    int id = mask_id;
    if (mode == SEQ_FUSED) id = r < B ? g.prev[b * B + r] : g.ids[b * B + r - B];
    else if (r < B) id = g.ids[b * B + r];
    g.fwd_ids[b * R + r] = id;
  }
}

// After a forward of R rows per sequence: finalize bookkeeping and / or the unmask decision.  One warp
// per sequence.
__global__ void gen_advance_kernel(GenState g, const float* __restrict__ conf, const float* __restrict__ ent,
                                   const int* __restrict__ argmax, int bs, int B, int R, int n_blocks, int gen_len,
                                   float tau, int decide_mode, int mask_id, int fuse, int eos_id, int max_seq,
                                   int refresh_every) {
  const int b = blockIdx.x;
  const int lane = threadIdx.x & 31;
  const int mode = g.mode[b];
  if (mode == SEQ_DONE) return;
  int* ids = g.ids + b * B;
  uint8_t* mask = g.mask + b * B;
  const int pl = g.prefix_len[b];  // before this kernel moves it
  __syncwarp();
  if (mode == SEQ_FINALIZE) {  // the block in `ids` is final and now cached: append it, next block or done
    const int j = g.block_idx[b];
    for (int r = lane; r < B; r += 32) {
      g.out_ids[static_cast<size_t>(b) * gen_len + j * B + r] = ids[r];
      g.hist[static_cast<size_t>(b) * max_seq + pl + r] = ids[r];
      ids[r] = mask_id;
      mask[r] = 1;
    }
    __syncwarp();
    if (lane == 0) {
      g.prefix_len[b] += B;
      g.block_idx[b] = j + 1;
      g.step[b] = 0;
      atomicAdd(reinterpret_cast<unsigned long long*>(&g.counters[1]), 1ull);
      if (j + 1 >= n_blocks) {
        g.mode[b] = SEQ_DONE;
        atomicAdd(reinterpret_cast<unsigned long long*>(&g.counters[4]), static_cast<unsigned long long>(-1ll));
      } else {
        g.mode[b] = SEQ_DENOISE;
        // periodic KV-refresh: the stored block count reached a multiple of the period
        if (refresh_every > 0 && (j + 1) % refresh_every == 0) {
          g.refresh_flag[b] = 1;
          atomicAdd(reinterpret_cast<unsigned long long*>(&g.counters[7]), 1ull);
        }
      }
    }
    return;
  }
  int stat_row0 = b * R;  // rows of the block that was denoised in this forward
  if (mode == SEQ_FUSED) {  // segment 0 finalized the block in `prev`: append it; segment 1 was a first denoise step
    const int j = g.block_idx[b] - 1;
    for (int r = lane; r < B; r += 32) {
      g.out_ids[static_cast<size_t>(b) * gen_len + j * B + r] = g.prev[b * B + r];
      g.hist[static_cast<size_t>(b) * max_seq + pl + r] = g.prev[b * B + r];
    }
    if (lane == 0) {
      g.prefix_len[b] += B;
      atomicAdd(reinterpret_cast<unsigned long long*>(&g.counters[1]), 1ull);
      atomicAdd(reinterpret_cast<unsigned long long*>(&g.counters[5]), static_cast<unsigned long long>(-1ll));
    }
    stat_row0 += B;
  }
  const int step = g.step[b] + 1;
  int* cs = g.commit_step ? g.commit_step + static_cast<size_t>(b) * gen_len + g.block_idx[b] * B : nullptr;
  // positions masked before the decision: those that are not afterwards were committed in this step
  bool was_masked[4];
#pragma unroll
  for (int q = 0; q < 4; ++q) was_masked[q] = lane + 32 * q < B && mask[lane + 32 * q] != 0;
  UnmaskOut r = unmask_block(conf + stat_row0, ent + stat_row0, argmax + stat_row0, ids, mask, B, tau, decide_mode,
                             nullptr, nullptr, cs, step, true, g.error_word);
  __syncwarp();
  if (lane == 0) atomicAdd(&g.commit_hist[r.committed], 1ull);
  // early stop: the end-of-sequence id was committed in this step.  The sequence is done; its current
  // block goes out as it is (mask id where nothing was decided), later blocks stay mask ids, and the
  // unfinished block is not cached.
  bool hit = false;
  if (eos_id >= 0) {
#pragma unroll
    for (int q = 0; q < 4; ++q) {
      const int pos = lane + 32 * q;
      if (was_masked[q] && mask[pos] == 0 && ids[pos] == eos_id) hit = true;
    }
  }
  if (__any_sync(0xffffffffu, hit)) {
    const int j = g.block_idx[b];
    for (int q = lane; q < B; q += 32) g.out_ids[static_cast<size_t>(b) * gen_len + j * B + q] = mask[q] ? mask_id : ids[q];
    if (lane == 0) {
      g.step[b] = step;
      g.mode[b] = SEQ_DONE;
      atomicAdd(reinterpret_cast<unsigned long long*>(&g.counters[0]), 1ull);
      atomicAdd(reinterpret_cast<unsigned long long*>(&g.counters[2]), static_cast<unsigned long long>(r.committed));
      atomicAdd(reinterpret_cast<unsigned long long*>(&g.counters[3]), static_cast<unsigned long long>(r.forced));
      atomicAdd(reinterpret_cast<unsigned long long*>(&g.counters[4]), static_cast<unsigned long long>(-1ll));
      atomicAdd(reinterpret_cast<unsigned long long*>(&g.counters[6]), 1ull);
    }
    return;
  }
  const bool complete = r.remaining == 0;
  const bool to_fused = complete && fuse && g.block_idx[b] + 1 < n_blocks;
  if (to_fused) {  // hand the finished block to the next forward's segment 0 and open the next block
    for (int q = lane; q < B; q += 32) {
      g.prev[b * B + q] = ids[q];
      ids[q] = mask_id;
      mask[q] = 1;
    }
  }
  __syncwarp();
  if (lane == 0) {
    atomicAdd(reinterpret_cast<unsigned long long*>(&g.counters[0]), 1ull);
    atomicAdd(reinterpret_cast<unsigned long long*>(&g.counters[2]), static_cast<unsigned long long>(r.committed));
    atomicAdd(reinterpret_cast<unsigned long long*>(&g.counters[3]), static_cast<unsigned long long>(r.forced));
    if (to_fused) {
      g.mode[b] = SEQ_FUSED;
      g.block_idx[b] += 1;
      g.step[b] = 0;
      atomicAdd(reinterpret_cast<unsigned long long*>(&g.counters[5]), 1ull);
    } else {
      g.step[b] = step;
      g.mode[b] = complete ? SEQ_FINALIZE : SEQ_DENOISE;
    }
  }
}

__global__ void gen_init_kernel(GenState g, int bs, int B, int mask_id, int gen_len) {
  const int b = blockIdx.x;
  for (int r = threadIdx.x; r < B; r += blockDim.x) {
    g.ids[b * B + r] = mask_id;
    g.mask[b * B + r] = 1;
  }
  // what is never decoded (early stop) reads as the mask id
  for (int r = threadIdx.x; r < gen_len; r += blockDim.x) g.out_ids[static_cast<size_t>(b) * gen_len + r] = mask_id;
  if (threadIdx.x == 0) {
    g.mode[b] = SEQ_DENOISE;
    g.block_idx[b] = 0;
    g.step[b] = 0;
    g.refresh_flag[b] = 0;
    if (b == 0) {
      g.counters[0] = g.counters[1] = g.counters[2] = g.counters[3] = g.counters[5] = g.counters[6] = g.counters[7] = 0;
      g.counters[4] = bs;
    }
  }
  if (b == 0)
    for (int i = threadIdx.x; i < COMMIT_HIST_BINS; i += blockDim.x) g.commit_hist[i] = 0ull;
}

// ----------------------------------------------------------------------------- multi-block decoding
// Several consecutive blocks of a sequence are in flight at once (Sec. 3.2, multi-block decoding): a
// window of up to `max_active` blocks starting at the first block that is not in the cache yet.  One
// round = one forward over the windows' rows (segment-limited attention: a block sees the cache,
// the earlier blocks of the window and itself) + this bookkeeping.
struct MbState {
  int* lo;          // [bs] first block in flight
  int* n_win;       // [bs] blocks in flight (0: the sequence is done)
  int* prefix_len;  // [bs]
  int* ids;         // [bs, W * B] the window's blocks, oldest first
  uint8_t* mask;    // [bs, W * B]
  int* fwd_ids;     // [bs, R] ids of the next forward
  int* out_ids;     // [bs, gen_len]
  int* commit_round;  // [bs, gen_len] or null
  long long* counters;  // [0] block decisions taken, [1] blocks stored in the cache, [2] tokens, [3] forced commits,
                        // [4] sequences not done, [5] largest window of the next round, [6] rows of valid work so far,
                        // [7] sequences stopped early on the end-of-sequence id
  int* stab;            // [bs, W] stabilizing forwards each block in flight has had
  int* hist;            // [bs, max_seq] ids of the stored prefix
  unsigned long long* commit_hist;  // [COMMIT_HIST_BINS] block decisions that committed k tokens
  uint32_t* error_word;
};
constexpr int MB_MAX_WINDOW = 8;

__global__ void mb_init_kernel(MbState g, int bs, int B, int W, int mask_id, int gen_len) {
  const int b = blockIdx.x;
  for (int r = threadIdx.x; r < W * B; r += blockDim.x) {
    g.ids[b * W * B + r] = mask_id;
    g.mask[b * W * B + r] = 1;
  }
  for (int r = threadIdx.x; r < gen_len; r += blockDim.x) g.out_ids[static_cast<size_t>(b) * gen_len + r] = mask_id;
  if (threadIdx.x < W) g.stab[b * W + threadIdx.x] = 0;
  if (threadIdx.x == 0) {
    g.lo[b] = 0;
    g.n_win[b] = 1;
    if (b == 0) {
      for (int i = 0; i < 8; ++i) g.counters[i] = 0;
      g.counters[4] = bs;
      g.counters[5] = 1;
    }
  }
  if (b == 0)
    for (int i = threadIdx.x; i < COMMIT_HIST_BINS; i += blockDim.x) g.commit_hist[i] = 0ull;
}

// Row map and input ids of the next round (rows_per_seq = R >= the largest window).  One block per sequence.
__global__ void mb_rowmap_kernel(MbState g, int bs, int B, int W, int R, int mask_id, int* pos_base, int* n_valid, int* kv_len) {
  const int b = blockIdx.x;
  const int rows = g.n_win[b] * B;
  if (threadIdx.x == 0) {
    pos_base[b] = g.prefix_len[b];
    n_valid[b] = rows;
    kv_len[b] = rows > 0 ? g.prefix_len[b] + rows : 0;
    if (b == 0) g.counters[5] = 0;  // the next round's largest window is gathered by mb_advance_kernel
  }
  for (int r = threadIdx.x; r < R; r += blockDim.x) g.fwd_ids[b * R + r] = r < rows ? g.ids[b * W * B + r] : mask_id;
}

// After the forward of a round.  States are read from the masks as they stood before the forward:
// a block without masks has just had a stabilizing forward (it is stored after `cache_delay` of
// them); a block whose predecessor in the
// window is at least 95 % unmasked (or that is the oldest) is Fully-Activated and commits at least
// one token; the others are Activated and commit only what clears the threshold.  Then the leading
// complete blocks enter the cache, and a new block is opened once the newest one is 10 % unmasked.
// One warp per sequence.
__global__ void mb_advance_kernel(MbState g, const float* __restrict__ conf, const float* __restrict__ ent,
                                  const int* __restrict__ argmax, int bs, int B, int W, int R, int n_blocks, int gen_len,
                                  float tau, int decide_mode, int mask_id, int max_active, int round, int cache_delay,
                                  int max_seq, int eos_id) {
  const int b = blockIdx.x;
  const int lane = threadIdx.x & 31;
  int n = g.n_win[b];
  if (n == 0) return;
  int* ids = g.ids + b * W * B;
  uint8_t* mask = g.mask + b * W * B;
  const int lo = g.lo[b];
  const int pl = g.prefix_len[b];
  int unmasked[MB_MAX_WINDOW], stab[MB_MAX_WINDOW];
#pragma unroll
  for (int w = 0; w < MB_MAX_WINDOW; ++w) stab[w] = w < n ? g.stab[b * W + w] : 0;
  __syncwarp();
#pragma unroll
  for (int w = 0; w < MB_MAX_WINDOW; ++w) {
    unmasked[w] = 0;
    if (w < n) {
      int cnt = 0;
      for (int r0 = 0; r0 < B; r0 += 32) {
        const int r = r0 + lane;
        cnt += __popc(__ballot_sync(0xffffffffu, r < B && mask[w * B + r] == 0));
      }
      unmasked[w] = cnt;
    }
  }
  // positions masked before the decisions (bit w * 4 + q = position lane + 32 q of block w): what is
  // unmasked afterwards was committed in this round
  unsigned was_masked = 0;
  if (eos_id >= 0) {
#pragma unroll
    for (int w = 0; w < MB_MAX_WINDOW; ++w)
#pragma unroll
      for (int q = 0; q < 4; ++q)
        if (w < n && lane + 32 * q < B && mask[w * B + lane + 32 * q] != 0) was_masked |= 1u << (w * 4 + q);
  }
  long long committed = 0, forced = 0, decisions = 0;
#pragma unroll
  for (int w = 0; w < MB_MAX_WINDOW; ++w) {
    if (w < n && unmasked[w] < B) {
      const bool fully = w == 0 || 100 * unmasked[w - 1] >= 95 * B;
      const int row0 = b * R + w * B;
      int* cr = g.commit_round ? g.commit_round + static_cast<size_t>(b) * gen_len + (lo + w) * B : nullptr;
      UnmaskOut r = unmask_block(conf + row0, ent + row0, argmax + row0, ids + w * B, mask + w * B, B, tau, decide_mode,
                                 nullptr, nullptr, cr, round, fully, g.error_word);
      if (lane == 0) atomicAdd(&g.commit_hist[r.committed], 1ull);
      committed += r.committed;
      forced += r.forced;
      decisions += 1;
    }
  }
  __syncwarp();
  // early stop: the end-of-sequence id was committed in this round.  Everything in flight goes out as
  // it stands (mask id where nothing was decided) and is not stored; the sequence is done.
  if (eos_id >= 0) {
    bool hit = false;
#pragma unroll
    for (int w = 0; w < MB_MAX_WINDOW; ++w)
#pragma unroll
      for (int q = 0; q < 4; ++q) {
        const int pos = w * B + lane + 32 * q;
        if ((was_masked >> (w * 4 + q)) & 1u)
          if (mask[pos] == 0 && ids[pos] == eos_id) hit = true;
      }
    if (__any_sync(0xffffffffu, hit)) {
      for (int r = lane; r < n * B; r += 32)
        g.out_ids[static_cast<size_t>(b) * gen_len + lo * B + r] = mask[r] ? mask_id : ids[r];
      if (lane == 0) {
        g.n_win[b] = 0;
        atomicAdd(reinterpret_cast<unsigned long long*>(&g.counters[0]), static_cast<unsigned long long>(decisions));
        atomicAdd(reinterpret_cast<unsigned long long*>(&g.counters[2]), static_cast<unsigned long long>(committed));
        atomicAdd(reinterpret_cast<unsigned long long*>(&g.counters[3]), static_cast<unsigned long long>(forced));
        atomicAdd(reinterpret_cast<unsigned long long*>(&g.counters[4]), static_cast<unsigned long long>(-1ll));
        atomicAdd(reinterpret_cast<unsigned long long*>(&g.counters[7]), 1ull);
      }
      return;
    }
  }
  // blocks that were complete before this forward have had one more stabilizing round; the leading
  // ones that have had cache_delay of them go out and into the cache
#pragma unroll
  for (int w = 0; w < MB_MAX_WINDOW; ++w)
    if (w < n && unmasked[w] == B) stab[w] += 1;
  int k = 0;
#pragma unroll
  for (int w = 0; w < MB_MAX_WINDOW; ++w)
    if (w == k && w < n && stab[w] >= cache_delay) ++k;
  for (int q = 0; q < k; ++q)
    for (int r = lane; r < B; r += 32) {
      g.out_ids[static_cast<size_t>(b) * gen_len + (lo + q) * B + r] = ids[q * B + r];
      g.hist[static_cast<size_t>(b) * max_seq + pl + q * B + r] = ids[q * B + r];
    }
  __syncwarp();
  if (k > 0) {
    const int left = (n - k) * B;
    for (int r0 = 0; r0 < left; r0 += 32) {  // move the rest of the window down: read, then write
      const int r = r0 + lane;
      int v = 0;
      uint8_t m = 0;
      if (r < left) { v = ids[k * B + r]; m = mask[k * B + r]; }
      __syncwarp();
      if (r < left) { ids[r] = v; mask[r] = m; }
      __syncwarp();
    }
#pragma unroll
    for (int w = 0; w < MB_MAX_WINDOW; ++w) {  // k is not a compile-time constant: select instead of indexing
      int v = 0;
#pragma unroll
      for (int u = 0; u < MB_MAX_WINDOW; ++u)
        if (u == w + k) v = stab[u];
      stab[w] = v;
    }
    n -= k;
  }
  // a new block once the newest one in flight is 10 % unmasked, or when nothing is in flight
  const int nxt = lo + k + n;
  if (nxt < n_blocks && n < max_active) {
    bool open = n == 0;
    if (!open) {
      int cnt = 0;
      for (int r0 = 0; r0 < B; r0 += 32) {
        const int r = r0 + lane;
        cnt += __popc(__ballot_sync(0xffffffffu, r < B && mask[(n - 1) * B + r] == 0));
      }
      open = 100 * cnt >= 10 * B;
    }
    if (open) {
      for (int r = lane; r < B; r += 32) {
        ids[n * B + r] = mask_id;
        mask[n * B + r] = 1;
      }
#pragma unroll
      for (int w = 0; w < MB_MAX_WINDOW; ++w)
        if (w == n) stab[w] = 0;
      ++n;
    }
  }
  __syncwarp();
  if (lane == 0) {
#pragma unroll
    for (int w = 0; w < MB_MAX_WINDOW; ++w)
      if (w < W) g.stab[b * W + w] = w < n ? stab[w] : 0;
    g.lo[b] = lo + k;
    g.n_win[b] = n;
    g.prefix_len[b] += k * B;
    atomicAdd(reinterpret_cast<unsigned long long*>(&g.counters[0]), static_cast<unsigned long long>(decisions));
    atomicAdd(reinterpret_cast<unsigned long long*>(&g.counters[1]), static_cast<unsigned long long>(k));
    atomicAdd(reinterpret_cast<unsigned long long*>(&g.counters[2]), static_cast<unsigned long long>(committed));
    atomicAdd(reinterpret_cast<unsigned long long*>(&g.counters[3]), static_cast<unsigned long long>(forced));
    if (n == 0) atomicAdd(reinterpret_cast<unsigned long long*>(&g.counters[4]), static_cast<unsigned long long>(-1ll));
    atomicMax(reinterpret_cast<unsigned long long*>(&g.counters[5]), static_cast<unsigned long long>(n));
  }
}

// The ids of the stored prefix are kept per sequence (prompt at prefill, every block when it is
// stored), so that the cache can be recomputed from them (KV-refresh, Sec. 3.2).
// hist[b, off_b + r] = src[b * src_stride + r] for r < count_b; off = 0 when `off` is null,
// count = fixed_count when `count` is null.  One block per sequence.
__global__ void hist_store_kernel(const int* __restrict__ src, int src_stride, const int* __restrict__ count, int fixed_count,
                                  const int* __restrict__ off, int* __restrict__ hist, int max_seq) {
  const int b = blockIdx.x;
  int n = count ? count[b] : fixed_count;
  const int o = off ? off[b] : 0;
  n = n < 0 ? 0 : (n > src_stride ? src_stride : n);
  if (o + n > max_seq) n = max_seq - o;
  for (int r = threadIdx.x; r < n; r += blockDim.x) hist[static_cast<size_t>(b) * max_seq + o + r] = src[static_cast<size_t>(b) * src_stride + r];
}
// Row map and input ids of a KV-refresh forward over the stored prefixes: rows_per_seq = p_max, rows
// [0, prefix_len_b) of a sequence that takes part (flag null or set; flags are cleared here) are valid
// and sit at positions 0.., the rest is padding.  prefix_len is left alone.  One block per sequence.
__global__ void refresh_rowmap_kernel(const int* __restrict__ hist, int max_seq, const int* __restrict__ prefix_len,
                                      int* flag, const int* __restrict__ active, int p_max, int pad_id, int* __restrict__ dst_ids,
                                      int* pos_base, int* n_valid, int* kv_len, long long* pending) {
  const int b = blockIdx.x;
  const bool take = (flag == nullptr || flag[b] != 0) && (active == nullptr || active[b] > 0);
  int len = take ? prefix_len[b] : 0;
  len = len > p_max ? p_max : len;
  __syncthreads();
  if (threadIdx.x == 0) {
    pos_base[b] = 0;
    n_valid[b] = len;
    kv_len[b] = len;
    if (flag) flag[b] = 0;
    if (pending && b == 0) *pending = 0;
  }
  for (int r = threadIdx.x; r < p_max; r += blockDim.x)
    dst_ids[static_cast<size_t>(b) * p_max + r] = r < len ? hist[static_cast<size_t>(b) * max_seq + r] : pad_id;
}

// ----------------------------------------------------------------------------- pseudo-trajectory (Sec. 3.1)
// rank[b, i] = decoding step, counted from 1 over the whole response, at which position i was
// unmasked, from the per-block step indices the generate loop records: a block's steps follow all
// steps of the blocks before it.  One warp per sequence; blocks are walked in order.
__global__ void trajectory_rank_kernel(const int* __restrict__ commit_step, int gen_len, int B, int* __restrict__ rank) {
  const int b = blockIdx.x, lane = threadIdx.x & 31;
  const int* cs = commit_step + static_cast<size_t>(b) * gen_len;
  int* out = rank + static_cast<size_t>(b) * gen_len;
  int done = 0;
  for (int j0 = 0; j0 < gen_len; j0 += B) {
    int mx = 0;
    for (int r = lane; r < B; r += 32) {
      const int v = cs[j0 + r];
      out[j0 + r] = done + v;
      mx = v > mx ? v : mx;
    }
#pragma unroll
    for (int o = 16; o > 0; o >>= 1) {
      const int other = __shfl_xor_sync(0xffffffffu, mx, o);
      mx = other > mx ? other : mx;
    }
    done += mx;
  }
}
// The noisy sequence of Sec. 3.1 for a batch: with positions counted from 1, window start s, window
// length k and m = ceil(k t), position i keeps y_i if i <= s, is the mask id if i > s + k, and in
// between keeps y_i iff the trajectory had unmasked it by step s + m (rank <= s + m).
// grid (ceil(n / 256), bs).
__global__ void noisy_sequence_kernel(const int* __restrict__ y, const int* __restrict__ rank, const int* __restrict__ s_arr,
                                      const int* __restrict__ k_arr, const int* __restrict__ m_arr, int n, int mask_id,
                                      int* __restrict__ out) {
  const int b = blockIdx.y;
  const int i0 = blockIdx.x * blockDim.x + threadIdx.x;  // position - 1
  if (i0 >= n) return;
  const int s = s_arr[b], k = k_arr[b], m = m_arr[b];
  const size_t at = static_cast<size_t>(b) * n + i0;
  const int i = i0 + 1;
  int v;
  if (i <= s) v = y[at];
  else if (i > s + k) v = mask_id;
  else v = rank[at] <= s + m ? y[at] : mask_id;
  out[at] = v;
}

// Row maps for the explicit API.
__global__ void decode_rowmap_kernel(const int* prefix_len, int bs, int B, int* pos_base, int* n_valid, int* kv_len) {
  const int b = blockIdx.x * blockDim.x + threadIdx.x;
  if (b >= bs) return;
  pos_base[b] = prefix_len[b];
  n_valid[b] = B;
  kv_len[b] = prefix_len[b] + B;
}
__global__ void prefill_rowmap_kernel(const int* prompt_lens, int bs, int p_max, int* prefix_len, int* pos_base,
                                      int* n_valid, int* kv_len) {
  const int b = blockIdx.x * blockDim.x + threadIdx.x;
  if (b >= bs) return;
  int len = prompt_lens[b];
  len = len < 0 ? 0 : (len > p_max ? p_max : len);
  prefix_len[b] = len;
  pos_base[b] = 0;
  n_valid[b] = len;
  kv_len[b] = len;
}
__global__ void add_prefix_kernel(int* prefix_len, int bs, int B) {
  const int b = blockIdx.x * blockDim.x + threadIdx.x;
  if (b < bs) prefix_len[b] += B;
}

template <typename T>
__global__ void cast_to_f32_kernel(const T* __restrict__ src, float* __restrict__ dst, size_t n) {
  size_t i = static_cast<size_t>(blockIdx.x) * blockDim.x + threadIdx.x;
  if (i < n) dst[i] = TypeOps<T>::to_f(src[i]);
}
template <typename T>
__global__ void cast_from_f32_kernel(const float* __restrict__ src, T* __restrict__ dst, size_t n) {
  size_t i = static_cast<size_t>(blockIdx.x) * blockDim.x + threadIdx.x;
  if (i < n) dst[i] = TypeOps<T>::from_f(src[i]);
}

// Weight repacking on the device: dst rows [r0, r0+rows) <- src rows; and gate/up interleave.
template <typename T>
__global__ void copy_rows_kernel(const T* __restrict__ src, T* __restrict__ dst, size_t n) {
  size_t i = static_cast<size_t>(blockIdx.x) * blockDim.x + threadIdx.x;
  if (i < n) dst[i] = src[i];
}
// dst [2f, d]: row 2j = gate row j, row 2j+1 = up row j.
template <typename T>
__global__ void interleave_gate_up_kernel(const T* __restrict__ gate, const T* __restrict__ up, T* __restrict__ dst,
                                          int f, int d) {
  const int row = blockIdx.x;  // 0 .. 2f-1 in dst
  const T* src = ((row & 1) ? up : gate) + static_cast<size_t>(row >> 1) * d;
  for (int i = threadIdx.x; i < d; i += blockDim.x) dst[static_cast<size_t>(row) * d + i] = src[i];
}
// Tiled weight layout for the tensor-core matmul: the [n, k] row-major matrix is cut into blocks of
// 128 rows x 64 columns, each stored contiguously (16 KB, rows of 128 bytes) in the order
// (row tile, column slab); rows and columns beyond n, k are zero.  Inside a block the eight 16-byte
// chunks of row r are stored at positions chunk ^ (r & 7): the 128-byte shared-memory swizzle that
// the MMA descriptors expect, applied once here, so that a plain bulk copy of the block is a ready
// operand tile.  A CTA that walks along K of one row tile reads one contiguous stretch of memory.
// grid (k_chunks, n_tiles), 256 threads.
__global__ void pack_tiled_kernel(const __nv_bfloat16* __restrict__ src, __nv_bfloat16* __restrict__ dst, int n, int k) {
  const int kc = blockIdx.x, nt = blockIdx.y, k_chunks = gridDim.x;
  uint4* out = reinterpret_cast<uint4*>(dst + (static_cast<size_t>(nt) * k_chunks + kc) * 128 * 64);
  for (int e = threadIdx.x; e < 128 * 8; e += blockDim.x) {  // 8 chunks of 8 elements per row
    const int r = e >> 3, ch = e & 7;
    const int row = nt * 128 + r, col = kc * 64 + ch * 8;
    uint4 v = make_uint4(0u, 0u, 0u, 0u);
    if (row < n) {
      const __nv_bfloat16* s = src + static_cast<size_t>(row) * k + col;
      if (col + 8 <= k && (k & 7) == 0) {
        v = *reinterpret_cast<const uint4*>(s);
      } else {
        __nv_bfloat16 t[8];
#pragma unroll
        for (int j = 0; j < 8; ++j) t[j] = (col + j < k) ? s[j] : __float2bfloat16_rn(0.f);
        v = *reinterpret_cast<uint4*>(t);
      }
    }
    out[r * 8 + (ch ^ (r & 7))] = v;
  }
}

// RoPE-pair packing of q / k projection rows: inside each head, dst row 2i = src row i and dst row
// 2i+1 = src row i + dh/2.
template <typename T>
__global__ void pack_rope_rows_kernel(const T* __restrict__ src, T* __restrict__ dst, int dh, int d) {
  const int row = blockIdx.x;  // dst row
  const int head = row / dh, w = row % dh;
  const int s = head * dh + (w >> 1) + (w & 1) * (dh / 2);
  for (int i = threadIdx.x; i < d; i += blockDim.x)
    dst[static_cast<size_t>(row) * d + i] = src[static_cast<size_t>(s) * d + i];
}

}  // namespace d3

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
      if (j0 + lane >= kv_len) s = -INFINITY;
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

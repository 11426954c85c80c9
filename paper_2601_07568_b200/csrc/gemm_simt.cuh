// Plain SIMT matmul Y[M,N] = X[M,K] . W[N,K]^T with fp32 accumulation and the same epilogues as the
// tensor-core kernel.  It is the fp32 path (TF32 tensor cores cannot hold 1e-4 relative on logits)
// and a debugging cross-check for bf16.  Tile 32 x 128, K slabs of 32, 256 threads, 4 x 4 outputs each.
#pragma once
#include "common.cuh"

namespace d3 {
namespace simt {

constexpr int BM = 32, BN = 128, BK = 32, THREADS = 256;

template <typename T, int EPI>
__global__ void __launch_bounds__(THREADS) gemm_simt_kernel(const T* __restrict__ X, const T* __restrict__ W, int M,
                                                            int N, int K, EpiParams ep) {
  __shared__ float Xs[BM][BK + 1];
  __shared__ float Ws[BN][BK + 1];
  __shared__ float Cs[BM][BN + 1];
  const int m0 = blockIdx.y * BM, n0 = blockIdx.x * BN;
  const int t = threadIdx.x, ty = t / 32, tx = t % 32;
  float acc[4][4];
#pragma unroll
  for (int i = 0; i < 4; ++i)
#pragma unroll
    for (int j = 0; j < 4; ++j) acc[i][j] = 0.f;

  for (int k0 = 0; k0 < K; k0 += BK) {
    for (int e = t; e < BM * BK; e += THREADS) {
      int r = e / BK, c = e % BK;
      int m = m0 + r, k = k0 + c;
      Xs[r][c] = (m < M && k < K) ? TypeOps<T>::to_f(X[static_cast<size_t>(m) * K + k]) : 0.f;
    }
    for (int e = t; e < BN * BK; e += THREADS) {
      int r = e / BK, c = e % BK;
      int n = n0 + r, k = k0 + c;
      Ws[r][c] = (n < N && k < K) ? TypeOps<T>::to_f(W[static_cast<size_t>(n) * K + k]) : 0.f;
    }
    __syncthreads();
#pragma unroll 8
    for (int kk = 0; kk < BK; ++kk) {
      float a[4], b[4];
#pragma unroll
      for (int i = 0; i < 4; ++i) a[i] = Xs[ty * 4 + i][kk];
#pragma unroll
      for (int j = 0; j < 4; ++j) b[j] = Ws[tx + 32 * j][kk];
#pragma unroll
      for (int i = 0; i < 4; ++i)
#pragma unroll
        for (int j = 0; j < 4; ++j) acc[i][j] = fmaf(a[i], b[j], acc[i][j]);
    }
    __syncthreads();
  }
#pragma unroll
  for (int i = 0; i < 4; ++i)
#pragma unroll
    for (int j = 0; j < 4; ++j) Cs[ty * 4 + i][tx + 32 * j] = acc[i][j];
  __syncthreads();

  if constexpr (EPI == EPI_F32 || EPI == EPI_RESID || EPI == EPI_T) {
    for (int e = t; e < BM * BN; e += THREADS) {
      int r = e / BN, c = e % BN;
      int m = m0 + r, n = n0 + c;
      if (m < M && n < N) {
        size_t o = static_cast<size_t>(m) * ep.ldy + n;
        if constexpr (EPI == EPI_F32) static_cast<float*>(ep.y)[o] = Cs[r][c] * ep.scale;
        else if constexpr (EPI == EPI_RESID) static_cast<float*>(ep.y)[o] += Cs[r][c];
        else static_cast<T*>(ep.y)[o] = TypeOps<T>::from_f(Cs[r][c]);
      }
    }
  } else if constexpr (EPI == EPI_SWIGLU) {
    // packed rows of W: 2j = gate row of hidden unit j, 2j+1 = its up row
    const int F = N / 2;
    for (int e = t; e < BM * 64; e += THREADS) {
      int r = e / 64, c = e % 64;
      int m = m0 + r, h = n0 / 2 + c;
      if (m < M && h < F)
        static_cast<T*>(ep.y)[static_cast<size_t>(m) * ep.ldy + h] =
            TypeOps<T>::from_f(silu_f(Cs[r][2 * c]) * Cs[r][2 * c + 1]);
    }
  } else if constexpr (EPI == EPI_STATS) {
    // one warp per row (8 warps, 4 rows each): lanes stride the 128 columns, fixed shuffle tree
    const int warp = t / 32, lane = t % 32;
    for (int r = warp; r < BM; r += THREADS / 32) {
      int m = m0 + r;
      SoftStat st = stat_empty();
      for (int c = lane; c < BN; c += 32) {
        int n = n0 + c;
        if (n < N && n != ep.mask_id) stat_add(st, Cs[r][c] * ep.scale, n);
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
      if (lane == 0 && m < M)
        ep.stat_part[static_cast<size_t>(m) * ep.n_tiles + blockIdx.x] =
            make_float4(st.m, st.z, st.s, __int_as_float(st.a));
      if (ep.sample_part != nullptr && m < M) {  // temperature sampling: largest l + T * g of the tile
        SampleStat sp = sample_empty();
        const SampleRow sr = sample_row(ep, m);
        for (int c = lane; c < BN; c += 32) {
          const int n = n0 + c;
          if (n < N && n != ep.mask_id) {
            const uint4 bits = philox4x32_10(make_uint4(static_cast<uint32_t>(n >> 2), sr.pos, sr.step, sr.seq), ep.seed_lo, ep.seed_hi);
            const uint32_t w = (n & 3) == 0 ? bits.x : (n & 3) == 1 ? bits.y : (n & 3) == 2 ? bits.z : bits.w;
            const float l = Cs[r][c] * ep.scale;
            sample_add(sp, __fadd_rn(l, __fmul_rn(ep.temperature, gumbel_from_bits(w))), l, n);
          }
        }
#pragma unroll
        for (int o = 16; o > 0; o >>= 1) {
          SampleStat other;
          other.pm = __shfl_xor_sync(0xffffffffu, sp.pm, o);
          other.la = __shfl_xor_sync(0xffffffffu, sp.la, o);
          other.pa = __shfl_xor_sync(0xffffffffu, sp.pa, o);
          sp = sample_merge(sp, other);
        }
        if (lane == 0)
          ep.sample_part[static_cast<size_t>(m) * ep.n_tiles + blockIdx.x] = make_float4(sp.pm, sp.la, __int_as_float(sp.pa), 0.f);
      }
    }
  }
}

}  // namespace simt
}  // namespace d3

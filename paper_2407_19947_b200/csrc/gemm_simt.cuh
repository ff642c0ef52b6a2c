// Plain SIMT weight-streaming GEMM for few rows: out[t, n] = sum_k A[t, k] * W[n, k].
//
// One warp per output feature n; the lanes stride the K dimension in 16-byte vectors and
// keep one fp32 accumulator per row; a butterfly reduction finishes the dot product.  The
// order of the additions for a given (t, n) depends on K only, never on how many rows are in
// the call or where the row sits, so stair rows and single-row greedy decoding agree bit
// for bit.  This is the reference GPU path (and the only one for fp32 weights); bf16 models
// use the tensor-core kernel when the shape allows.
#pragma once
#include <type_traits>

#include "common.cuh"

namespace stairs {

enum GemmEpilogue {
  EPI_STORE_F32 = 0,   // out_f32[t*ldo + n] = acc
  EPI_ADD_F32 = 1,     // out_f32[t*ldo + n] += acc                (residual update)
  EPI_GELU = 2,        // out_act[t*ldo + n] = gelu(acc)           (two-matrix MLP)
  EPI_SWIGLU = 3       // out_act[t*ldo + n] = silu(acc0) * acc1   (gate and up rows)
};

__device__ __forceinline__ float gelu_erf(float v) { return 0.5f * v * (1.0f + erff(v * 0.70710678118654752f)); }
__device__ __forceinline__ float silu_f(float v) { return v / (1.0f + expf(-v)); }

template <typename WT, int TT, bool DUAL>
__global__ void __launch_bounds__(256)
k_gemm_rows(const WT* __restrict__ W0, const WT* __restrict__ W1, const WT* __restrict__ A,
            int T, int N, int K, int epi, float* __restrict__ out_f32, WT* __restrict__ out_act, int ldo) {
  constexpr int VN = Vec16<WT>::N;
  const int lane = threadIdx.x & 31, warp = threadIdx.x >> 5;
  const int n = blockIdx.x * 8 + warp;
  const int t0 = blockIdx.y * TT;
  if (n >= N) return;
  float acc0[TT], acc1[TT];
#pragma unroll
  for (int t = 0; t < TT; ++t) { acc0[t] = 0.f; acc1[t] = 0.f; }
  const WT* w0 = W0 + (size_t)n * K;
  const WT* w1 = DUAL ? W1 + (size_t)n * K : nullptr;
  const WT* arow[TT];
#pragma unroll
  for (int t = 0; t < TT; ++t) arow[t] = A + (size_t)min(t0 + t, T - 1) * K;
#pragma unroll 2
  for (int k0 = lane * VN; k0 < K; k0 += 32 * VN) {
    float wv0[VN], wv1[VN];
    Vec16<WT>::load_stream(w0 + k0, wv0);
    if (DUAL) Vec16<WT>::load_stream(w1 + k0, wv1);
#pragma unroll
    for (int t = 0; t < TT; ++t) {
      float av[VN];
      Vec16<WT>::load(arow[t] + k0, av);
#pragma unroll
      for (int j = 0; j < VN; ++j) {
        acc0[t] = fmaf(wv0[j], av[j], acc0[t]);
        if (DUAL) acc1[t] = fmaf(wv1[j], av[j], acc1[t]);
      }
    }
  }
#pragma unroll
  for (int t = 0; t < TT; ++t) {
    acc0[t] = warp_sum(acc0[t]);
    if (DUAL) acc1[t] = warp_sum(acc1[t]);
  }
#pragma unroll
  for (int t = 0; t < TT; ++t) {
    if (lane == t && t0 + t < T) {
      const size_t o = (size_t)(t0 + t) * ldo + n;
      if (epi == EPI_STORE_F32) out_f32[o] = acc0[t];
      else if (epi == EPI_ADD_F32) out_f32[o] += acc0[t];
      else if (epi == EPI_GELU) out_act[o] = from_f32<WT>(gelu_erf(acc0[t]));
      else out_act[o] = from_f32<WT>(silu_f(acc0[t]) * acc1[t]);
    }
  }
}

template <typename WT, bool DUAL>
inline void launch_gemm_rows(cudaStream_t st, const WT* W0, const WT* W1, const WT* A, int T, int N,
                             int K, int epi, float* out_f32, WT* out_act, int ldo) {
  dim3 block(256);
  auto go = [&](auto tt) {
    constexpr int TT = decltype(tt)::value;
    dim3 grid((N + 7) / 8, (T + TT - 1) / TT);
    k_gemm_rows<WT, TT, DUAL><<<grid, block, 0, st>>>(W0, W1, A, T, N, K, epi, out_f32, out_act, ldo);
  };
  if (T <= 1) go(std::integral_constant<int, 1>());
  else if (T <= 2) go(std::integral_constant<int, 2>());
  else if (T <= 4) go(std::integral_constant<int, 4>());
  else go(std::integral_constant<int, 8>());
}

}  // namespace stairs

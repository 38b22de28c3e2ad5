// Importance Predictor head (Section 4.1, Eq. 7; Appendix A): a three-layer MLP d -> 2d -> d/2 -> 1
// on the final hidden state of each sequence.  With a decode batch of a few sequences every layer
// is a matrix-vector product bound by reading its bf16 weights once (6 d^2 bytes in all), so the
// kernels stream weight rows with 16-byte loads and do the arithmetic as fp32 FMAs; nothing here
// is shaped into a GEMM.
//
//   mlp_layer_kernel   y_part[ks][n][r] = sum over the K-slice ks of W[r][k] * x[n][k].
//                      grid = (row blocks of 64, K slices, batch tiles); 8 warps x 8 rows.  The
//                      input slice of the batch tile sits in shared memory as fp32.  The input is
//                      either the bf16 hidden state, or the previous layer's partial sums, which
//                      are reduced (fixed order), biased and activated while they are loaded -- so
//                      a layer split over K needs no reduction pass and no atomics.
//   mlp_head_kernel    the last layer (one output): one CTA per sequence.
#pragma once

#include "common.cuh"

namespace dynts {

constexpr int kMlpThreads = 256;
constexpr int kMlpRowsPerWarp = 8;
constexpr int kMlpRowsPerCta = (kMlpThreads / 32) * kMlpRowsPerWarp;  // 64
constexpr int kMlpBatchTile = 8;

struct MlpLayerParams {
  const __nv_bfloat16* W;   // [rows][K] row-major
  const __nv_bfloat16* xh;  // [Nb][K] bf16 input, or NULL
  const float* xparts;      // [n_parts][Nb][K] partial sums of the previous layer (when xh is NULL)
  const float* xbias;       // [K] or NULL, added to the reduced partial sums
  float* yparts;            // [k_slices][Nb][rows]
  int rows, K, Nb, n_parts, act, k_slice;  // k_slice = K / k_slices, a multiple of 256
};

__device__ __forceinline__ float mlp_act(float x, int act) { return act == 1 ? fmaxf(x, 0.f) : x; }

__global__ void __launch_bounds__(kMlpThreads) mlp_layer_kernel(const MlpLayerParams p) {
  extern __shared__ __align__(16) float sx[];  // [tile sequences][k_slice]
  const int tid = threadIdx.x, warp = tid >> 5, lane = tid & 31;
  const int ks = blockIdx.y;
  const int n0 = blockIdx.z * kMlpBatchTile;
  const int nt = min(kMlpBatchTile, p.Nb - n0);
  const int k0 = ks * p.k_slice;

  // input slice -> shared memory (fp32)
  for (int e = tid; e < nt * p.k_slice; e += kMlpThreads) {
    const int n = e / p.k_slice, k = e - n * p.k_slice;
    float v;
    if (p.xh) {
      v = __bfloat162float(p.xh[(size_t)(n0 + n) * p.K + k0 + k]);
    } else {
      v = 0.f;
      for (int q = 0; q < p.n_parts; ++q) v += p.xparts[((size_t)q * p.Nb + n0 + n) * p.K + k0 + k];
      if (p.xbias) v += p.xbias[k0 + k];
      v = mlp_act(v, p.act);
    }
    sx[e] = v;
  }
  __syncthreads();

  const int r0 = blockIdx.x * kMlpRowsPerCta + warp * kMlpRowsPerWarp;
  float acc[kMlpRowsPerWarp][kMlpBatchTile];
#pragma unroll
  for (int r = 0; r < kMlpRowsPerWarp; ++r)
#pragma unroll
    for (int n = 0; n < kMlpBatchTile; ++n) acc[r][n] = 0.f;

  // lane owns the 16-byte pieces lane, lane + 32, ... of the K-slice
  for (int c = lane; c * 8 < p.k_slice; c += 32) {
    uint4 w[kMlpRowsPerWarp];
#pragma unroll
    for (int r = 0; r < kMlpRowsPerWarp; ++r) {
      const int row = min(r0 + r, p.rows - 1);  // clamped: rows past the end are computed and dropped
      w[r] = ldg_stream(p.W + (size_t)row * p.K + k0 + c * 8);
    }
#pragma unroll
    for (int n = 0; n < kMlpBatchTile; ++n) {
      if (n < nt) {
        const float4 xa = *reinterpret_cast<const float4*>(sx + (size_t)n * p.k_slice + c * 8);
        const float4 xb = *reinterpret_cast<const float4*>(sx + (size_t)n * p.k_slice + c * 8 + 4);
#pragma unroll
        for (int r = 0; r < kMlpRowsPerWarp; ++r) {
          // a bf16 is the upper half of an fp32
          float a = acc[r][n];
          a = fmaf(__uint_as_float(w[r].x << 16), xa.x, a);
          a = fmaf(__uint_as_float(w[r].x & 0xffff0000u), xa.y, a);
          a = fmaf(__uint_as_float(w[r].y << 16), xa.z, a);
          a = fmaf(__uint_as_float(w[r].y & 0xffff0000u), xa.w, a);
          a = fmaf(__uint_as_float(w[r].z << 16), xb.x, a);
          a = fmaf(__uint_as_float(w[r].z & 0xffff0000u), xb.y, a);
          a = fmaf(__uint_as_float(w[r].w << 16), xb.z, a);
          a = fmaf(__uint_as_float(w[r].w & 0xffff0000u), xb.w, a);
          acc[r][n] = a;
        }
      }
    }
  }
  // reduce over the lanes; lane 0 writes
#pragma unroll
  for (int r = 0; r < kMlpRowsPerWarp; ++r) {
#pragma unroll
    for (int n = 0; n < kMlpBatchTile; ++n) {
      float a = acc[r][n];
#pragma unroll
      for (int o = 16; o > 0; o >>= 1) a += __shfl_xor_sync(0xffffffffu, a, o);
      if (lane == 0 && n < nt && r0 + r < p.rows) p.yparts[((size_t)ks * p.Nb + n0 + n) * p.rows + r0 + r] = a;
    }
  }
}

// score[n] = W3 . act(sum of partial sums + b2) + b3; one CTA per sequence.
__global__ void __launch_bounds__(256) mlp_head_kernel(const __nv_bfloat16* W3, const float* xparts, const float* xbias,
                                                       const float* b3, float* scores, int K, int Nb, int n_parts, int act) {
  const int n = blockIdx.x, tid = threadIdx.x;
  __shared__ float red[8];
  float a = 0.f;
  for (int k = tid; k < K; k += 256) {
    float v = 0.f;
    for (int q = 0; q < n_parts; ++q) v += xparts[((size_t)q * Nb + n) * K + k];
    if (xbias) v += xbias[k];
    a = fmaf(__bfloat162float(W3[k]), mlp_act(v, act), a);
  }
#pragma unroll
  for (int o = 16; o > 0; o >>= 1) a += __shfl_xor_sync(0xffffffffu, a, o);
  if ((tid & 31) == 0) red[tid >> 5] = a;
  __syncthreads();
  if (tid == 0) {
    float s = 0.f;
    for (int w = 0; w < 8; ++w) s += red[w];
    scores[n] = s + (b3 ? b3[0] : 0.f);
  }
}

}  // namespace dynts

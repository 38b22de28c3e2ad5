// Importance Predictor head (Section 4.1, Eq. 7; Appendix A): a three-layer MLP d -> 2d -> d/2 -> 1
// on the final hidden state of each sequence.  With a decode batch of a few sequences every layer
// is a matrix-vector product bound by reading its bf16 weights once (6 d^2 bytes in all), so the
// kernels stream weight rows with 16-byte loads and do the arithmetic as fp32 FMAs; nothing here
// is shaped into a GEMM.
//
//   mlp_layer_kernel   y_part[ks][n][r] = sum over the K-slice ks of W[r][k] * x[n][k].
//                      grid = (batch tiles, row blocks of 64, K slices); 8 warps x 8 rows.  The
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

// NT = sequences of the batch tile (1, 2, 4 or 8): the accumulators are [8 rows][NT] registers.
// grid = (batch tiles, row blocks, K slices): the tiles of one weight block run side by side and
// share its lines in L2.
template <int NT>
__global__ void __launch_bounds__(kMlpThreads, NT >= 4 ? 1 : 2) mlp_layer_kernel(const MlpLayerParams p) {
  extern __shared__ __align__(16) float sx[];  // [tile sequences][k_slice]
  const int tid = threadIdx.x, warp = tid >> 5, lane = tid & 31;
  const int ks = blockIdx.z;
  const int n0 = blockIdx.x * NT;
  const int nt = min(NT, p.Nb - n0);
  const int k0 = ks * p.k_slice;
  const int r0 = blockIdx.y * kMlpRowsPerCta + warp * kMlpRowsPerWarp;
  const int n_chunks = p.k_slice >> 3;  // 16-byte pieces of a row's K-slice; lane owns lane, lane + 32, ...

  auto load_w = [&](uint4 (&w)[kMlpRowsPerWarp], int c) {
#pragma unroll
    for (int r = 0; r < kMlpRowsPerWarp; ++r) {
      const int row = min(r0 + r, p.rows - 1);  // clamped: rows past the end are computed and dropped
      w[r] = ldg_stream(p.W + (size_t)row * p.K + k0 + c * 8);
    }
  };
  // The first weight pieces are requested before the input slice is staged: their latency overlaps it.
  uint4 wa[kMlpRowsPerWarp], wb[kMlpRowsPerWarp];
  if (lane < n_chunks) load_w(wa, lane);
  if (lane + 32 < n_chunks) load_w(wb, lane + 32);

  // input slice -> shared memory (fp32), eight elements per thread and step.  Piece c of sequence n
  // is stored as two float4: sxa[n * n_chunks + c] (elements 0-3) and sxb[...] (elements 4-7), so that
  // the lanes of a warp, which own consecutive pieces, read consecutive 16-byte words.  Sequences
  // past the end of the batch are zero.
  float4* sxa = reinterpret_cast<float4*>(sx);
  float4* sxb = sxa + (size_t)NT * n_chunks;
#pragma unroll 2
  for (int g = tid; g < NT * n_chunks; g += kMlpThreads) {
    const int n = g / n_chunks, c = g - n * n_chunks;
    float v[8];
#pragma unroll
    for (int i = 0; i < 8; ++i) v[i] = 0.f;
    if (n < nt) {
      const size_t off = (size_t)(n0 + n) * p.K + k0 + c * 8;
      if (p.xh) {
        const uint4 w = *reinterpret_cast<const uint4*>(p.xh + off);
        v[0] = __uint_as_float(w.x << 16); v[1] = __uint_as_float(w.x & 0xffff0000u);
        v[2] = __uint_as_float(w.y << 16); v[3] = __uint_as_float(w.y & 0xffff0000u);
        v[4] = __uint_as_float(w.z << 16); v[5] = __uint_as_float(w.z & 0xffff0000u);
        v[6] = __uint_as_float(w.w << 16); v[7] = __uint_as_float(w.w & 0xffff0000u);
      } else {
        for (int q = 0; q < p.n_parts; ++q) {
          const float4 a4 = *reinterpret_cast<const float4*>(p.xparts + (size_t)q * p.Nb * p.K + off);
          const float4 b4 = *reinterpret_cast<const float4*>(p.xparts + (size_t)q * p.Nb * p.K + off + 4);
          v[0] += a4.x; v[1] += a4.y; v[2] += a4.z; v[3] += a4.w;
          v[4] += b4.x; v[5] += b4.y; v[6] += b4.z; v[7] += b4.w;
        }
        if (p.xbias) {
          const float4 a4 = *reinterpret_cast<const float4*>(p.xbias + k0 + c * 8);
          const float4 b4 = *reinterpret_cast<const float4*>(p.xbias + k0 + c * 8 + 4);
          v[0] += a4.x; v[1] += a4.y; v[2] += a4.z; v[3] += a4.w;
          v[4] += b4.x; v[5] += b4.y; v[6] += b4.z; v[7] += b4.w;
        }
#pragma unroll
        for (int i = 0; i < 8; ++i) v[i] = mlp_act(v[i], p.act);
      }
    }
    sxa[g] = make_float4(v[0], v[1], v[2], v[3]);
    sxb[g] = make_float4(v[4], v[5], v[6], v[7]);
  }
  __syncthreads();

  float acc[kMlpRowsPerWarp][NT];
#pragma unroll
  for (int r = 0; r < kMlpRowsPerWarp; ++r)
#pragma unroll
    for (int n = 0; n < NT; ++n) acc[r][n] = 0.f;

  auto fma_chunk = [&](const uint4 (&w)[kMlpRowsPerWarp], int c) {
#pragma unroll
    for (int n = 0; n < NT; ++n) {
      const float4 xa = sxa[n * n_chunks + c];
      const float4 xb = sxb[n * n_chunks + c];
#pragma unroll
      for (int r = 0; r < kMlpRowsPerWarp; ++r) {
        float a = acc[r][n];  // a bf16 is the upper half of an fp32
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
  };
  // two pieces per row in flight per lane: compute one while the one after next is fetched
  for (int c = lane; c < n_chunks; c += 64) {
    fma_chunk(wa, c);
    if (c + 64 < n_chunks) load_w(wa, c + 64);
    if (c + 32 < n_chunks) {
      fma_chunk(wb, c + 32);
      if (c + 96 < n_chunks) load_w(wb, c + 96);
    }
  }
  // reduce over the lanes; lane 0 writes
#pragma unroll
  for (int r = 0; r < kMlpRowsPerWarp; ++r) {
#pragma unroll
    for (int n = 0; n < NT; ++n) {
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

// Importance Predictor head (Section 4.1, Eq. 7; Appendix A): a three-layer MLP d -> 2d -> d/2 -> 1
// on the final hidden state of each sequence.  With a decode batch of a few sequences every layer
// is bound by reading its bf16 weights once (6 d^2 bytes in all): the kernels stream weight rows
// with 16-byte loads straight into tensor-core fragments; the activations wait in shared memory.
//
//   mlp_layer_kernel   the K-slice ks of y[n][r] = act(b[r] + sum over k of W[r][k] * x[n][k]).
//                      grid = (batch tiles, row blocks of 64, K slices); 4 warps x 16 rows.  The
//                      input slice of the batch tile sits in shared memory as bf16 (an fp32 input
//                      as two bf16 halves).  The K slices of a row block form a thread-block
//                      cluster (up to 8): each CTA leaves its 64 x batch-tile partial sums in its
//                      shared memory, and after a cluster barrier every CTA sums, in the fixed order
//                      of the slices, its share of the rows over the cluster's shared memories, adds
//                      the bias, applies the activation and writes the finished values -- no
//                      partial sums in global memory, no atomics, no reduction pass, and the next
//                      layer stages one array.  This is the path of batches above 8, where every
//                      consumer CTA re-reducing the partial sums of 16 sequences costs more than the
//                      weights it reads; small batches (and layers too long for 8 slices) write
//                      partial sums to global memory, which the consumer reduces (fixed order),
//                      biases and activates while it stages them.
//   mlp_head_kernel    the last layer (one output): one CTA per sequence.
#pragma once

#include <cooperative_groups.h>

#include "common.cuh"

namespace dynts {

constexpr int kMlpWarps = 4;        // warps per CTA, 16 weight rows each
constexpr int kMlpRowsPerCta = 16 * kMlpWarps;
constexpr int kMlpBatchTile = 16;  // at most; 8 for batches up to 8

struct MlpLayerParams {
  const __nv_bfloat16* W;   // [rows][K] row-major
  const __nv_bfloat16* xh;  // [Nb][K] bf16 input, or NULL
  const float* xparts;      // [n_parts][Nb][K] partial sums of the previous layer (when xh is NULL)
  const float* xbias;       // [K] or NULL, added to the reduced partial sums
  float* yparts;            // [k_slices][Nb][rows] partial sums, or [Nb][rows] finished values (cluster_reduce)
  const float* ybias;       // [rows] or NULL: added to the finished values (cluster_reduce)
  int rows, K, Nb, n_parts, act, k_slice;  // k_slice = K / k_slices, a multiple of 256; act applies to the input
  int cluster_reduce;       // the K slices of a row block are one cluster (gridDim.z CTAs, a power of two <= 8)
  int yact;                 // activation of the finished values (cluster_reduce)
};

__device__ __forceinline__ float mlp_act(float x, int act) { return act == 1 ? fmaxf(x, 0.f) : x; }

// NB = blocks of 8 sequences per batch tile (1 or 2).  grid = (batch tiles, row blocks of 64, K
// slices): the tiles of one weight block run side by side and share its lines in L2.  4 warps, each
// 16 weight rows.
//
// The products run on the tensor pipe (mma.sync m16n8k16, bf16 x bf16 -> fp32): A = 16 weight rows,
// loaded from global memory straight into fragment registers as 16-byte pieces (a dot product does
// not care in which order k is summed, so the 8 consecutive elements a thread loads are declared
// to be its fragment's k-indices and the activations are read with the same permutation);
// B = the activations of 8 sequences.  fp32 activations are split into two bf16 halves, x = hi + lo
// with lo = bf16(x - hi), and multiplied in two mma, which keeps about 16 bits of x; a bf16 input
// (the hidden state) needs one.
constexpr int kMlpPad = 32;  // bf16 elements of padding per staged sequence: rows land in different banks

__device__ __forceinline__ void mlp_mma(float (&c)[4], uint32_t a0, uint32_t a1, uint32_t a2, uint32_t a3, uint32_t b0,
                                        uint32_t b1) {
  asm volatile(
      "mma.sync.aligned.m16n8k16.row.col.f32.bf16.bf16.f32 {%0,%1,%2,%3}, {%4,%5,%6,%7}, {%8,%9}, {%0,%1,%2,%3};"
      : "+f"(c[0]), "+f"(c[1]), "+f"(c[2]), "+f"(c[3])
      : "r"(a0), "r"(a1), "r"(a2), "r"(a3), "r"(b0), "r"(b1));
}

template <int NB, int WARPS>
__global__ void __launch_bounds__(WARPS * 32) mlp_layer_kernel(const MlpLayerParams p) {
  constexpr int kRows = 16 * WARPS;  // weight rows per CTA
  extern __shared__ __align__(16) __nv_bfloat16 sxh[];  // [8 NB sequences][k_slice + pad] hi, then the same for lo
  constexpr int NT = 8 * NB;
  const int tid = threadIdx.x, warp = tid >> 5, lane = tid & 31;
  const int gid = lane >> 2, tig = lane & 3;
  const int ks = blockIdx.z;
  const int n0 = blockIdx.x * NT;
  const int nt = min(NT, p.Nb - n0);
  const int k0 = ks * p.k_slice;
  const int r0 = blockIdx.y * kRows + warp * 16;
  const int n_chunks = p.k_slice >> 3;   // 16-byte pieces of a row's K-slice
  const int stride = p.k_slice + kMlpPad;  // staged row length in elements
  __nv_bfloat16* sxl = sxh + (size_t)NT * stride;
  const bool split = p.xh == nullptr;    // fp32 input: hi + lo

  const __nv_bfloat16* wrow0 = p.W + (size_t)min(r0 + gid, p.rows - 1) * p.K + k0;      // clamped rows are computed
  const __nv_bfloat16* wrow1 = p.W + (size_t)min(r0 + gid + 8, p.rows - 1) * p.K + k0;  // and dropped
  // Thread (gid, tig) owns the pieces tig + 4i of rows gid and gid + 8; a group of 4 i is one step.
  auto load_w = [&](uint4 (&w)[8], int step) {
#pragma unroll
    for (int i = 0; i < 4; ++i) {
      const int c = 16 * step + tig + 4 * i;
      w[2 * i] = ldg_stream(wrow0 + c * 8);
      w[2 * i + 1] = ldg_stream(wrow1 + c * 8);
    }
  };
  const int n_steps = n_chunks >> 4;  // k_slice is a multiple of 256 = 16 pieces x 2 ... host guarantees 128 | k_slice
  uint4 wa[8], wb[8];
  load_w(wa, 0);
  if (n_steps > 1) load_w(wb, 1);
  // The weights do not depend on the kernel before this one in the stream; the activations do
  // (launched with programmatic stream serialisation).  While it waits, the CTA asks the rest of its
  // weight slice into L2, so that HBM stays busy across the boundary between the two kernels.
  {
    const int lines = n_chunks >> 3;  // 128-byte lines per row of the slice
    for (int i = lane; i < 16 * lines; i += 32) {
      const int rr = min(r0 + i / lines, p.rows - 1), ln = i % lines;
      if (ln >= 4) asm volatile("prefetch.global.L2 [%0];" ::"l"(p.W + (size_t)rr * p.K + k0 + ln * 64));
    }
  }
  asm volatile("griddepcontrol.wait;" ::: "memory");

  // stage the input slice: 8 elements per thread and step
#pragma unroll 2
  // (Only the sequences that exist are staged: a column of the accumulator depends on its own
  // sequence alone, and the columns of the others are never written out.)
  for (int g = tid; g < nt * n_chunks; g += WARPS * 32) {
    const int n = g / n_chunks, c = g - n * n_chunks;
    uint4 hi = make_uint4(0u, 0u, 0u, 0u), lo = hi;
    {
      const size_t off = (size_t)(n0 + n) * p.K + k0 + c * 8;
      if (!split) {
        hi = *reinterpret_cast<const uint4*>(p.xh + off);
      } else {
        float v[8];
#pragma unroll
        for (int i = 0; i < 8; ++i) v[i] = 0.f;
        // The partial sums of four K-slices at a time: all their loads are issued before the first
        // addition (one after the other they cost a trip to L2 each: 32 us of a 72 us call at batch 16).
        // The order of the additions stays q = 0, 1, ...
        for (int q0 = 0; q0 < p.n_parts; q0 += 4) {
          float4 a4[4], b4[4];
#pragma unroll
          for (int u = 0; u < 4; ++u) {
            a4[u] = make_float4(0.f, 0.f, 0.f, 0.f);
            b4[u] = a4[u];
            if (q0 + u < p.n_parts) {
              a4[u] = *reinterpret_cast<const float4*>(p.xparts + (size_t)(q0 + u) * p.Nb * p.K + off);
              b4[u] = *reinterpret_cast<const float4*>(p.xparts + (size_t)(q0 + u) * p.Nb * p.K + off + 4);
            }
          }
#pragma unroll
          for (int u = 0; u < 4; ++u) {
            v[0] += a4[u].x; v[1] += a4[u].y; v[2] += a4[u].z; v[3] += a4[u].w;
            v[4] += b4[u].x; v[5] += b4[u].y; v[6] += b4[u].z; v[7] += b4[u].w;
          }
        }
        if (p.xbias) {
          const float4 a4 = *reinterpret_cast<const float4*>(p.xbias + k0 + c * 8);
          const float4 b4 = *reinterpret_cast<const float4*>(p.xbias + k0 + c * 8 + 4);
          v[0] += a4.x; v[1] += a4.y; v[2] += a4.z; v[3] += a4.w;
          v[4] += b4.x; v[5] += b4.y; v[6] += b4.z; v[7] += b4.w;
        }
        uint32_t hw[4], lw[4];
#pragma unroll
        for (int i = 0; i < 4; ++i) {
          const float x0 = mlp_act(v[2 * i], p.act), x1 = mlp_act(v[2 * i + 1], p.act);
          const __nv_bfloat16 h0 = __float2bfloat16_rn(x0), h1 = __float2bfloat16_rn(x1);
          const __nv_bfloat16 l0 = __float2bfloat16_rn(x0 - __bfloat162float(h0));
          const __nv_bfloat16 l1 = __float2bfloat16_rn(x1 - __bfloat162float(h1));
          hw[i] = (uint32_t)__bfloat16_as_ushort(h0) | ((uint32_t)__bfloat16_as_ushort(h1) << 16);
          lw[i] = (uint32_t)__bfloat16_as_ushort(l0) | ((uint32_t)__bfloat16_as_ushort(l1) << 16);
        }
        hi = make_uint4(hw[0], hw[1], hw[2], hw[3]);
        lo = make_uint4(lw[0], lw[1], lw[2], lw[3]);
      }
    }
    *reinterpret_cast<uint4*>(sxh + (size_t)n * stride + c * 8) = hi;
    if (split) *reinterpret_cast<uint4*>(sxl + (size_t)n * stride + c * 8) = lo;
  }
  __syncthreads();

  float acc[NB][4];
#pragma unroll
  for (int b = 0; b < NB; ++b)
#pragma unroll
    for (int e = 0; e < 4; ++e) acc[b][e] = 0.f;

  auto mma_step = [&](const uint4 (&w)[8], int step) {
#pragma unroll
    for (int i = 0; i < 4; ++i) {
      const int c = 16 * step + tig + 4 * i;
#pragma unroll
      for (int b = 0; b < NB; ++b) {
        const uint4 xh4 = *reinterpret_cast<const uint4*>(sxh + (size_t)(8 * b + gid) * stride + c * 8);
        mlp_mma(acc[b], w[2 * i].x, w[2 * i + 1].x, w[2 * i].y, w[2 * i + 1].y, xh4.x, xh4.y);
        mlp_mma(acc[b], w[2 * i].z, w[2 * i + 1].z, w[2 * i].w, w[2 * i + 1].w, xh4.z, xh4.w);
        if (split) {
          const uint4 xl4 = *reinterpret_cast<const uint4*>(sxl + (size_t)(8 * b + gid) * stride + c * 8);
          mlp_mma(acc[b], w[2 * i].x, w[2 * i + 1].x, w[2 * i].y, w[2 * i + 1].y, xl4.x, xl4.y);
          mlp_mma(acc[b], w[2 * i].z, w[2 * i + 1].z, w[2 * i].w, w[2 * i + 1].w, xl4.z, xl4.w);
        }
      }
    }
  };
  // two steps (2 x 8 pieces of 16 bytes per thread) in flight
  for (int st = 0; st < n_steps; st += 2) {
    mma_step(wa, st);
    if (st + 2 < n_steps) load_w(wa, st + 2);
    if (st + 1 < n_steps) {
      mma_step(wb, st + 1);
      if (st + 3 < n_steps) load_w(wb, st + 3);
    }
  }
  // accumulator: rows gid (c0, c1) and gid + 8 (c2, c3), sequences 2 tig and 2 tig + 1 of the block
  if (!p.cluster_reduce) {
#pragma unroll
    for (int b = 0; b < NB; ++b) {
#pragma unroll
      for (int e = 0; e < 4; ++e) {
        const int row = r0 + gid + (e >> 1) * 8, n = 8 * b + 2 * tig + (e & 1);
        if (row < p.rows && n < nt) p.yparts[((size_t)ks * p.Nb + n0 + n) * p.rows + row] = acc[b][e];
      }
    }
    return;
  }
  // The cluster's reduction: partial sums into this CTA's shared memory (over the staged input,
  // which every warp has finished reading), then rank r finishes rows [r, r + 1) * 64 / S of the block.
  namespace cg = cooperative_groups;
  cg::cluster_group cluster = cg::this_cluster();
  const int S = (int)gridDim.z;
  __syncthreads();
  float* red = reinterpret_cast<float*>(sxh);  // [64 rows][NT]
#pragma unroll
  for (int b = 0; b < NB; ++b) {
#pragma unroll
    for (int e = 0; e < 4; ++e) red[(warp * 16 + gid + (e >> 1) * 8) * NT + 8 * b + 2 * tig + (e & 1)] = acc[b][e];
  }
  cluster.sync();
  const int rows_per = kRows / S;
  for (int idx = tid; idx < rows_per * NT; idx += WARPS * 32) {
    const int rl = ks * rows_per + idx / NT, n = idx % NT;
    float v = 0.f;
    for (int q = 0; q < S; ++q) v += *cluster.map_shared_rank(red + rl * NT + n, q);
    const int row = blockIdx.y * kRows + rl;
    if (row < p.rows && n < nt) {
      if (p.ybias) v += p.ybias[row];
      p.yparts[(size_t)(n0 + n) * p.rows + row] = mlp_act(v, p.yact);
    }
  }
  cluster.sync();  // no CTA leaves while its shared memory is still being read
}

// score[n] = W3 . act(sum of partial sums + b2) + b3; one CTA per sequence.  A thread takes four
// consecutive inputs at a time and issues the loads of up to eight partial sums of them before it
// adds the first (in the order q = 0, 1, ...).
constexpr int kMlpHeadThreads = 512;

__global__ void __launch_bounds__(kMlpHeadThreads) mlp_head_kernel(const __nv_bfloat16* W3, const float* xparts, const float* xbias,
                                                                   const float* b3, float* scores, int K, int Nb, int n_parts,
                                                                   int act) {
  const int n = blockIdx.x, tid = threadIdx.x;
  __shared__ float red[kMlpHeadThreads / 32];
  asm volatile("griddepcontrol.wait;" ::: "memory");
  float a = 0.f;
  for (int k = 4 * tid; k < K; k += 4 * kMlpHeadThreads) {  // K is a multiple of 256
    float4 v = make_float4(0.f, 0.f, 0.f, 0.f);
    for (int q0 = 0; q0 < n_parts; q0 += 8) {
      float4 x[8];
#pragma unroll
      for (int u = 0; u < 8; ++u) {
        x[u] = make_float4(0.f, 0.f, 0.f, 0.f);
        if (q0 + u < n_parts) x[u] = *reinterpret_cast<const float4*>(xparts + ((size_t)(q0 + u) * Nb + n) * K + k);
      }
#pragma unroll
      for (int u = 0; u < 8; ++u) {
        v.x += x[u].x; v.y += x[u].y; v.z += x[u].z; v.w += x[u].w;
      }
    }
    if (xbias) {
      const float4 b = *reinterpret_cast<const float4*>(xbias + k);
      v.x += b.x; v.y += b.y; v.z += b.z; v.w += b.w;
    }
    const uint2 w = *reinterpret_cast<const uint2*>(W3 + k);
    a = fmaf(__uint_as_float(w.x << 16), mlp_act(v.x, act), a);
    a = fmaf(__uint_as_float(w.x & 0xffff0000u), mlp_act(v.y, act), a);
    a = fmaf(__uint_as_float(w.y << 16), mlp_act(v.z, act), a);
    a = fmaf(__uint_as_float(w.y & 0xffff0000u), mlp_act(v.w, act), a);
  }
#pragma unroll
  for (int o = 16; o > 0; o >>= 1) a += __shfl_xor_sync(0xffffffffu, a, o);
  if ((tid & 31) == 0) red[tid >> 5] = a;
  __syncthreads();
  if (tid == 0) {
    float s = 0.f;
    for (int w = 0; w < kMlpHeadThreads / 32; ++w) s += red[w];
    scores[n] = s + (b3 ? b3[0] : 0.f);
  }
}

}  // namespace dynts

// Prefill attention for sm_100a: every prompt position attends to the positions up to and
// including itself (Eq. 4-5 with t = 1..M), bf16, head_dim 128, grouped query heads.  This is the
// phase that fills the question window (Section 4.2); unlike the decode step it is a dense
// contraction (M x M x d per head), so all of it runs on the tensor pipe.
//
// One CTA = 64 query rows of one query head (4 warps x 16 rows); it walks the key/value rows in
// tiles of 64 up to the diagonal.  K and V tiles are staged in shared memory by 16-byte cp.async
// copies, double-buffered, with the 16-byte pieces of a row XOR-swizzled by the row index so that
// ldmatrix reads are bank-conflict-free.  S = Q K^T and O += P V are mma.sync m16n8k16 (bf16 in,
// fp32 accumulate); the S accumulators are re-used in registers as the A operand of the second
// product; the softmax is kept online per row (running max and sum, rescale of O).
#pragma once

#include <math_constants.h>

#include "common.cuh"
#include "decode_attn.cuh"  // mma_bf16_m16n8k16, pack_bf16x2

namespace dynts {

constexpr int kPfRows = 64;      // query rows per CTA and key rows per tile
constexpr int kPfThreads = 128;
constexpr int kPfTileBytes = kPfRows * 256;  // 64 rows x 128 bf16
constexpr int kPfSmemBytes = 4 * kPfTileBytes;  // K x 2, V x 2; the Q tile borrows the second K buffer until its fragments are in registers

struct PrefillAttnParams {
  const __nv_bfloat16* q;  // [L, Nb, Hq, T, 128]
  const __nv_bfloat16* k;  // [L, Nb, Hkv, T, 128]
  const __nv_bfloat16* v;
  __nv_bfloat16* out;      // [L, Nb, Hq, T, 128]
  int T, Hq, Hkv;
  float scale_log2;
};

__device__ __forceinline__ void cp_async_16(uint32_t dst, const void* src, bool valid) {
  const int bytes = valid ? 16 : 0;  // src-size 0: the destination is filled with zeros
  asm volatile("cp.async.cg.shared.global [%0], [%1], 16, %2;" ::"r"(dst), "l"(src), "r"(bytes) : "memory");
}
__device__ __forceinline__ void cp_async_commit() { asm volatile("cp.async.commit_group;" ::: "memory"); }
template <int N>
__device__ __forceinline__ void cp_async_wait() {
  asm volatile("cp.async.wait_group %0;" ::"n"(N) : "memory");
}
__device__ __forceinline__ void pf_ldmatrix_x4(uint32_t addr, uint32_t& r0, uint32_t& r1, uint32_t& r2, uint32_t& r3) {
  asm volatile("ldmatrix.sync.aligned.m8n8.x4.shared.b16 {%0,%1,%2,%3}, [%4];"
               : "=r"(r0), "=r"(r1), "=r"(r2), "=r"(r3)
               : "r"(addr));
}
__device__ __forceinline__ void pf_ldmatrix_x4_trans(uint32_t addr, uint32_t& r0, uint32_t& r1, uint32_t& r2, uint32_t& r3) {
  asm volatile("ldmatrix.sync.aligned.m8n8.x4.trans.shared.b16 {%0,%1,%2,%3}, [%4];"
               : "=r"(r0), "=r"(r1), "=r"(r2), "=r"(r3)
               : "r"(addr));
}

// Copies rows [row0, row0 + 64) of a [T][128] bf16 matrix into a swizzled tile: piece c (16 bytes)
// of tile row r lands at r * 256 + ((c ^ (r & 7)) * 16).  Rows at or beyond T become zeros.
__device__ __forceinline__ void pf_load_tile(uint32_t tile, const __nv_bfloat16* src, int row0, int T, int tid) {
#pragma unroll
  for (int i = 0; i < (kPfRows * 16) / kPfThreads; ++i) {
    const int e = tid + i * kPfThreads;
    const int r = e >> 4, c = e & 15;
    const bool ok = row0 + r < T;
    const __nv_bfloat16* s = src + (size_t)(ok ? row0 + r : 0) * 128 + c * 8;
    cp_async_16(tile + r * 256 + ((c ^ (r & 7)) << 4), s, ok);
  }
}

// grid = (query tiles, Hq, L * Nb); tiles are taken from the last (longest) to the first.
__global__ void __launch_bounds__(kPfThreads, 3) prefill_attn_kernel(const PrefillAttnParams p) {
  extern __shared__ __align__(128) uint8_t pf_smem[];
  const int tid = threadIdx.x, warp = tid >> 5, lane = tid & 31;
  const int gid = lane >> 2, tig = lane & 3;
  const int T = p.T;
  const int qt = (int)gridDim.x - 1 - (int)blockIdx.x;
  const int hq = blockIdx.y, lb = blockIdx.z;
  const int h = hq / (p.Hq / p.Hkv);
  const __nv_bfloat16* Q = p.q + ((size_t)lb * p.Hq + hq) * T * 128;
  const __nv_bfloat16* K = p.k + ((size_t)lb * p.Hkv + h) * T * 128;
  const __nv_bfloat16* V = p.v + ((size_t)lb * p.Hkv + h) * T * 128;
  __nv_bfloat16* O = p.out + ((size_t)lb * p.Hq + hq) * T * 128;
  const uint32_t sK = (uint32_t)__cvta_generic_to_shared(pf_smem), sV = sK + 2 * kPfTileBytes;  // two buffers each
  const uint32_t sQ = sK + kPfTileBytes;  // = K buffer 1, free until the first prefetch
  const int q0 = qt * kPfRows;

  pf_load_tile(sQ, Q, q0, T, tid);
  pf_load_tile(sK, K, 0, T, tid);
  pf_load_tile(sV, V, 0, T, tid);
  cp_async_commit();
  cp_async_wait<0>();
  __syncthreads();

  // Q fragments of this warp's 16 rows: A operand of all 8 k-steps
  uint32_t qa[8][4];
  {
    const int r = warp * 16 + ((lane >> 3) & 1) * 8 + (lane & 7);
#pragma unroll
    for (int kk = 0; kk < 8; ++kk) {
      const int c = 2 * kk + (lane >> 4);
      pf_ldmatrix_x4(sQ + r * 256 + ((c ^ (r & 7)) << 4), qa[kk][0], qa[kk][1], qa[kk][2], qa[kk][3]);
    }
  }
  __syncthreads();  // every warp has its Q fragments: the buffer may be overwritten by the first prefetch
  float o[16][4];
#pragma unroll
  for (int db = 0; db < 16; ++db)
#pragma unroll
    for (int e = 0; e < 4; ++e) o[db][e] = 0.f;
  float m_run[2] = {-CUDART_INF_F, -CUDART_INF_F}, l_run[2] = {0.f, 0.f};
  const int qi0 = q0 + warp * 16 + gid;  // this thread's rows: qi0 and qi0 + 8

  for (int kt = 0; kt <= qt; ++kt) {
    const int buf = kt & 1;
    if (kt < qt) {  // prefetch the next tile into the other buffer
      pf_load_tile(sK + (buf ^ 1) * kPfTileBytes, K, (kt + 1) * kPfRows, T, tid);
      pf_load_tile(sV + (buf ^ 1) * kPfTileBytes, V, (kt + 1) * kPfRows, T, tid);
      cp_async_commit();
      cp_async_wait<1>();
    } else {
      cp_async_wait<0>();
    }
    __syncthreads();
    const uint32_t tK = sK + buf * kPfTileBytes, tV = sV + buf * kPfTileBytes;

    // S = Q K^T: 8 blocks of 8 keys
    float sacc[8][4];
#pragma unroll
    for (int nb = 0; nb < 8; ++nb)
#pragma unroll
      for (int e = 0; e < 4; ++e) sacc[nb][e] = 0.f;
#pragma unroll
    for (int j = 0; j < 4; ++j) {  // pairs of key blocks
      const int r = 16 * j + (lane >> 4) * 8 + (lane & 7);
#pragma unroll
      for (int kk = 0; kk < 8; ++kk) {
        const int c = 2 * kk + ((lane >> 3) & 1);
        uint32_t b0, b1, b2, b3;
        pf_ldmatrix_x4(tK + r * 256 + ((c ^ (r & 7)) << 4), b0, b1, b2, b3);
        mma_bf16_m16n8k16(sacc[2 * j], qa[kk][0], qa[kk][1], qa[kk][2], qa[kk][3], b0, b1);
        mma_bf16_m16n8k16(sacc[2 * j + 1], qa[kk][0], qa[kk][1], qa[kk][2], qa[kk][3], b2, b3);
      }
    }
    // scale, causal mask (only the diagonal tile needs it), online softmax of rows qi0 and qi0 + 8
    float mx[2] = {-CUDART_INF_F, -CUDART_INF_F};
#pragma unroll
    for (int nb = 0; nb < 8; ++nb) {
#pragma unroll
      for (int e = 0; e < 4; ++e) {
        const int kj = kt * kPfRows + 8 * nb + 2 * tig + (e & 1);
        const int qi = qi0 + (e >> 1) * 8;
        float x = sacc[nb][e] * p.scale_log2;
        if (kt == qt && (kj > qi || kj >= T)) x = -CUDART_INF_F;
        sacc[nb][e] = x;
        mx[e >> 1] = fmaxf(mx[e >> 1], x);
      }
    }
    float corr[2], ms[2];
#pragma unroll
    for (int r = 0; r < 2; ++r) {
      mx[r] = fmaxf(mx[r], __shfl_xor_sync(0xffffffffu, mx[r], 1));
      mx[r] = fmaxf(mx[r], __shfl_xor_sync(0xffffffffu, mx[r], 2));
      const float mn = fmaxf(m_run[r], mx[r]);
      ms[r] = (mn == -CUDART_INF_F) ? 0.f : mn;  // a row past the end of the prompt sees nothing
      corr[r] = fast_exp2(m_run[r] - ms[r]);
      m_run[r] = mn;
    }
    float ls[2] = {0.f, 0.f};
    uint32_t pa[4][4];  // P as A fragments of the 4 k-steps (16 keys each)
#pragma unroll
    for (int nb = 0; nb < 8; ++nb) {
      const float p0 = fast_exp2(sacc[nb][0] - ms[0]), p1 = fast_exp2(sacc[nb][1] - ms[0]);
      const float p2 = fast_exp2(sacc[nb][2] - ms[1]), p3 = fast_exp2(sacc[nb][3] - ms[1]);
      ls[0] += p0 + p1;
      ls[1] += p2 + p3;
      pa[nb >> 1][(nb & 1) * 2] = pack_bf16x2(p0, p1);      // a0 / a2: row gid
      pa[nb >> 1][(nb & 1) * 2 + 1] = pack_bf16x2(p2, p3);  // a1 / a3: row gid + 8
    }
#pragma unroll
    for (int r = 0; r < 2; ++r) l_run[r] = l_run[r] * corr[r] + ls[r];
#pragma unroll
    for (int db = 0; db < 16; ++db) {
      o[db][0] *= corr[0];
      o[db][1] *= corr[0];
      o[db][2] *= corr[1];
      o[db][3] *= corr[1];
    }
    // O += P V
#pragma unroll
    for (int t = 0; t < 4; ++t) {
      const int r = 16 * t + ((lane >> 3) & 1) * 8 + (lane & 7);
#pragma unroll
      for (int cp = 0; cp < 8; ++cp) {
        const int c = 2 * cp + (lane >> 4);
        uint32_t b0, b1, b2, b3;
        pf_ldmatrix_x4_trans(tV + r * 256 + ((c ^ (r & 7)) << 4), b0, b1, b2, b3);
        mma_bf16_m16n8k16(o[2 * cp], pa[t][0], pa[t][1], pa[t][2], pa[t][3], b0, b1);
        mma_bf16_m16n8k16(o[2 * cp + 1], pa[t][0], pa[t][1], pa[t][2], pa[t][3], b2, b3);
      }
    }
    __syncthreads();  // the buffer is overwritten by the prefetch of the next iteration
  }

#pragma unroll
  for (int r = 0; r < 2; ++r) {
    l_run[r] += __shfl_xor_sync(0xffffffffu, l_run[r], 1);
    l_run[r] += __shfl_xor_sync(0xffffffffu, l_run[r], 2);
  }
#pragma unroll
  for (int r = 0; r < 2; ++r) {
    const int qi = qi0 + 8 * r;
    if (qi < T) {
      const float inv = 1.0f / l_run[r];
      __nv_bfloat16* row = O + (size_t)qi * 128;
#pragma unroll
      for (int db = 0; db < 16; ++db)
        *reinterpret_cast<uint32_t*>(row + 8 * db + 2 * tig) = pack_bf16x2(o[db][2 * r] * inv, o[db][2 * r + 1] * inv);
    }
  }
}

}  // namespace dynts

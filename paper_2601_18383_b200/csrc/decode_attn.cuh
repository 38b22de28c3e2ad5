// Fused decode attention + importance accumulation (Eq. 4-6) for sm_100a.
//
// Work decomposition.  One thread-block CLUSTER handles one slab (layer, sequence, KV head); the
// slab's rows are split into contiguous ranges, one per CTA of the cluster (split-K).  Each CTA
// streams its K/V rows once from HBM, keeps its logits in shared memory and produces a partial
// (max, sum, unnormalised output).  The CTAs then exchange the partials through distributed
// shared memory: every CTA derives the row-global softmax normaliser, turns its stored logits
// into final attention weights and does the single read-modify-write of its own score rows,
// while the output combine is divided among the CTAs.  No scratch in global memory, no float
// atomics: every score row and every output element has exactly one writer, so results are
// deterministic.
//
// Two compute variants share the epilogue:
//   * decode_attn_generic_kernel<T>: fp32 FMA, any head_dim <= 256, fp32 or bf16 slabs.
//   * decode_attn_mma_kernel: bf16, head_dim 128, G <= 8.  QK^T and PV run on the tensor pipe
//     (mma.sync m16n8k16, fp32 accumulate) with operands loaded straight from global memory
//     into fragment registers as 16-byte vectors.  This works because a dot product does not
//     care in which order the head_dim (for QK^T) or the tokens (for PV) are summed: each
//     thread's contiguous 16 bytes are simply declared to be the fragment's k-indices.
#pragma once

#include <cooperative_groups.h>
#include <math_constants.h>

#include <type_traits>

#include "common.cuh"

namespace dynts {

namespace cg = cooperative_groups;

struct UnitCoords {
  size_t slab;   // index into the full [L, Nb, Hkv] slab arrays
  size_t qoff;   // element offset of the group's first query head in q/out of this launch
  size_t kvoff;  // element offset of the slab's row in k_new/v_new of this launch
  int b;
};

__device__ __forceinline__ UnitCoords unit_coords(const DecodeParams& p, unsigned cluster_size) {
  const unsigned ul = blockIdx.x / cluster_size;
  const int h = ul % p.Hkv;
  const int b = (ul / p.Hkv) % p.Nb;
  const int lrel = ul / (p.Hkv * p.Nb);
  UnitCoords u;
  u.b = b;
  u.slab = ((size_t)(p.layer0 + lrel) * p.Nb + b) * p.Hkv + h;
  u.qoff = (((size_t)lrel * p.Nb + b) * p.Hkv + h) * (size_t)p.G * p.d;
  u.kvoff = (((size_t)lrel * p.Nb + b) * p.Hkv + h) * (size_t)p.d;
  return u;
}

// Rows [t_begin, t_end) of the slab (n rows after the append) that this CTA owns.
__device__ __forceinline__ bool cta_range(const DecodeParams& p, int n, unsigned rank, unsigned cluster_size,
                                          int& t_begin, int& t_end) {
  const int units = (n + 15) >> 4;
  const int per_rank = (units + (int)cluster_size - 1) / (int)cluster_size;
  const int span = per_rank * 16;
  t_begin = (int)rank * span;
  t_end = min(n, t_begin + span);
  if (t_end < t_begin) t_end = t_begin;
  return span <= p.tile_tokens;
}

// Cluster-wide softmax normalisation, output combine and score update.
//   part_m[g], part_l[g], part_O[g*d + c]: this CTA's partial (log2-domain max, sum of
//   exp2(e - max), unnormalised output).  tile[(j - t_begin)*G + g]: log2-domain logit e, or
//   (TILE_IS_P) exp2(e - part_m[g]).  All arrays sit at the same shared-memory offsets in every
//   CTA of the cluster.
template <typename T, bool TILE_IS_P>
__device__ __forceinline__ void cluster_epilogue(const DecodeParams& p, float* part_m, float* part_l, float* part_O,
                                                 float* fin_M, float* fin_f, const float* tile, int n_old,
                                                 int t_begin, int t_end, const UnitCoords& u) {
  cg::cluster_group cluster = cg::this_cluster();
  const unsigned S = cluster.num_blocks();
  const unsigned rank = cluster.block_rank();
  const int G = p.G, d = p.d;
  cluster.sync();  // every CTA's partial is in its shared memory

  if ((int)threadIdx.x < G) {
    const int g = threadIdx.x;
    float M = -CUDART_INF_F;
    for (unsigned r = 0; r < S; ++r) M = fmaxf(M, *cluster.map_shared_rank(part_m + g, r));
    float L = 0.f;
    for (unsigned r = 0; r < S; ++r) {
      const float mr = *cluster.map_shared_rank(part_m + g, r);
      const float lr = *cluster.map_shared_rank(part_l + g, r);
      L += lr * fast_exp2(mr - M);
    }
    fin_M[g] = M;
    fin_f[g] = 1.0f / L;
  }
  __syncthreads();

  // Output: element range divided among the CTAs of the cluster.
  {
    const int total = G * d;
    const int chunk = (total + (int)S - 1) / (int)S;
    const int e0 = (int)rank * chunk;
    const int e1 = min(total, e0 + chunk);
    T* out = reinterpret_cast<T*>(p.out) + u.qoff;
    for (int e = e0 + (int)threadIdx.x; e < e1; e += (int)blockDim.x) {
      const int g = e / d;
      const float M = fin_M[g];
      float acc = 0.f;
      for (unsigned r = 0; r < S; ++r) {
        const float mr = *cluster.map_shared_rank(part_m + g, r);
        const float orr = *cluster.map_shared_rank(part_O + e, r);
        acc += orr * fast_exp2(mr - M);
      }
      from_float(out + e, acc * fin_f[g] * p.out_scale);
    }
  }

  // Scores: final weights of this CTA's own rows (Eq. 6, summed over the group's heads).
  {
    float w[kMaxGroup], M[kMaxGroup];
#pragma unroll
    for (int g = 0; g < kMaxGroup; ++g) {
      if (g < G) {
        M[g] = fin_M[g];
        w[g] = TILE_IS_P ? fast_exp2(part_m[g] - fin_M[g]) * fin_f[g] : fin_f[g];
      } else {
        M[g] = 0.f;
        w[g] = 0.f;
      }
    }
    float* score = p.score + u.slab * (size_t)p.cap;
    float* comp = p.comp + u.slab * (size_t)p.cap;
    float* dout = p.delta_out ? p.delta_out + u.slab * (size_t)p.cap : nullptr;
    for (int j = t_begin + (int)threadIdx.x; j < t_end; j += (int)blockDim.x) {
      const float* t = tile + (size_t)(j - t_begin) * G;
      float dl = 0.f;
#pragma unroll
      for (int g = 0; g < kMaxGroup; ++g) {
        if (g < G) dl += TILE_IS_P ? t[g] * w[g] : fast_exp2(t[g] - M[g]) * w[g];
      }
      if (p.accumulate) {
        float s = (j == n_old) ? 0.f : score[j];
        float cc = (j == n_old) ? 0.f : comp[j];
        kahan_add(s, cc, dl);
        score[j] = s;
        comp[j] = cc;
      } else if (j == n_old) {  // external scores: the new row starts at 0 until the caller sets it
        score[j] = 0.f;
        comp[j] = 0.f;
      }
      if (dout) dout[j] = dl;
    }
  }
  cluster.sync();  // no CTA may exit while its shared memory is still being read remotely
}

// ---------------------------------------------------------------------------------------------
// Generic variant: fp32 FMA arithmetic, fp32 or bf16 slabs, head_dim <= 256 (multiple of 8).
// ---------------------------------------------------------------------------------------------
constexpr int kGenericThreads = 256;

// KV8: the slabs hold E4M3 codes (q, k_new, v_new, out stay of type T); the new row is encoded before
// anything reads it, so this step already sees the value later steps will see.
template <typename T, bool KV8 = false>
__global__ void __launch_bounds__(kGenericThreads) decode_attn_generic_kernel(const DecodeParams p) {
  using TS = typename std::conditional<KV8, uint8_t, T>::type;  // slab element
  cg::cluster_group cluster = cg::this_cluster();
  const unsigned S = cluster.num_blocks();
  const unsigned rank = cluster.block_rank();
  const UnitCoords u = unit_coords(p, S);
  if (!p.active[u.b]) {  // uniform over the cluster
    finish_ticket(p);
    return;
  }
  const int G = p.G, d = p.d;
  const int tid = threadIdx.x, warp = tid >> 5, lane = tid & 31;
  const int n_old = p.len[u.b];
  const int n = n_old + 1;
  int t_begin, t_end;
  const bool fits = cta_range(p, n, rank, S, t_begin, t_end);
  if (!fits || n > p.cap) {  // uniform over the cluster; the host mirror prevents it
    if (tid == 0) atomicOr(p.err, !fits ? kErrTileOverflow : kErrLenOverflow);
    finish_ticket(p);
    return;
  }

  extern __shared__ __align__(16) float smem[];
  float* part_m = smem;
  float* part_l = smem + 8;
  float* fin_M = smem + 16;
  float* fin_f = smem + 24;
  float* part_O = smem + 32;
  float* tile = part_O + G * d;
  float* sQ = tile + (size_t)p.tile_tokens * G;
  const int ncols = d;
  const int ngroups = kGenericThreads / ncols > 0 ? kGenericThreads / ncols : 1;
  float* stage = sQ + G * d;  // [ngroups][G][d]

  const T* q = reinterpret_cast<const T*>(p.q) + u.qoff;
  const T* knew = reinterpret_cast<const T*>(p.k_new) + u.kvoff;
  const T* vnew = reinterpret_cast<const T*>(p.v_new) + u.kvoff;
  TS* Ks = reinterpret_cast<TS*>(p.K) + u.slab * (size_t)p.cap * d;
  TS* Vs = reinterpret_cast<TS*>(p.V) + u.slab * (size_t)p.cap * d;
  auto slab_val = [](TS x) -> float {
    if constexpr (KV8) return e4m3_to_float(x);
    else return to_float(x);
  };

  for (int e = tid; e < G * d; e += kGenericThreads) sQ[e] = to_float(q[e]);
  // a1: append the new row (its score is written by the epilogue)
  if (n_old >= t_begin && n_old < t_end) {
    for (int c = tid; c < d; c += kGenericThreads) {
      if constexpr (KV8) {
        Ks[(size_t)n_old * d + c] = store_e4m3(to_float(knew[c]), p.k_scale);
        Vs[(size_t)n_old * d + c] = store_e4m3(to_float(vnew[c]), p.v_scale);
      } else {
        Ks[(size_t)n_old * d + c] = knew[c];
        Vs[(size_t)n_old * d + c] = vnew[c];
      }
    }
    if (tid == 0) p.pos[u.slab * (size_t)p.cap + n_old] = p.tot[u.b];
  }
  __syncthreads();

  // a2: logits, one warp per row
  for (int j = t_begin + warp; j < t_end; j += kGenericThreads / 32) {
    float acc[kMaxGroup];
#pragma unroll
    for (int g = 0; g < kMaxGroup; ++g) acc[g] = 0.f;
    for (int c = lane; c < d; c += 32) {
      float kv;
      if constexpr (KV8) kv = slab_val(Ks[(size_t)j * d + c]);  // the appended row was written by this CTA above
      else kv = (j == n_old) ? to_float(knew[c]) : slab_val(Ks[(size_t)j * d + c]);
#pragma unroll
      for (int g = 0; g < kMaxGroup; ++g)
        if (g < G) acc[g] = fmaf(kv, sQ[g * d + c], acc[g]);
    }
#pragma unroll
    for (int g = 0; g < kMaxGroup; ++g) {
      if (g < G) {
        float a = acc[g];
#pragma unroll
        for (int o = 16; o > 0; o >>= 1) a += __shfl_xor_sync(0xffffffffu, a, o);
        if (lane == 0) tile[(size_t)(j - t_begin) * G + g] = a * p.scale_log2;
      }
    }
  }
  __syncthreads();

  // a3: CTA-local max and sum per head; logits are replaced by exp2(e - max)
  for (int g = warp; g < G; g += kGenericThreads / 32) {
    float m = -CUDART_INF_F;
    for (int j = lane; j < t_end - t_begin; j += 32) m = fmaxf(m, tile[(size_t)j * G + g]);
#pragma unroll
    for (int o = 16; o > 0; o >>= 1) m = fmaxf(m, __shfl_xor_sync(0xffffffffu, m, o));
    float l = 0.f;
    for (int j = lane; j < t_end - t_begin; j += 32) {
      const float pj = fast_exp2(tile[(size_t)j * G + g] - m);
      tile[(size_t)j * G + g] = pj;
      l += pj;
    }
#pragma unroll
    for (int o = 16; o > 0; o >>= 1) l += __shfl_xor_sync(0xffffffffu, l, o);
    if (lane == 0) {
      part_m[g] = m;
      part_l[g] = l;
    }
  }
  __syncthreads();

  // a4: unnormalised output, thread = (row group, column)
  {
    const int tg = tid / ncols, c = tid % ncols;
    float acc[kMaxGroup];
#pragma unroll
    for (int g = 0; g < kMaxGroup; ++g) acc[g] = 0.f;
    if (tg < ngroups) {
      for (int j = t_begin + tg; j < t_end; j += ngroups) {
        float vv;
        if constexpr (KV8) vv = slab_val(Vs[(size_t)j * d + c]);
        else vv = (j == n_old) ? to_float(vnew[c]) : slab_val(Vs[(size_t)j * d + c]);
        const float* t = tile + (size_t)(j - t_begin) * G;
#pragma unroll
        for (int g = 0; g < kMaxGroup; ++g)
          if (g < G) acc[g] = fmaf(t[g], vv, acc[g]);
      }
#pragma unroll
      for (int g = 0; g < kMaxGroup; ++g)
        if (g < G) stage[((size_t)tg * G + g) * d + c] = acc[g];
    }
    __syncthreads();
    for (int e = tid; e < G * d; e += kGenericThreads) {
      float a = 0.f;
      for (int k = 0; k < ngroups; ++k) a += stage[(size_t)k * G * d + e];
      part_O[e] = a;
    }
  }
  // (the epilogue's first cluster.sync orders these writes before any read)
  cluster_epilogue<T, true>(p, part_m, part_l, part_O, fin_M, fin_f, tile, n_old, t_begin, t_end, u);
  finish_ticket(p);
}

inline size_t generic_smem_bytes(int G, int d, int tile_tokens) {
  const int ngroups = kGenericThreads / d > 0 ? kGenericThreads / d : 1;
  return sizeof(float) * (32 + (size_t)G * d + (size_t)tile_tokens * G + (size_t)G * d + (size_t)ngroups * G * d);
}

// ---------------------------------------------------------------------------------------------
// Tensor-pipe variant: bf16 slabs, head_dim 128, G <= 8.
// ---------------------------------------------------------------------------------------------
constexpr int kMmaWarps = 4;
constexpr int kMmaThreads = kMmaWarps * 32;

__device__ __forceinline__ void mma_bf16_m16n8k16(float (&c)[4], uint32_t a0, uint32_t a1, uint32_t a2, uint32_t a3,
                                                  uint32_t b0, uint32_t b1) {
  asm volatile(
      "mma.sync.aligned.m16n8k16.row.col.f32.bf16.bf16.f32 {%0,%1,%2,%3}, {%4,%5,%6,%7}, {%8,%9}, {%0,%1,%2,%3};"
      : "+f"(c[0]), "+f"(c[1]), "+f"(c[2]), "+f"(c[3])
      : "r"(a0), "r"(a1), "r"(a2), "r"(a3), "r"(b0), "r"(b1));
}

__device__ __forceinline__ uint32_t pack_bf16x2(float lo, float hi) {
  __nv_bfloat162 v = __floats2bfloat162_rn(lo, hi);
  return *reinterpret_cast<uint32_t*>(&v);
}

__device__ __forceinline__ uint32_t word_of(const uint4& v, int i) {
  return i == 0 ? v.x : (i == 1 ? v.y : (i == 2 ? v.z : v.w));
}

__global__ void __launch_bounds__(kMmaThreads, 3) decode_attn_mma_kernel(const DecodeParams p) {
  cg::cluster_group cluster = cg::this_cluster();
  const unsigned S = cluster.num_blocks();
  const unsigned rank = cluster.block_rank();
  const UnitCoords u = unit_coords(p, S);
  if (!p.active[u.b]) {
    finish_ticket(p);
    return;
  }
  constexpr int d = 128;
  const int G = p.G;
  const int tid = threadIdx.x, warp = tid >> 5, lane = tid & 31;
  const int gid = lane >> 2, tig = lane & 3;
  const int n_old = p.len[u.b];
  const int n = n_old + 1;
  int t_begin, t_end;
  const bool fits = cta_range(p, n, rank, S, t_begin, t_end);
  if (!fits || n > p.cap) {
    if (tid == 0) atomicOr(p.err, !fits ? kErrTileOverflow : kErrLenOverflow);
    finish_ticket(p);
    return;
  }

  extern __shared__ __align__(16) float smem[];
  float* part_m = smem;
  float* part_l = smem + 8;
  float* fin_M = smem + 16;
  float* fin_f = smem + 24;
  float* part_O = smem + 32;
  float* tile = part_O + G * d;
  float* wm = tile + (((size_t)p.tile_tokens * G + 3) & ~(size_t)3);  // [warps][8]
  float* wl = wm + kMmaWarps * 8;
  float* wO = wl + kMmaWarps * 8;  // [warps][8][128]

  const __nv_bfloat16* q = reinterpret_cast<const __nv_bfloat16*>(p.q) + u.qoff;
  const __nv_bfloat16* knew = reinterpret_cast<const __nv_bfloat16*>(p.k_new) + u.kvoff;
  const __nv_bfloat16* vnew = reinterpret_cast<const __nv_bfloat16*>(p.v_new) + u.kvoff;
  __nv_bfloat16* Ks = reinterpret_cast<__nv_bfloat16*>(p.K) + u.slab * (size_t)p.cap * d;
  __nv_bfloat16* Vs = reinterpret_cast<__nv_bfloat16*>(p.V) + u.slab * (size_t)p.cap * d;

  // a1: append.  Readers of row n_old take it from k_new/v_new directly, so the slab write
  // below is never read back inside this launch.
  if (n_old >= t_begin && n_old < t_end) {
    if (tid < 16) {
      reinterpret_cast<uint4*>(Ks + (size_t)n_old * d)[tid] = reinterpret_cast<const uint4*>(knew)[tid];
    } else if (tid < 32) {
      reinterpret_cast<uint4*>(Vs + (size_t)n_old * d)[tid - 16] = reinterpret_cast<const uint4*>(vnew)[tid - 16];
    } else if (tid == 32) {
      p.pos[u.slab * (size_t)p.cap + n_old] = p.tot[u.b];
    }
  }

  // Query fragments.  Thread (gid, tig) holds, of query head gid, the 16-byte chunks tig + 4i:
  // the words of chunk i are the A-fragment k-pairs of k-steps 2i and 2i+1.
  uint32_t qa[8][2];
#pragma unroll
  for (int i = 0; i < 4; ++i) {
    uint4 w = make_uint4(0u, 0u, 0u, 0u);
    if (gid < G) w = *reinterpret_cast<const uint4*>(q + (size_t)gid * d + (tig + 4 * i) * 8);
    qa[2 * i][0] = w.x;
    qa[2 * i][1] = w.y;
    qa[2 * i + 1][0] = w.z;
    qa[2 * i + 1][1] = w.w;
  }

  float o[8][4];
#pragma unroll
  for (int mb = 0; mb < 8; ++mb)
#pragma unroll
    for (int e = 0; e < 4; ++e) o[mb][e] = 0.f;
  float m_run = -CUDART_INF_F, l_part = 0.f;

  const int u_begin = t_begin >> 4;
  const int u_end = (t_end + 15) >> 4;
  uint4 kb[2][4], vb[4][2];
  const uint4 zero4 = make_uint4(0u, 0u, 0u, 0u);

  auto load_k = [&](int un) {
#pragma unroll
    for (int nb = 0; nb < 2; ++nb) {
      const int tok = un * 16 + nb * 8 + gid;
      const __nv_bfloat16* row = (tok == n_old) ? knew : Ks + (size_t)tok * d;
      const bool ok = tok < t_end;
#pragma unroll
      for (int i = 0; i < 4; ++i) kb[nb][i] = ok ? ldg_stream(row + (tig + 4 * i) * 8) : zero4;
    }
  };
  auto load_v = [&](int un) {
#pragma unroll
    for (int k = 0; k < 4; ++k) {
      const int tok = un * 16 + 2 * tig + (k & 1) + ((k >> 1) << 3);
      const __nv_bfloat16* row = (tok == n_old) ? vnew : Vs + (size_t)tok * d;
      const bool ok = tok < t_end;
#pragma unroll
      for (int j = 0; j < 2; ++j) vb[k][j] = ok ? ldg_stream(row + (gid + 8 * j) * 8) : zero4;
    }
  };

  int un = u_begin + warp;
  if (un < u_end) load_k(un);
  for (; un < u_end; un += kMmaWarps) {
    load_v(un);
    // a2: S^T[head][token] = Q K^T for two blocks of 8 tokens
    float s0[4] = {0.f, 0.f, 0.f, 0.f}, s1[4] = {0.f, 0.f, 0.f, 0.f};
#pragma unroll
    for (int i = 0; i < 4; ++i) {
      mma_bf16_m16n8k16(s0, qa[2 * i][0], 0u, qa[2 * i][1], 0u, kb[0][i].x, kb[0][i].y);
      mma_bf16_m16n8k16(s0, qa[2 * i + 1][0], 0u, qa[2 * i + 1][1], 0u, kb[0][i].z, kb[0][i].w);
      mma_bf16_m16n8k16(s1, qa[2 * i][0], 0u, qa[2 * i][1], 0u, kb[1][i].x, kb[1][i].y);
      mma_bf16_m16n8k16(s1, qa[2 * i + 1][0], 0u, qa[2 * i + 1][1], 0u, kb[1][i].z, kb[1][i].w);
    }
    if (un + kMmaWarps < u_end) load_k(un + kMmaWarps);

    // a3: online softmax for head gid over this unit's 16 tokens
    const int tk = un * 16 + 2 * tig;
    float x[4];
    x[0] = (gid < G && tk < t_end) ? s0[0] * p.scale_log2 : -CUDART_INF_F;
    x[1] = (gid < G && tk + 1 < t_end) ? s0[1] * p.scale_log2 : -CUDART_INF_F;
    x[2] = (gid < G && tk + 8 < t_end) ? s1[0] * p.scale_log2 : -CUDART_INF_F;
    x[3] = (gid < G && tk + 9 < t_end) ? s1[1] * p.scale_log2 : -CUDART_INF_F;
    if (gid < G) {
      float* t = tile + (size_t)(tk - t_begin) * G + gid;
      if (tk < t_end) t[0] = x[0];
      if (tk + 1 < t_end) t[G] = x[1];
      if (tk + 8 < t_end) t[8 * G] = x[2];
      if (tk + 9 < t_end) t[9 * G] = x[3];
    }
    float um = fmaxf(fmaxf(x[0], x[1]), fmaxf(x[2], x[3]));
    um = fmaxf(um, __shfl_xor_sync(0xffffffffu, um, 1));
    um = fmaxf(um, __shfl_xor_sync(0xffffffffu, um, 2));
    const float m_new = fmaxf(m_run, um);
    const float m_safe = (m_new == -CUDART_INF_F) ? 0.f : m_new;
    const float corr = fast_exp2(m_run - m_safe);
    const float p0 = fast_exp2(x[0] - m_safe), p1 = fast_exp2(x[1] - m_safe);
    const float p2 = fast_exp2(x[2] - m_safe), p3 = fast_exp2(x[3] - m_safe);
    l_part = l_part * corr + ((p0 + p1) + (p2 + p3));
    m_run = m_new;
    const uint32_t pb0 = pack_bf16x2(p0, p1);  // B fragment: tokens 2tig, 2tig+1, head gid
    const uint32_t pb1 = pack_bf16x2(p2, p3);  // tokens 2tig+8, 2tig+9

    // rescale the output accumulators: columns are heads 2tig and 2tig+1
    const float c_even = __shfl_sync(0xffffffffu, corr, 8 * tig);
    const float c_odd = __shfl_sync(0xffffffffu, corr, 8 * tig + 4);
#pragma unroll
    for (int mb = 0; mb < 8; ++mb) {
      o[mb][0] *= c_even;
      o[mb][1] *= c_odd;
      o[mb][2] *= c_even;
      o[mb][3] *= c_odd;
    }

    // a4: O^T[d][head] += V^T P.  Thread (gid, tig) holds rows 2tig, 2tig+1, 2tig+8, 2tig+9 of V
    // at the 16-byte chunks gid and gid+8; byte permutes pair two tokens of one column.
#pragma unroll
    for (int j = 0; j < 2; ++j) {
#pragma unroll
      for (int qq = 0; qq < 4; ++qq) {
        const uint32_t w0 = word_of(vb[0][j], qq), w1 = word_of(vb[1][j], qq);
        const uint32_t w2 = word_of(vb[2][j], qq), w3 = word_of(vb[3][j], qq);
        const uint32_t a0 = __byte_perm(w0, w1, 0x5410);
        const uint32_t a1 = __byte_perm(w0, w1, 0x7632);
        const uint32_t a2 = __byte_perm(w2, w3, 0x5410);
        const uint32_t a3 = __byte_perm(w2, w3, 0x7632);
        mma_bf16_m16n8k16(o[4 * j + qq], a0, a1, a2, a3, pb0, pb1);
      }
    }
  }

  // Warp partials to shared memory.  Accumulator o[4j+qq] holds columns 8*(gid+8j) + 2qq (+1)
  // for heads 2tig (elements 0, 2) and 2tig+1 (elements 1, 3).
  l_part += __shfl_xor_sync(0xffffffffu, l_part, 1);
  l_part += __shfl_xor_sync(0xffffffffu, l_part, 2);
  if (tig == 0) {
    wm[warp * 8 + gid] = m_run;
    wl[warp * 8 + gid] = l_part;
  }
#pragma unroll
  for (int j = 0; j < 2; ++j) {
    float* base0 = wO + ((size_t)warp * 8 + 2 * tig) * d + 8 * (gid + 8 * j);
    float* base1 = base0 + d;
    reinterpret_cast<float4*>(base0)[0] = make_float4(o[4 * j][0], o[4 * j][2], o[4 * j + 1][0], o[4 * j + 1][2]);
    reinterpret_cast<float4*>(base0)[1] =
        make_float4(o[4 * j + 2][0], o[4 * j + 2][2], o[4 * j + 3][0], o[4 * j + 3][2]);
    reinterpret_cast<float4*>(base1)[0] = make_float4(o[4 * j][1], o[4 * j][3], o[4 * j + 1][1], o[4 * j + 1][3]);
    reinterpret_cast<float4*>(base1)[1] =
        make_float4(o[4 * j + 2][1], o[4 * j + 2][3], o[4 * j + 3][1], o[4 * j + 3][3]);
  }
  __syncthreads();
  // CTA partial = warps combined
  for (int e = tid; e < G * d; e += kMmaThreads) {
    const int g = e >> 7, c = e & 127;
    float mc = -CUDART_INF_F;
#pragma unroll
    for (int w = 0; w < kMmaWarps; ++w) mc = fmaxf(mc, wm[w * 8 + g]);
    const float ms = (mc == -CUDART_INF_F) ? 0.f : mc;
    float acc = 0.f;
#pragma unroll
    for (int w = 0; w < kMmaWarps; ++w) acc += wO[((size_t)w * 8 + g) * d + c] * fast_exp2(wm[w * 8 + g] - ms);
    part_O[e] = acc;
    if (c == 0) {
      float l = 0.f;
#pragma unroll
      for (int w = 0; w < kMmaWarps; ++w) l += wl[w * 8 + g] * fast_exp2(wm[w * 8 + g] - ms);
      part_m[g] = mc;
      part_l[g] = l;
    }
  }
  cluster_epilogue<__nv_bfloat16, false>(p, part_m, part_l, part_O, fin_M, fin_f, tile, n_old, t_begin, t_end, u);
  finish_ticket(p);
}

inline size_t mma_smem_bytes(int G, int tile_tokens) {
  const size_t tile = ((size_t)tile_tokens * G + 3) & ~(size_t)3;
  return sizeof(float) * (32 + (size_t)G * 128 + tile + 2 * kMmaWarps * 8 + (size_t)kMmaWarps * 8 * 128);
}

}  // namespace dynts

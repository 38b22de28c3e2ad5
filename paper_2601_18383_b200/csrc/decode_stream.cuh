// Persistent streaming variant of the fused decode attention + importance accumulation
// (Eq. 4-6) for sm_100a: bf16 or 8-bit (E4M3) slabs, head_dim 128, G <= 8.
//
// Work decomposition.  Every slab (layer, sequence, KV head) of n rows is cut into chunks of 32
// rows; the chunks of all slabs of the launch form one list, ordered slab by slab, and the
// persistent grid (two CTAs per SM) cuts that list into equal contiguous pieces, one per CTA
// ("stream-K": a CTA usually starts in the middle of one slab, covers some slabs completely and
// stops in the middle of another; when all slabs are equally long and there are at least about as
// many as CTAs, a piece is a whole number of slabs instead and no slab is shared).  Inside a CTA
// one producer thread walks the piece and issues TMA tile loads (cp.async.bulk.tensor.3d over one
// tensor map [K|V][rows][128], 128-byte swizzle, each tile to one CTA only): one load brings the K
// box and the V box of a chunk (two loads for bf16 rows, one per half of head_dim) into a
// shared-memory ring (6 stages of 16 KB; 12 of 8 KB for 8-bit rows) with a "full" mbarrier per
// stage and an "empty" mbarrier per group of stages, running ahead of the four consumer warps
// across chunk and slab boundaries, so the HBM stream never pauses for an epilogue.  The producer
// thread's own latency bounds a CTA (a barrier wait costs it about 300 cycles even on a completed
// phase, arming a stage and issuing a load about 100), hence the grouped waits, the combined
// loads and a per-chunk loop that carries only counters.  Chunk i of a CTA goes to stage
// i mod NS and to the warp pair i mod 2; with an even stage count every stage is always consumed
// by the same two warps, which is what makes the parity wait on its barrier unambiguous (a
// waiter is never two phases away from the barrier).  The consumer warps take 16 rows each:
// K Q^T (the unit's 16 tokens on M, the heads on N) and V^T P (head_dim on M, the heads on N) run
// on the tensor pipe (mma.sync m16n8k16, fp32 accumulate, 16 mma per unit) with operands
// fetched by ldmatrix from the swizzled tiles; online softmax in registers, P transposed by
// movmatrix.  The rows per slab of every sequence normally come with the launch (DecodeParams::
// n_host), so the kernel reads no length from global memory and needs no ticket at its end.
//
// The final softmax normaliser of a slab is known only when all its chunks are done, and the
// importance score needs the normalised weights (Eq. 6).  So every row's scaled logits go to a
// scratch array (fp32, [slab][head][row], 4*G bytes per row beside the 512 bytes of K and V), and
// each CTA that finishes its part of a slab publishes a partial (max, sum, unnormalised output)
// and takes a ticket on the slab's arrival counter.  Whoever arrives last combines the partials,
// writes the output and then walks the slab's logits once to do the single read-modify-write of
// every score row.  Nobody ever waits for another CTA: there is no inter-CTA spin, no float
// atomic, one writer per score row and per output element.  While a CTA still has chunks to
// stream, that pass is handed to a sixth warp (the scorer) through a two-slot task queue in shared
// memory, so the consumer warps go straight on to the next slab.  The pass after a CTA's last chunk
// has nothing left to overlap with: with whole-slab pieces it is recorded instead (DecodeParams::
// defer) and applied by the scorer warp of the next launch, or by the eviction kernel.
//
// 8-bit slabs (KV8 = true): a stage holds one 32 x 128-byte box of K codes and one of V codes.
// ldmatrix moves bytes, so the same 8 x 16-byte matrices are fetched; a thread's 32-bit register
// then holds four codes, which cvt.rn.f16x2.e4m3x2 turns (exactly) into two f16 pairs, and the
// products run as f16 mma with fp32 accumulation.  For Q K^T the four codes of a register are four
// consecutive head_dim indices of one token; a dot product does not care in which order head_dim
// is summed, so the query fragment is simply loaded with the same permutation.  For P V the
// transposed ldmatrix pairs two tokens of two adjacent columns in a register; a byte permute
// regroups them into (token, token+1) pairs per column, and the accumulator rows are declared to be
// columns 16mb + 2gid and 16mb + 2gid + 1.  q is converted to f16 (|q| must stay below 65504).
#pragma once

#include <cuda.h>
#include <math_constants.h>

#include "common.cuh"
#include "decode_attn.cuh"

namespace dynts {

constexpr int kStRows = 32;                      // rows per chunk = per ring stage
constexpr int kStStages = 6;                     // even: chunk i of a CTA goes to stage i % 6 and to the warp pair i % 2,
constexpr int kStStages8 = 12;                   // 8-bit slabs: stages of half the bytes, twice as many (the same bytes in flight)
                                                 // so every stage is always consumed by the same two warps
constexpr int kStConsumerWarps = 4;
constexpr int kStConsumers = kStConsumerWarps * 32;
constexpr int kStThreads = kStConsumers + 64;    // + one producer warp + one scorer warp
constexpr int kStBoxBytes = kStRows * 128;       // one TMA box: 32 rows x 64 bf16
constexpr int kStStageBytes = 4 * kStBoxBytes;   // K low/high half of head_dim, V low/high
constexpr int kStCombFloats = kStConsumerWarps * 4 * 128;
constexpr int kStMaxCtas = 320;                  // partial slots exist for this many CTAs
constexpr int kStPartStride = 8 * 128 + 16;      // floats per partial: O[8][128], m[8], l[8]
constexpr int kStMaxBatch = 512;                 // sequences whose chunk prefix fits shared memory
constexpr uint32_t kStSpinLimit = 1u << 22;      // bounded mbarrier polling: the default limit (DecodeParams::spin_limit)
constexpr int kStPendWords = 20;                 // a recorded score pass: n, n_old, M[8], 1/L[8], 2 spare

__host__ __device__ inline size_t stream_smem_bytes(int Nb) {
  return 1024 /* alignment slack */ + (size_t)kStStages * kStStageBytes + sizeof(float) * kStCombFloats +
         sizeof(float) * (2 * kStConsumerWarps * 8 + kStConsumerWarps * 8 + 4 * 8) + 16 * kStStages8 + 128 + 256 +
         sizeof(int) * (4 * (size_t)Nb + 2);
}

// ---- PTX wrappers ---------------------------------------------------------------------------
__device__ __forceinline__ uint32_t smem_u32(const void* p) { return (uint32_t)__cvta_generic_to_shared(p); }

__device__ __forceinline__ void mbar_init(uint32_t bar, uint32_t count) {
  asm volatile("mbarrier.init.shared::cta.b64 [%0], %1;" ::"r"(bar), "r"(count) : "memory");
}
__device__ __forceinline__ void mbar_arrive_expect_tx(uint32_t bar, uint32_t bytes) {
  asm volatile("mbarrier.arrive.expect_tx.shared::cta.b64 _, [%0], %1;" ::"r"(bar), "r"(bytes) : "memory");
}
__device__ __forceinline__ void mbar_arrive(uint32_t bar) {
  asm volatile("mbarrier.arrive.shared::cta.b64 _, [%0];" ::"r"(bar) : "memory");
}
__device__ __forceinline__ bool mbar_try_wait(uint32_t bar, uint32_t parity) {
  uint32_t ok;
  asm volatile(
      "{\n\t.reg .pred p;\n\tmbarrier.try_wait.parity.shared::cta.b64 p, [%1], %2;\n\tselp.u32 %0, 1, 0, p;\n\t}"
      : "=r"(ok)
      : "r"(bar), "r"(parity)
      : "memory");
  return ok != 0;
}
// Non-blocking test of a phase: the answer takes a few hundred cycles to come back, so it is asked
// one unit of work ahead and only read when that work is done.
__device__ __forceinline__ bool mbar_test_wait(uint32_t bar, uint32_t parity) {
  uint32_t ok;
  asm volatile(
      "{\n\t.reg .pred p;\n\tmbarrier.test_wait.parity.shared::cta.b64 p, [%1], %2;\n\tselp.u32 %0, 1, 0, p;\n\t}"
      : "=r"(ok)
      : "r"(bar), "r"(parity)
      : "memory");
  return ok != 0;
}
// Polls with an iteration limit.  On expiry the status word gets the timeout bit and the CTA-wide
// abort flag is raised; every later wait of the CTA then returns at once, so the kernel ends (its
// results are void, which the status word says).
__device__ __forceinline__ void mbar_wait(uint32_t bar, uint32_t parity, volatile int* abort_flag, int* err, uint32_t limit) {
  if (*abort_flag) return;
  for (uint32_t i = 0; i < limit; ++i) {
    if (mbar_try_wait(bar, parity)) return;
    if ((i & 1023u) == 1023u && *abort_flag) return;
  }
  *abort_flag = 1;
  atomicOr(err, kErrTimeout);
}
// K and V rows are read once per step: their L2 lines are marked evict-first so that the stream
// does not push the scores and the logit scratch (which are re-read soon) out of L2.
__device__ __forceinline__ uint64_t l2_evict_first_policy() {
  uint64_t pol;
  asm volatile("createpolicy.fractional.L2::evict_first.b64 %0, 1.0;" : "=l"(pol));
  return pol;
}
__device__ __forceinline__ void tma_load_2d(uint32_t dst, const CUtensorMap* map, int x, int y, uint32_t bar,
                                            uint64_t policy) {
  asm volatile(
      "cp.async.bulk.tensor.2d.shared::cluster.global.tile.mbarrier::complete_tx::bytes.L2::cache_hint"
      " [%0], [%1, {%2, %3}], [%4], %5;" ::"r"(dst),
      "l"(reinterpret_cast<uint64_t>(map)), "r"(x), "r"(y), "r"(bar), "l"(policy)
      : "memory");
}
__device__ __forceinline__ void tma_load_3d(uint32_t dst, const CUtensorMap* map, int x, int y, int z, uint32_t bar,
                                            uint64_t policy) {
  asm volatile(
      "cp.async.bulk.tensor.3d.shared::cluster.global.tile.mbarrier::complete_tx::bytes.L2::cache_hint"
      " [%0], [%1, {%2, %3, %4}], [%5], %6;" ::"r"(dst),
      "l"(reinterpret_cast<uint64_t>(map)), "r"(x), "r"(y), "r"(z), "r"(bar), "l"(policy)
      : "memory");
}
__device__ __forceinline__ void ldmatrix_x4(uint32_t addr, uint32_t& r0, uint32_t& r1, uint32_t& r2, uint32_t& r3) {
  asm volatile("ldmatrix.sync.aligned.m8n8.x4.shared.b16 {%0,%1,%2,%3}, [%4];"
               : "=r"(r0), "=r"(r1), "=r"(r2), "=r"(r3)
               : "r"(addr));
}
__device__ __forceinline__ void ldmatrix_x4_trans(uint32_t addr, uint32_t& r0, uint32_t& r1, uint32_t& r2,
                                                  uint32_t& r3) {
  asm volatile("ldmatrix.sync.aligned.m8n8.x4.trans.shared.b16 {%0,%1,%2,%3}, [%4];"
               : "=r"(r0), "=r"(r1), "=r"(r2), "=r"(r3)
               : "r"(addr));
}
__device__ __forceinline__ void mma_f16_m16n8k16(float (&c)[4], uint32_t a0, uint32_t a1, uint32_t a2, uint32_t a3,
                                                 uint32_t b0, uint32_t b1) {
  asm volatile(
      "mma.sync.aligned.m16n8k16.row.col.f32.f16.f16.f32 {%0,%1,%2,%3}, {%4,%5,%6,%7}, {%8,%9}, {%0,%1,%2,%3};"
      : "+f"(c[0]), "+f"(c[1]), "+f"(c[2]), "+f"(c[3])
      : "r"(a0), "r"(a1), "r"(a2), "r"(a3), "r"(b0), "r"(b1));
}
// Four E4M3 codes in a register -> f16 pairs of bytes (0, 1) and (2, 3).
__device__ __forceinline__ void e4m3x4_to_half2x2(uint32_t r, uint32_t& lo, uint32_t& hi) {
  asm("{\n\t.reg .b16 l, h;\n\tmov.b32 {l, h}, %2;\n\tcvt.rn.f16x2.e4m3x2 %0, l;\n\tcvt.rn.f16x2.e4m3x2 %1, h;\n\t}"
      : "=r"(lo), "=r"(hi)
      : "r"(r));
}
// Transposes the 8x8 matrix of 16-bit elements a warp holds as one register per thread (row gid,
// columns 2tig, 2tig+1): afterwards the thread holds elements [2tig][gid] and [2tig+1][gid].
__device__ __forceinline__ uint32_t movmatrix_trans(uint32_t a) {
  uint32_t d_;
  asm volatile("movmatrix.sync.aligned.m8n8.trans.b16 %0, %1;" : "=r"(d_) : "r"(a));
  return d_;
}
__device__ __forceinline__ uint32_t pack_half2(float lo, float hi) {
  __half2 v = __floats2half2_rn(lo, hi);
  return *reinterpret_cast<uint32_t*>(&v);
}
// Two bf16 in a word -> the same two values as f16.
__device__ __forceinline__ uint32_t bf16x2_to_half2(uint32_t w) {
  return pack_half2(__uint_as_float(w << 16), __uint_as_float(w & 0xffff0000u));
}
__device__ __forceinline__ void consumer_sync() { asm volatile("bar.sync 1, %0;" ::"n"(kStConsumers) : "memory"); }

// ---- the chunk list ---------------------------------------------------------------------------
// Chunk index g (within the launch) -> layer-major, then sequence, KV head, chunk of the slab.
// s_cnt[b] = chunks of one slab of sequence b (0 if inactive); s_off[b] = Hkv * sum of s_cnt
// below b; s_off[Nb] = chunks per layer.
struct StCursor {
  int lrel, b, h, chunk, cb;
};

__device__ __forceinline__ void cursor_seek(StCursor& c, long long g, const int* s_off, const int* s_cnt, int Nb) {
  const int per_layer = s_off[Nb];
  int r;
  if (g <= 0x7fffffffLL) {  // (64-bit division costs a lone thread several hundred cycles)
    const unsigned g32 = (unsigned)g, pl = (unsigned)per_layer;
    c.lrel = (int)(g32 / pl);
    r = (int)(g32 - (unsigned)c.lrel * pl);
  } else {
    c.lrel = (int)(g / per_layer);
    r = (int)(g % per_layer);
  }
  int lo = 0, hi = Nb;  // largest b with s_off[b] <= r and s_cnt[b] > 0
  while (hi - lo > 1) {
    const int mid = (lo + hi) >> 1;
    if (s_off[mid] <= r) lo = mid; else hi = mid;
  }
  c.b = lo;
  c.cb = s_cnt[lo];
  r -= s_off[lo];
  c.h = r / c.cb;
  c.chunk = r % c.cb;
}

// Moves to chunk 0 of the next slab in list order.
__device__ __forceinline__ void cursor_next_slab(StCursor& c, const int* s_cnt, int Nb, int Hkv) {
  c.chunk = 0;
  if (++c.h < Hkv) return;
  c.h = 0;
  do {
    if (++c.b == Nb) {
      c.b = 0;
      ++c.lrel;
    }
  } while (s_cnt[c.b] == 0);
  c.cb = s_cnt[c.b];
}


// a5 for one slab: score[j] += sum over the group's heads of exp2(logit[g][j] - M[g]) / L[g], the
// appended row n_old starting from zero.  GG is the group size at compile time so that every load
// of a pass is issued before the first use (one memory round trip per pass).
template <int GG, int VB>
__device__ __forceinline__ void score_pass_vec(bool accumulate, float* __restrict__ score, float* __restrict__ comp, float* __restrict__ dout,
                                               const float* __restrict__ lg, int cap, int n, int n_old,
                                               const float* s_finM, const float* s_finf, int tid, int nthr) {
  float M[GG], f[GG];
#pragma unroll
  for (int g = 0; g < GG; ++g) {
    M[g] = s_finM[g];
    f[g] = s_finf[g];
  }
  const bool drop_lines = (cap & 31) == 0;  // then every head's row range starts on a 128-byte line
  for (int v0 = tid; 4 * v0 < n; v0 += VB * nthr) {
    float4 sc[VB], cc[VB], e[VB][GG];
#pragma unroll
    for (int i = 0; i < VB; ++i) {
      const int j = min(4 * (v0 + i * nthr), cap - 4);  // clamped: always a valid address
      sc[i] = *reinterpret_cast<const float4*>(score + j);
      cc[i] = *reinterpret_cast<const float4*>(comp + j);
#pragma unroll
      for (int g = 0; g < GG; ++g) e[i][g] = __ldcg(reinterpret_cast<const float4*>(lg + (size_t)g * cap + j));
    }
#pragma unroll
    for (int i = 0; i < VB; ++i) {
      const int j = 4 * (v0 + i * nthr);
      if (j >= n) continue;
      float4 dl = make_float4(0.f, 0.f, 0.f, 0.f);
#pragma unroll
      for (int g = 0; g < GG; ++g) {
        dl.x += fast_exp2(e[i][g].x - M[g]) * f[g];
        dl.y += fast_exp2(e[i][g].y - M[g]) * f[g];
        dl.z += fast_exp2(e[i][g].z - M[g]) * f[g];
        dl.w += fast_exp2(e[i][g].w - M[g]) * f[g];
      }
      // The logits of these rows are dead now: drop their L2 lines instead of letting them be
      // written back to DRAM (each 128-byte line was read by eight lanes of this warp in one load).
      if (drop_lines && (tid & 7) == 0) {
#pragma unroll
        for (int g = 0; g < GG; ++g)
          asm volatile("discard.global.L2 [%0], 128;" ::"l"(lg + (size_t)g * cap + j) : "memory");
      }
      const int z = n_old - j;  // the appended row starts from zero
      if (z == 0) sc[i].x = cc[i].x = 0.f;
      if (z == 1) sc[i].y = cc[i].y = 0.f;
      if (z == 2) sc[i].z = cc[i].z = 0.f;
      if (z == 3) sc[i].w = cc[i].w = 0.f;
      kahan_add(sc[i].x, cc[i].x, dl.x);
      kahan_add(sc[i].y, cc[i].y, dl.y);
      kahan_add(sc[i].z, cc[i].z, dl.z);
      kahan_add(sc[i].w, cc[i].w, dl.w);
      if (j + 4 <= n) {
        if (accumulate) {
          *reinterpret_cast<float4*>(score + j) = sc[i];
          *reinterpret_cast<float4*>(comp + j) = cc[i];
        }
        if (dout) *reinterpret_cast<float4*>(dout + j) = dl;
      } else {  // rows past the end are left alone
        if (accumulate) {
          score[j] = sc[i].x;
          comp[j] = cc[i].x;
          if (j + 1 < n) score[j + 1] = sc[i].y, comp[j + 1] = cc[i].y;
          if (j + 2 < n) score[j + 2] = sc[i].z, comp[j + 2] = cc[i].z;
        }
        if (dout) {
          dout[j] = dl.x;
          if (j + 1 < n) dout[j + 1] = dl.y;
          if (j + 2 < n) dout[j + 2] = dl.z;
        }
      }
    }
  }
}

template <int GG>
__device__ __forceinline__ void score_pass(bool accumulate, float* score, float* comp, float* dout, const float* lg, int cap,
                                           int n, int n_old, const float* s_finM, const float* s_finf, int tid, int nthr) {
  if ((cap & 3) == 0 && cap >= 4) {
    score_pass_vec<GG, (GG <= 4 ? 5 : 2)>(accumulate, score, comp, dout, lg, cap, n, n_old, s_finM, s_finf, tid, nthr);
  } else {
    for (int j = tid; j < n; j += nthr) {
      float dl = 0.f;
#pragma unroll
      for (int g = 0; g < GG; ++g) dl += fast_exp2(__ldcg(lg + (size_t)g * cap + j) - s_finM[g]) * s_finf[g];
      if (accumulate) {
        float sj = j == n_old ? 0.f : score[j], cj = j == n_old ? 0.f : comp[j];
        kahan_add(sj, cj, dl);
        score[j] = sj;
        comp[j] = cj;
      }
      if (dout) dout[j] = dl;
    }
  }
}

// The slab's last arriver combines the partials of the k CTAs p_first..p_first+k-1 that worked on
// it; thread tid produces output column tid of every head.  The partials are taken four at a time:
// all loads of a group are issued before the first use, and a running (max, sum, output) is
// rescaled between groups, so the cost is one memory round trip per four contributors.
template <int GG>
__device__ __forceinline__ void combine_partials(const float* part, int p_first, int k, long long g0, long long per_cta,
                                                 __nv_bfloat16* out, float out_scale, float* s_finM, float* s_finf, int tid) {
  constexpr int d = 128;
  float M[GG], L[GG], acc[GG];
#pragma unroll
  for (int g = 0; g < GG; ++g) {
    M[g] = -CUDART_INF_F;
    L[g] = 0.f;
    acc[g] = 0.f;
  }
  for (int q0 = 0; q0 < k; q0 += 4) {
    const float* pp[4];
#pragma unroll
    for (int qi = 0; qi < 4; ++qi) {
      const int q = p_first + min(q0 + qi, k - 1);  // clamped copies beyond k are loaded and ignored
      const int slot = (g0 <= per_cta * q) ? 0 : 1;  // 0: the slab is the first of CTA q's piece
      pp[qi] = part + ((size_t)q * 2 + slot) * kStPartStride;
    }
    float pm[4][GG], pl[4][GG], po[4][GG];
#pragma unroll
    for (int qi = 0; qi < 4; ++qi) {
#pragma unroll
      for (int g = 0; g < GG; ++g) {
        pm[qi][g] = __ldcg(pp[qi] + 8 * d + g);
        pl[qi][g] = __ldcg(pp[qi] + 8 * d + 8 + g);
        po[qi][g] = __ldcg(pp[qi] + (size_t)g * d + tid);
      }
    }
#pragma unroll
    for (int g = 0; g < GG; ++g) {
      float Mn = M[g];
#pragma unroll
      for (int qi = 0; qi < 4; ++qi)
        if (q0 + qi < k) Mn = fmaxf(Mn, pm[qi][g]);
      const float r = fast_exp2(M[g] - Mn);  // 0 for the first group (M = -inf; every partial max is finite)
      float Ln = L[g] * r, an = acc[g] * r;
#pragma unroll
      for (int qi = 0; qi < 4; ++qi) {
        if (q0 + qi < k) {
          const float w = fast_exp2(pm[qi][g] - Mn);
          Ln += pl[qi][g] * w;
          an += po[qi][g] * w;
        }
      }
      M[g] = Mn;
      L[g] = Ln;
      acc[g] = an;
    }
  }
#pragma unroll
  for (int g = 0; g < GG; ++g) {
    out[(size_t)g * d + tid] = __float2bfloat16_rn(acc[g] / L[g] * out_scale);
    if (tid == 0) {
      s_finM[g] = M[g];
      s_finf[g] = 1.0f / L[g];
    }
  }
}

// The same pass with one group of loads in flight per thread: for callers that must stay small in
// registers (the eviction kernel applies recorded passes with it).
template <int GG>
__device__ __forceinline__ void score_pass_lean(float* score, float* comp, const float* lg, int cap, int n, int n_old,
                                                const float* s_finM, const float* s_finf, int tid, int nthr) {
  if ((cap & 3) == 0 && cap >= 4) {
    score_pass_vec<GG, 1>(true, score, comp, nullptr, lg, cap, n, n_old, s_finM, s_finf, tid, nthr);
  } else {
    for (int j = tid; j < n; j += nthr) {
      float dl = 0.f;
#pragma unroll
      for (int g = 0; g < GG; ++g) dl += fast_exp2(__ldcg(lg + (size_t)g * cap + j) - s_finM[g]) * s_finf[g];
      float sj = j == n_old ? 0.f : score[j], cj = j == n_old ? 0.f : comp[j];
      kahan_add(sj, cj, dl);
      score[j] = sj;
      comp[j] = cj;
    }
  }
}

// A score pass handed from the consumer warps to the scorer warp.
struct StScoreTask {
  long long slab;  // < 0: no more tasks
  int n, n_old;
  float M[8], f[8];
};

#define DYNTS_DISPATCH_GROUP(G, CALL) \
  switch (G) {                        \
    case 1: { constexpr int GG = 1; CALL; } break; \
    case 2: { constexpr int GG = 2; CALL; } break; \
    case 3: { constexpr int GG = 3; CALL; } break; \
    case 4: { constexpr int GG = 4; CALL; } break; \
    case 5: { constexpr int GG = 5; CALL; } break; \
    case 6: { constexpr int GG = 6; CALL; } break; \
    case 7: { constexpr int GG = 7; CALL; } break; \
    default: { constexpr int GG = 8; CALL; } break; \
  }

// DEFER: the instantiation that can record / apply deferred score passes (DecodeParams::defer).  The
// 8-bit instantiation has no register to spare, so it carries that code only in the variant the
// host launches for whole-slab pieces.
template <bool KV8, bool DEFER = !KV8>
__global__ void __launch_bounds__(kStThreads, 2)
decode_attn_stream_kernel(const DecodeParams p, const __grid_constant__ CUtensorMap tmKV) {
  constexpr int d = 128;
  constexpr int kTxBytes = KV8 ? 2 * kStBoxBytes : 4 * kStBoxBytes;  // bytes a stage holds and receives
  constexpr int NS = KV8 ? kStStages8 : kStStages;                    // ring stages (NS * kTxBytes = 96 KB either way)
  // A stage holds the boxes [K, V] (8-bit rows) or [K low half, V low half, K high half, V high half]
  // of head_dim (bf16 rows): one tile load brings the K box and the V box of the same columns.
  constexpr int kHalf = 2 * kStBoxBytes;                               // bf16: offset of the high-half boxes
  // Stages are released to the producer in groups: one wait of the producer thread per group.
  constexpr int kGS = KV8 ? 4 : 2, kNG = NS / kGS;
  const int G = p.G, Nb = p.Nb, Hkv = p.Hkv;
  const int tid = threadIdx.x, warp = tid >> 5, lane = tid & 31;

  extern __shared__ uint8_t st_smem_raw[];
  uint8_t* sm = reinterpret_cast<uint8_t*>((reinterpret_cast<uintptr_t>(st_smem_raw) + 1023) & ~(uintptr_t)1023);
  uint8_t* s_stage = sm;                                             // [stages][4 boxes]
  float* s_comb = reinterpret_cast<float*>(s_stage + NS * kTxBytes);  // [warps][4 heads][128]
  float* s_wm = s_comb + kStCombFloats;                              // [warps][8]
  float* s_wl = s_wm + kStConsumerWarps * 8;
  float* s_sc = s_wl + kStConsumerWarps * 8;                         // [warps][8] rescale of each warp's partial
  float* s_cm = s_sc + kStConsumerWarps * 8;                         // [8] CTA partial max
  float* s_cl = s_cm + 8;                                            // [8] CTA partial sum
  float* s_finM = s_cl + 8;                                          // [8] slab max
  float* s_finf = s_finM + 8;                                        // [8] 1 / slab sum
  uint64_t* s_bar = reinterpret_cast<uint64_t*>(s_finf + 8);         // full[stages], empty[stages]
  int* s_flags = reinterpret_cast<int*>(s_bar + 2 * NS);      // [0] abort, [1] last arriver, [8] uniform chunk count, [10] pass handed off, [16+s] armed phase of stage s
  int* s_cnt = s_flags + 32;                                         // [Nb]
  int* s_off = s_cnt + Nb;                                           // [Nb + 1]
  int* s_len = s_off + Nb + 1;                                       // [Nb] rows per slab before this step, -1: inactive
  int* s_tot = s_len + Nb;                                           // [Nb] tokens seen so far (next position id)
  // hand-off of score passes to the scorer warp: two task slots and their full/empty barriers
  uint64_t* s_tbar = reinterpret_cast<uint64_t*>((reinterpret_cast<uintptr_t>(s_tot + Nb) + 15) & ~(uintptr_t)15);
  StScoreTask* s_task = reinterpret_cast<StScoreTask*>(s_tbar + 5);  // (s_tbar[4]: the recorded passes of this CTA's slabs are done)
  volatile int* s_abort = s_flags;

  const uint32_t bar_full = smem_u32(s_bar), bar_empty = smem_u32(s_bar + NS);
  const uint32_t tbar_full = smem_u32(s_tbar), tbar_empty = smem_u32(s_tbar + 2);

  // ---- per-CTA set-up: barriers and the chunk prefix of the sequences -------------------------
  if (tid == 0) {
    for (int s = 0; s < NS; ++s) {
      mbar_init(bar_full + 8 * s, 1);
      mbar_init(bar_empty + 8 * s, 2 * kGS);  // (used for s < kNG) the two warps that consume each stage of group s
    }
    for (int s = 0; s < 2; ++s) {
      mbar_init(tbar_full + 8 * s, 1);
      mbar_init(tbar_empty + 8 * s, 1);
    }
    mbar_init(smem_u32(s_tbar + 4), 1);
    for (int i = 0; i < 8; ++i) s_flags[i] = 0;  // (s_flags[8] belongs to the prefix warp below)
    for (int i = 16; i < 32; ++i) s_flags[i] = 0;
    asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory");
    asm volatile("fence.proxy.async.shared::cta;" ::: "memory");
  }
  // The launch may overlap the tail of the kernel before it in the stream (programmatic dependent
  // launch): nothing above touches global memory; everything below waits until that kernel has
  // completed and its writes are visible.
  if (tid == 32) {  // the descriptors are kernel parameters: fetching them needs no earlier kernel
    asm volatile("prefetch.tensormap [%0];" ::"l"(reinterpret_cast<uint64_t>(&tmKV)) : "memory");
  }
  asm volatile("griddepcontrol.wait;" ::: "memory");
  if (warp == 1) {
    int carry = 0, cmin = 0x7fffffff, cmax = 0;
    for (int b0 = 0; b0 < Nb; b0 += 32) {
      const int b = b0 + lane;
      int ln = -1, tt = 0;
      if (b < Nb) {
        if (p.n_host > 0) {
          // Constant indices, so that the parameter block is not copied to local memory; the uniform
          // bounds keep the launch from touching more of it than the batch needs (every first touch
          // of a line of the block is a constant-cache miss of a few hundred cycles).
          ln = p.len_host[0];
          tt = p.tot_host[0];
          if (Nb > 1) {
#pragma unroll
            for (int i = 1; i < 8; ++i)
              if (i == b) {
                ln = p.len_host[i];
                tt = p.tot_host[i];
              }
          }
          if (Nb > 8) {
#pragma unroll
            for (int i = 8; i < 32; ++i)
              if (i == b) {
                ln = p.len_host[i];
                tt = p.tot_host[i];
              }
          }
          if (Nb > 32) {
#pragma unroll
            for (int i = 32; i < kHostLens; ++i)
              if (i == b) {
                ln = p.len_host[i];
                tt = p.tot_host[i];
              }
          }
        } else if (p.active[b]) {
          ln = p.len[b];
          tt = p.tot[b];
        }
        s_len[b] = ln;
        s_tot[b] = tt;
      }
      const int c = ln >= 0 ? (ln + 1 + kStRows - 1) / kStRows : 0;
      if (c > 0) {
        cmin = min(cmin, c);
        cmax = max(cmax, c);
      }
      int incl = c;
#pragma unroll
      for (int o = 1; o < 32; o <<= 1) {
        const int v = __shfl_up_sync(0xffffffffu, incl, o);
        if (lane >= o) incl += v;
      }
      if (b < Nb) {
        s_cnt[b] = c;
        s_off[b] = (carry + incl - c) * Hkv;
      }
      carry += __shfl_sync(0xffffffffu, incl, 31);
    }
#pragma unroll
    for (int o = 16; o > 0; o >>= 1) {
      cmin = min(cmin, __shfl_xor_sync(0xffffffffu, cmin, o));
      cmax = max(cmax, __shfl_xor_sync(0xffffffffu, cmax, o));
    }
    if (lane == 0) {
      s_off[Nb] = carry * Hkv;
      s_flags[8] = (cmin == cmax) ? cmax : 0;  // chunks per slab if all slabs are equally long
    }
  }
  __syncthreads();
  if (p.n_host > 0 && p.advance && blockIdx.x == 0 && warp == 0) {
    // nobody in this launch reads the lengths from global memory: publish the advanced values now
    for (int b = lane; b < Nb; b += 32)
      if (s_len[b] >= 0) {
        p.len[b] = s_len[b] + 1;
        p.tot[b] = s_tot[b] + 1;
      }
  }

  const long long per_layer = s_off[Nb];
  const long long total = per_layer * p.n_layers;
  // Piece length: whole slabs per CTA where the host asked for it and the slabs are equally long
  // (no slab is then shared between CTAs), else an equal share of the chunk list.
  const long long per_cta = (p.slabs_per_cta > 0 && s_flags[8] > 0) ? (long long)p.slabs_per_cta * s_flags[8]
                                                                   : (total + gridDim.x - 1) / gridDim.x;
  // (whole-slab pieces only; evaluated where it is used: the consumer loop has no register to spare)
  auto defer_on = [&]() {
    if constexpr (!DEFER) return false;
    else return p.defer != 0 && p.slabs_per_cta > 0 && s_flags[8] > 0;
  };
  const long long g_begin = per_cta * blockIdx.x;
  long long g_end = g_begin + per_cta;
  if (g_end > total) g_end = total;
  const int cnt = g_end > g_begin ? (int)(g_end - g_begin) : 0;

  if (cnt > 0 && warp == kStConsumerWarps) {
    // =========================== producer: one thread feeds the ring ===========================
    // Every barrier operation and tile-load issue costs this one thread a few hundred cycles of
    // latency, and its rate bounds the CTA.  So per chunk it does only: arm the stage's barrier,
    // issue one load (two for bf16 rows) that brings the K and the V box together, bump counters.
    // It waits for free stages once per group of kGS stages, and everything that depends on the
    // slab is recomputed only when the cursor moves to the next slab.
    if (lane == 0) {
      StCursor c;
      cursor_seek(c, g_begin, s_off, s_cnt, Nb);
      const uint64_t pol = l2_evict_first_policy();
      const uint32_t sbase = smem_u32(s_stage);
      int stage = 0, grp = 0, in_grp = 0;
      uint32_t ph = 0;  // parity of the round (it / NS)
      int n_old = s_len[c.b];
      int row = (int)((((size_t)(p.layer0 + c.lrel) * Nb + c.b) * Hkv + c.h) * (size_t)p.cap) + c.chunk * kStRows;
      bool ok = c.lrel < p.n_layers && c.b < Nb && c.h < Hkv && n_old + 1 <= p.cap && c.cb * kStRows <= p.cap + kStRows &&
                (sbase & 1023u) == 0u;
      for (int it = 0; it < cnt; ++it) {
        if (in_grp == 0) {  // the group's stages of the previous round have all been consumed
          mbar_wait(bar_empty + 8 * grp, ph ^ 1u, s_abort, p.err, p.spin_limit);
          if (*s_abort) break;
        }
        if (!ok) {
          // the chunk list and the slab bounds disagree: record, stop feeding, let the waits expire
          atomicOr(p.err, kErrStreamBounds);
          p.dbg[0] = c.lrel; p.dbg[1] = c.b; p.dbg[2] = c.h; p.dbg[3] = c.chunk; p.dbg[4] = n_old; p.dbg[5] = it;
          p.dbg[6] = (int)blockIdx.x; p.dbg[7] = (int)sbase;
          *s_abort = 1;
          break;
        }
        const uint32_t full = bar_full + 8 * stage;
        const uint32_t dst = sbase + (uint32_t)stage * kTxBytes;
        // (p.drop_item >= 0, for tests of the timeout path: CTA 0 neither arms nor loads that item, so
        // the consumers' bounded wait for it runs out)
        if (!(p.drop_item == it && blockIdx.x == 0)) {
          mbar_arrive_expect_tx(full, kTxBytes);
          s_flags[16 + stage] = 1 + (int)ph;  // phase of the loads now in flight, for the drain below
          tma_load_3d(dst, &tmKV, 0, row, 0, full, pol);
          if constexpr (!KV8) tma_load_3d(dst + kHalf, &tmKV, 64, row, 0, full, pol);
        }
        row += kStRows;
        ++stage;
        if (++in_grp == kGS) {
          in_grp = 0;
          if (++grp == kNG) {
            grp = 0;
            stage = 0;
            ph ^= 1u;
          }
        }
        if (++c.chunk == c.cb && it + 1 < cnt) {
          cursor_next_slab(c, s_cnt, Nb, Hkv);
          n_old = s_len[c.b];
          row = (int)((((size_t)(p.layer0 + c.lrel) * Nb + c.b) * Hkv + c.h) * (size_t)p.cap);
          ok = c.lrel < p.n_layers && c.b < Nb && c.h < Hkv && n_old + 1 <= p.cap && c.cb * kStRows <= p.cap + kStRows;
        }
      }
    }
  } else if (cnt > 0 && warp < kStConsumerWarps) {
    // ================================== consumers ============================================
    const int gid = lane >> 2, tig = lane & 3;
    const int pair = warp >> 1, u16 = (warp & 1) * 16;  // pair: parity of the chunks (items) this warp takes
    // ldmatrix lane address inside a box: row of the warp's 16-row unit, 16-byte chunk parity
    const int lrow = u16 + ((lane >> 4) << 3) + (lane & 7);
    const int lchk = (lane >> 3) & 1;
    StCursor c;
    cursor_seek(c, g_begin, s_off, s_cnt, Nb);
    int it = 0;
    int n_posted = 0;  // score passes handed to the scorer warp (thread 0's copy counts)
    // The warp's next item is item + 2; whether its tile has landed is asked while this item is
    // being worked on (a wait costs about 300 cycles even when the tile is long there).
    bool peek_ok = false;  // the tile of this warp's next item was seen to have landed
    int cs = pair;         // ring stage and phase parity of this warp's next item (its items are pair, pair + 2, ...)
    uint32_t cp = 0;
    while (it < cnt) {
      // ---- one segment: chunks [c.chunk, c.chunk + seg) of one slab -----------------------------
      const int seg = min(c.cb - c.chunk, cnt - it);
      const size_t unit = ((size_t)c.lrel * Nb + c.b) * Hkv + c.h;
      const size_t slab = ((size_t)(p.layer0 + c.lrel) * Nb + c.b) * Hkv + c.h;
      const int n_old = s_len[c.b];
      const int n = n_old + 1;
      float* lg = p.logit + slab * (size_t)G * p.cap;  // [G][cap]
      const bool need_pass = p.accumulate || p.delta_out != nullptr;  // else the logits are not needed again
      if (c.lrel >= p.n_layers || c.b >= Nb || c.h >= Hkv || n > p.cap || seg < 1 || c.chunk + seg > c.cb) {
        if (tid == 0) {
          atomicOr(p.err, kErrStreamBounds);
          p.dbg[8] = c.lrel; p.dbg[9] = c.b; p.dbg[10] = c.h; p.dbg[11] = c.chunk; p.dbg[12] = n; p.dbg[13] = it;
          p.dbg[14] = (int)blockIdx.x; p.dbg[15] = seg;
          *s_abort = 1;
        }
        break;  // uniform over the consumer warps
      }

      // Query fragments of the group, straight from global memory (2 KB at most, L2-resident):
      // a0 = Q[head gid][16kk + 2tig, +1], a2 = Q[head gid][16kk + 8 + 2tig, +1].
      // (8-bit slabs: k-step kk covers head_dim 16kk..16kk+15 and this thread's four k-indices are
      // 16kk + 4tig + {0, 1 | 2, 3}, the order in which its register of codes holds them; f16.)
      uint32_t qa[8][2];
      {
        const uint32_t* hq = reinterpret_cast<const uint32_t*>(reinterpret_cast<const __nv_bfloat16*>(p.q) + unit * (size_t)G * d);
#pragma unroll
        for (int kk = 0; kk < 8; ++kk) {
          if constexpr (KV8) {
            const uint2 w = gid < G ? __ldg(reinterpret_cast<const uint2*>(hq + gid * 64 + 8 * kk + 2 * tig)) : make_uint2(0u, 0u);
            qa[kk][0] = bf16x2_to_half2(w.x);
            qa[kk][1] = bf16x2_to_half2(w.y);
          } else {
            qa[kk][0] = gid < G ? __ldg(hq + gid * 64 + 8 * kk + tig) : 0u;
            qa[kk][1] = gid < G ? __ldg(hq + gid * 64 + 8 * kk + 4 + tig) : 0u;
          }
        }
      }

      float o[8][4];
#pragma unroll
      for (int mb = 0; mb < 8; ++mb)
#pragma unroll
        for (int e = 0; e < 4; ++e) o[mb][e] = 0.f;
      // running max and sum of heads 2tig (A) and 2tig+1 (B); the sums cover this thread's tokens only
      float mA_run = -CUDART_INF_F, mB_run = -CUDART_INF_F, lA = 0.f, lB = 0.f;

      for (int k = (pair ^ it) & 1; k < seg; k += 2) {
        const int item = it + k;  // item & 1 == pair
        const int stage = cs;     // == item % NS
        const int row0 = (c.chunk + k) * kStRows;
        if (!peek_ok) mbar_wait(bar_full + 8 * stage, cp, s_abort, p.err, p.spin_limit);
        __syncwarp();
        cs += 2;
        if (cs >= NS) {
          cs -= NS;
          cp ^= 1u;
        }
        if constexpr (KV8) peek_ok = item + 2 < cnt && mbar_test_wait(bar_full + 8 * cs, cp);  // (bf16 rows: HBM-bound, no gain)
        uint8_t* st = s_stage + (size_t)stage * kTxBytes;
        const int t0 = row0 + u16;  // first row of this warp's unit
        if (t0 < n) {
          if (n_old >= t0 && n_old < t0 + 16) {
            // a1: the appended row.  The tile holds whatever the slab had at row n_old; overwrite
            // it in shared memory with k_new / v_new and store the row to the slab.
            const int r = n_old - row0;
            if constexpr (KV8) {
              // lanes 0-15: 16-byte piece ch of the K (lanes 0-7) or V (8-15) row = 16 elements, encoded here
              if (lane < 16) {
                const int ch = lane & 7, isv = lane >> 3;
                const __nv_bfloat16* nrow = reinterpret_cast<const __nv_bfloat16*>(isv ? p.v_new : p.k_new) + unit * d + 16 * ch;
                const uint4 a = __ldg(reinterpret_cast<const uint4*>(nrow)), b = __ldg(reinterpret_cast<const uint4*>(nrow) + 1);
                const float sc = isv ? p.v_scale : p.k_scale;
                const uint32_t w[8] = {a.x, a.y, a.z, a.w, b.x, b.y, b.z, b.w};
                uint32_t o4[4];
#pragma unroll
                for (int i = 0; i < 4; ++i) {
                  const float f0 = __fdiv_rn(__uint_as_float(w[2 * i] << 16), sc);
                  const float f1 = __fdiv_rn(__uint_as_float(w[2 * i] & 0xffff0000u), sc);
                  const float f2 = __fdiv_rn(__uint_as_float(w[2 * i + 1] << 16), sc);
                  const float f3 = __fdiv_rn(__uint_as_float(w[2 * i + 1] & 0xffff0000u), sc);
                  o4[i] = (uint32_t)float2_to_e4m3x2(f0, f1) | ((uint32_t)float2_to_e4m3x2(f2, f3) << 16);
                }
                const uint4 val = make_uint4(o4[0], o4[1], o4[2], o4[3]);
                *reinterpret_cast<uint4*>(st + isv * kStBoxBytes + r * 128 + ((ch ^ (r & 7)) << 4)) = val;
                uint8_t* grow = reinterpret_cast<uint8_t*>(isv ? p.V : p.K) + (slab * (size_t)p.cap + n_old) * d;
                reinterpret_cast<uint4*>(grow)[ch] = val;
              }
            } else {
              const int ch = lane & 15, isv = lane >> 4;
              const __nv_bfloat16* nrow = reinterpret_cast<const __nv_bfloat16*>(isv ? p.v_new : p.k_new) + unit * d;
              const uint4 val = __ldg(reinterpret_cast<const uint4*>(nrow) + ch);
              uint8_t* box = st + (isv + 2 * (ch >> 3)) * kStBoxBytes;
              *reinterpret_cast<uint4*>(box + r * 128 + (((ch & 7) ^ (r & 7)) << 4)) = val;
              __nv_bfloat16* grow = reinterpret_cast<__nv_bfloat16*>(isv ? p.V : p.K) + (slab * (size_t)p.cap + n_old) * d;
              reinterpret_cast<uint4*>(grow)[ch] = val;
            }
            if (lane == 0) {
              p.pos[slab * (size_t)p.cap + n_old] = s_tot[c.b];
              if (!p.accumulate) {  // external scores: the new row starts at 0 until the caller sets it
                p.score[slab * (size_t)p.cap + n_old] = 0.f;
                p.comp[slab * (size_t)p.cap + n_old] = 0.f;
              }
            }
            asm volatile("fence.proxy.async.shared::cta;" ::: "memory");
            __syncwarp();
          }
          // a2: S[token][head] = K Q^T: the unit's 16 tokens on M, the group's heads on N, one mma per
          // 16 head_dim indices (two accumulators, summed, so that the chain of dependent mma is half as long)
          // (all fragment loads of a phase are issued before its mma chain, so their shared-memory
          // latency overlaps; the V fragments are fetched before the softmax arithmetic)
          float s0[4] = {0.f, 0.f, 0.f, 0.f}, s1[4] = {0.f, 0.f, 0.f, 0.f};
          const uint32_t kbase = smem_u32(st) + lrow * 128;
          const uint32_t vbase = kbase + kStBoxBytes;
          uint32_t fr[8][4];
          if constexpr (KV8) {
            // matrices of one ldmatrix: tokens 0-7 x piece 2j, tokens 0-7 x piece 2j+1, tokens 8-15 x the same
            uint32_t kr[4][4];
#pragma unroll
            for (int j = 0; j < 4; ++j)
              ldmatrix_x4(kbase + (((2 * j + lchk) ^ (lrow & 7)) << 4), kr[j][0], kr[j][1], kr[j][2], kr[j][3]);
#pragma unroll
            for (int j = 0; j < 4; ++j) {
              uint32_t a0, a1, a2, a3;  // piece 2j = k-step 2j: (tokens 0-7 | 8-15) x (codes 0, 1 | 2, 3 of the register)
              e4m3x4_to_half2x2(kr[j][0], a0, a2);
              e4m3x4_to_half2x2(kr[j][2], a1, a3);
              mma_f16_m16n8k16(s0, a0, a1, a2, a3, qa[2 * j][0], qa[2 * j][1]);
              e4m3x4_to_half2x2(kr[j][1], a0, a2);
              e4m3x4_to_half2x2(kr[j][3], a1, a3);
              mma_f16_m16n8k16(s1, a0, a1, a2, a3, qa[2 * j + 1][0], qa[2 * j + 1][1]);
            }
            // V: the transposed load gives (token 2tig, columns 2gid, 2gid+1 | token 2tig+1, the same
            // columns); the codes stay packed (16 registers instead of 32) until the second product.
#pragma unroll
            for (int j = 0; j < 4; ++j)  // fr[j][0..3]: tokens 0-7 x pieces 2j, 2j+1; tokens 8-15 x pieces 2j, 2j+1
              ldmatrix_x4_trans(vbase + (((2 * j + lchk) ^ (lrow & 7)) << 4), fr[j][0], fr[j][1], fr[j][2], fr[j][3]);
          } else {
            // registers of one ldmatrix: tokens 0-7 x k 0-7, tokens 0-7 x k 8-15, tokens 8-15 x the same
#pragma unroll
            for (int kk = 0; kk < 8; ++kk) {
              const int chk = ((2 * kk) & 7) + lchk;
              ldmatrix_x4(kbase + (kk >> 2) * kHalf + ((chk ^ (lrow & 7)) << 4), fr[kk][0], fr[kk][1], fr[kk][2], fr[kk][3]);
            }
#pragma unroll
            for (int kk = 0; kk < 8; kk += 2) {
              mma_bf16_m16n8k16(s0, fr[kk][0], fr[kk][2], fr[kk][1], fr[kk][3], qa[kk][0], qa[kk][1]);
              mma_bf16_m16n8k16(s1, fr[kk + 1][0], fr[kk + 1][2], fr[kk + 1][1], fr[kk + 1][3], qa[kk + 1][0], qa[kk + 1][1]);
            }
#pragma unroll
            for (int mb = 0; mb < 8; ++mb) {
              const int chk = ((2 * mb) & 7) + lchk;
              ldmatrix_x4_trans(vbase + (mb >> 2) * kHalf + ((chk ^ (lrow & 7)) << 4), fr[mb][0], fr[mb][1], fr[mb][2], fr[mb][3]);
            }
          }
          // a3: online softmax.  This thread holds tokens gid and gid+8 of heads 2tig and 2tig+1.
          const int tkA = t0 + gid, tkB = tkA + 8;
          const bool hA = 2 * tig < G, hB = 2 * tig + 1 < G;
          float x[4];
          x[0] = (hA && tkA < n) ? (s0[0] + s1[0]) * p.scale_log2 : -CUDART_INF_F;
          x[1] = (hB && tkA < n) ? (s0[1] + s1[1]) * p.scale_log2 : -CUDART_INF_F;
          x[2] = (hA && tkB < n) ? (s0[2] + s1[2]) * p.scale_log2 : -CUDART_INF_F;
          x[3] = (hB && tkB < n) ? (s0[3] + s1[3]) * p.scale_log2 : -CUDART_INF_F;
          if (need_pass) {
            float* ta = lg + (size_t)(2 * tig) * p.cap;  // a warp's store covers 8 consecutive rows of 4 heads
            float* tb = ta + p.cap;
            if (hA && tkA < n) ta[tkA] = x[0];
            if (hB && tkA < n) tb[tkA] = x[1];
            if (hA && tkB < n) ta[tkB] = x[2];
            if (hB && tkB < n) tb[tkB] = x[3];
          }
          float umA = fmaxf(x[0], x[2]), umB = fmaxf(x[1], x[3]);
#pragma unroll
          for (int o_ = 4; o_ < 32; o_ <<= 1) {  // over the unit's tokens: lanes of equal tig
            umA = fmaxf(umA, __shfl_xor_sync(0xffffffffu, umA, o_));
            umB = fmaxf(umB, __shfl_xor_sync(0xffffffffu, umB, o_));
          }
          const float mA_new = fmaxf(mA_run, umA), mB_new = fmaxf(mB_run, umB);
          const float mA_safe = (mA_new == -CUDART_INF_F) ? 0.f : mA_new;
          const float mB_safe = (mB_new == -CUDART_INF_F) ? 0.f : mB_new;
          const float c_even = fast_exp2(mA_run - mA_safe), c_odd = fast_exp2(mB_run - mB_safe);
          const float p0 = fast_exp2(x[0] - mA_safe), p1 = fast_exp2(x[1] - mB_safe);
          const float p2 = fast_exp2(x[2] - mA_safe), p3 = fast_exp2(x[3] - mB_safe);
          lA = lA * c_even + (p0 + p2);
          lB = lB * c_odd + (p1 + p3);
          mA_run = mA_new;
          mB_run = mB_new;
          // P[token][head] -> the B fragment of P V (tokens 2tig, 2tig+1 | +8 of head gid): an 8x8 transpose per half
          const uint32_t pb0 = movmatrix_trans(KV8 ? pack_half2(p0, p1) : pack_bf16x2(p0, p1));
          const uint32_t pb1 = movmatrix_trans(KV8 ? pack_half2(p2, p3) : pack_bf16x2(p2, p3));
          // a4: O^T[d][head] += V^T P; accumulator mb covers d = 16mb + gid (+8), heads 2tig, 2tig+1
          // (8-bit slabs: d = 16mb + 2gid (+1); operand order a0..a3 = rows gid | gid+8, tokens 0-7 | 8-15)
          // (once the running maxima have settled, which is after the first few units of a slab, the
          // rescale factors are exactly 1 and the 32 multiplications are skipped)
          if (!__all_sync(0xffffffffu, (c_even == 1.0f || !hA) && (c_odd == 1.0f || !hB))) {  // (padding heads hold zeros)
#pragma unroll
            for (int mb = 0; mb < 8; ++mb) {
              o[mb][0] *= c_even;
              o[mb][1] *= c_odd;
              o[mb][2] *= c_even;
              o[mb][3] *= c_odd;
            }
          }
#pragma unroll
          for (int mb = 0; mb < 8; ++mb) {
            if constexpr (KV8) {
              // -> (token, token+1) pairs of column 2gid (low half) and 2gid+1 (high half)
              uint32_t a0, a1, a2, a3;
              e4m3x4_to_half2x2(__byte_perm(fr[mb >> 1][mb & 1], 0u, 0x3120), a0, a1);
              e4m3x4_to_half2x2(__byte_perm(fr[mb >> 1][2 + (mb & 1)], 0u, 0x3120), a2, a3);
              mma_f16_m16n8k16(o[mb], a0, a1, a2, a3, pb0, pb1);
            } else {
              mma_bf16_m16n8k16(o[mb], fr[mb][0], fr[mb][1], fr[mb][2], fr[mb][3], pb0, pb1);
            }
          }
        }
        __syncwarp();
        if (lane == 0) mbar_arrive(bar_empty + 8 * (stage / kGS));
      }

      // ---- segment end: warp partials -> CTA partial ---------------------------------------------
#pragma unroll
      for (int o_ = 4; o_ < 32; o_ <<= 1) {  // sums over the tokens held by the lanes of equal tig
        lA += __shfl_xor_sync(0xffffffffu, lA, o_);
        lB += __shfl_xor_sync(0xffffffffu, lB, o_);
      }
      if (gid == 0) {
        s_wm[warp * 8 + 2 * tig] = mA_run;
        s_wm[warp * 8 + 2 * tig + 1] = mB_run;
        s_wl[warp * 8 + 2 * tig] = lA;
        s_wl[warp * 8 + 2 * tig + 1] = lB;
      }
      // Who else works on this slab?  Chunk g0 is its first one.
      const long long g0 = g_begin + it - c.chunk;
      int p_first, p_last;
      if (total <= 0x7fffffffLL) {  // 32-bit division: this sits between a slab's last tile and its output
        const unsigned pc = (unsigned)per_cta;
        p_first = (int)((unsigned)g0 / pc);
        p_last = (int)(((unsigned)g0 + (unsigned)c.cb - 1u) / pc);
      } else {
        p_first = (int)(g0 / per_cta);
        p_last = (int)((g0 + c.cb - 1) / per_cta);
      }
      const bool exclusive = p_first == p_last;
      if (p_first < 0 || p_last >= (int)gridDim.x || (int)blockIdx.x < p_first || (int)blockIdx.x > p_last) {
        if (tid == 0) {
          atomicOr(p.err, kErrStreamBounds);
          p.dbg[16] = p_first; p.dbg[17] = p_last; p.dbg[18] = (int)blockIdx.x; p.dbg[19] = (int)g0;
          *s_abort = 1;
        }
        break;
      }
      const int my_slot = (g0 <= g_begin) ? 0 : 1;  // 0: the slab is the first of this CTA's piece
      float* my_part = p.part + ((size_t)blockIdx.x * 2 + my_slot) * kStPartStride;
      __nv_bfloat16* out = reinterpret_cast<__nv_bfloat16*>(p.out) + unit * (size_t)G * d;
      float* score = p.score + slab * (size_t)p.cap;
      // Thread tid owns output column tid of the four heads of a round.
      for (int rd = 0; rd * 4 < G; ++rd) {
        if (rd > 0) consumer_sync();  // the previous round's sums have been read
        if ((tig >> 1) == rd) {
          float* c0 = s_comb + ((size_t)warp * 4 + 2 * (tig & 1)) * d;
#pragma unroll
          for (int mb = 0; mb < 8; ++mb) {
            const int ca = KV8 ? 16 * mb + 2 * gid : 16 * mb + gid;      // column of accumulator rows gid
            const int cb2 = KV8 ? ca + 1 : ca + 8;                       // and gid + 8
            c0[ca] = o[mb][0];
            c0[d + ca] = o[mb][1];
            c0[cb2] = o[mb][2];
            c0[d + cb2] = o[mb][3];
          }
        }
        consumer_sync();  // also orders s_wm / s_wl
#pragma unroll
        for (int i = 0; i < 4; ++i) {
          const int g = 4 * rd + i;
          if (g < G) {
            float mc = -CUDART_INF_F;
#pragma unroll
            for (int w = 0; w < kStConsumerWarps; ++w) mc = fmaxf(mc, s_wm[w * 8 + g]);
            const float ms = (mc == -CUDART_INF_F) ? 0.f : mc;
            float acc = 0.f, l = 0.f;
#pragma unroll
            for (int w = 0; w < kStConsumerWarps; ++w) {
              const float f = fast_exp2(s_wm[w * 8 + g] - ms);
              acc += s_comb[((size_t)w * 4 + i) * d + tid] * f;
              l += s_wl[w * 8 + g] * f;
            }
            if (exclusive) {
              out[(size_t)g * d + tid] = __float2bfloat16_rn(acc / l * p.out_scale);
              if (tid == 0) {
                s_finM[g] = mc;
                s_finf[g] = 1.0f / l;
              }
            } else {
              my_part[(size_t)g * d + tid] = acc;
              if (tid == 0) {
                my_part[8 * d + g] = mc;
                my_part[8 * d + 8 + g] = l;
              }
            }
          }
        }
      }

      bool finish = exclusive;
      if (!exclusive) {
        __threadfence();  // partial and logits before the ticket
        consumer_sync();
        if (tid == 0) {
          const int k = p_last - p_first + 1;
          const int t = atomicAdd(p.arrive + slab, 1);
          const int last = t == k - 1;
          if (last) {
            p.arrive[slab] = 0;
            __threadfence();
          }
          s_flags[1] = last;
        }
        consumer_sync();
        finish = s_flags[1] != 0;
        if (finish) {
          // Last arriver: combine the partials of CTAs p_first..p_last; thread tid does column tid.
          const int k = p_last - p_first + 1;
          DYNTS_DISPATCH_GROUP(G, combine_partials<GG>(p.part, p_first, k, g0, per_cta, out, p.out_scale, s_finM, s_finf, tid));
        }
      }
      if (finish && need_pass) {
        // a5: final weights of every row of the slab, summed over the group's heads (Eq. 6)
        consumer_sync();  // s_finM / s_finf, and this CTA's own logits
        bool handed = false;
        if (it + seg < cnt) {
          // More chunks follow: leave the pass to the scorer warp (if it has a free task slot) and
          // go on streaming.  After the last chunk the four consumer warps do the pass themselves.
          if (tid == 0) {
            const int slot = n_posted & 1;
            int ok = 0;
            if (mbar_try_wait(tbar_empty + 8 * slot, (((uint32_t)n_posted >> 1) & 1u) ^ 1u)) {
              StScoreTask& tk = s_task[slot];
              tk.slab = (long long)slab;
              tk.n = n;
              tk.n_old = n_old;
#pragma unroll
              for (int g = 0; g < 8; ++g) {
                tk.M[g] = s_finM[g];
                tk.f[g] = s_finf[g];
              }
              mbar_arrive(tbar_full + 8 * slot);  // release: the task and, through the barrier above, the logits
              ++n_posted;
              ok = 1;
            }
            s_flags[10] = ok;
          }
          consumer_sync();
          handed = s_flags[10] != 0;
        }
        if (!handed && it + seg >= cnt && defer_on()) {
          // the CTA's last slab: nothing is left to overlap the pass with; record it for the next launch
          // (once the scorer warp is done with the record the previous launch left in the same place)
          mbar_wait(smem_u32(s_tbar + 4), 0u, s_abort, p.err, p.spin_limit);
          int* rec = p.pend + slab * kStPendWords;
          if (tid < 8) {
            reinterpret_cast<float*>(rec)[2 + tid] = s_finM[tid];
            reinterpret_cast<float*>(rec)[10 + tid] = s_finf[tid];
          } else if (tid == 8) {
            rec[1] = n_old;
            rec[0] = n;
          }
        } else if (!handed) {
          // (the recorded pass of this slab, if any, must have been applied first)
          if (defer_on()) mbar_wait(smem_u32(s_tbar + 4), 0u, s_abort, p.err, p.spin_limit);
          float* dout = p.delta_out ? p.delta_out + slab * (size_t)p.cap : nullptr;
          DYNTS_DISPATCH_GROUP(G, score_pass<GG>(p.accumulate != 0, score, p.comp + slab * (size_t)p.cap, dout, lg, p.cap, n,
                                                 n_old, s_finM, s_finf, tid, kStConsumers));
        }
      }
      consumer_sync();  // shared scratch is reused by the next segment
      it += seg;
      if (it < cnt) cursor_next_slab(c, s_cnt, Nb, Hkv);
    }
    if (tid == 0 && it >= cnt) {  // tell the scorer warp that nothing more will come
      const int slot = n_posted & 1;
      if (n_posted >= 2) mbar_wait(tbar_empty + 8 * slot, (((uint32_t)n_posted >> 1) & 1u) ^ 1u, s_abort, p.err, p.spin_limit);  // (else never used)
      s_task[slot].slab = -1;
      mbar_arrive(tbar_full + 8 * slot);
    }
  } else if (cnt > 0) {
    // ================= scorer: score passes of finished slabs, beside the streaming =================
    if (defer_on()) {
      // first the passes the previous launch recorded for this CTA's slabs (their logits are in the
      // other half of the scratch)
      StCursor c2;
      cursor_seek(c2, g_begin, s_off, s_cnt, Nb);
      const int n_sl = cnt / s_flags[8];
      for (int i = 0; i < n_sl; ++i) {
        const size_t slab = ((size_t)(p.layer0 + c2.lrel) * Nb + c2.b) * Hkv + c2.h;
        if (c2.lrel >= p.n_layers || c2.b >= Nb || c2.h >= Hkv) break;
        int* rec = p.pend + slab * kStPendWords;
        const int rn = rec[0];
        if (rn > 0 && rn <= p.cap) {
          const int rn_old = rec[1];
          const float* rM = reinterpret_cast<const float*>(rec) + 2;
          DYNTS_DISPATCH_GROUP(G, score_pass<GG>(true, p.score + slab * (size_t)p.cap, p.comp + slab * (size_t)p.cap, nullptr,
                                                 p.logit_prev + slab * (size_t)G * p.cap, p.cap, rn, rn_old, rM, rM + 8, lane, 32));
          __syncwarp();
          if (lane == 0) rec[0] = 0;
        }
        if (i + 1 < n_sl) cursor_next_slab(c2, s_cnt, Nb, Hkv);
      }
      __threadfence_block();
    }
    if (lane == 0) mbar_arrive(smem_u32(s_tbar + 4));
    for (int t = 0;; ++t) {
      const int slot = t & 1;
      mbar_wait(tbar_full + 8 * slot, (uint32_t)(t >> 1) & 1u, s_abort, p.err, p.spin_limit);
      __syncwarp();
      if (*s_abort) break;
      const StScoreTask& tk = s_task[slot];
      if (tk.slab < 0) break;
      const size_t slab = (size_t)tk.slab;
      float* dout = p.delta_out ? p.delta_out + slab * (size_t)p.cap : nullptr;
      DYNTS_DISPATCH_GROUP(G, score_pass<GG>(p.accumulate != 0, p.score + slab * (size_t)p.cap, p.comp + slab * (size_t)p.cap, dout,
                                             p.logit + slab * (size_t)G * p.cap, p.cap, tk.n, tk.n_old, tk.M, tk.f, lane, 32));
      __syncwarp();
      if (lane == 0) mbar_arrive(tbar_empty + 8 * slot);
    }
  }

  // Every tile load this CTA issued has been waited for by its consumers unless a wait gave up;
  // then give the loads in flight a bounded time to land before the shared memory is released.
  __syncthreads();
  if (*s_abort && tid == 0) {
    for (int s = 0; s < NS; ++s) {
      const int armed = s_flags[16 + s];
      if (armed == 0) continue;
      for (uint32_t i = 0; i < kStSpinLimit; ++i)  // (the full default limit: these loads were issued and will land)
        if (mbar_try_wait(bar_full + 8 * s, (uint32_t)(armed - 1))) break;
    }
  }
  if (p.n_host == 0) finish_ticket(p);
}

// Applies the score passes recorded by the last streaming launch (see DecodeParams::defer): one
// CTA per slab.  logit = the half of the scratch those launches wrote.
__global__ void __launch_bounds__(128) flush_pending_kernel(float* score, float* comp, const float* logit, int* pend, int G,
                                                            int cap) {
  const size_t slab = blockIdx.x;
  int* rec = pend + slab * kStPendWords;
  asm volatile("griddepcontrol.wait;" ::: "memory");  // (launched with programmatic stream serialisation)
  const int n = rec[0];
  if (n <= 0 || n > cap) return;  // uniform over the CTA
  const int n_old = rec[1];
  __shared__ float sM[8], sf[8];
  if (threadIdx.x < 8) {
    sM[threadIdx.x] = reinterpret_cast<const float*>(rec)[2 + threadIdx.x];
    sf[threadIdx.x] = reinterpret_cast<const float*>(rec)[10 + threadIdx.x];
  }
  __syncthreads();
  DYNTS_DISPATCH_GROUP(G, score_pass<GG>(true, score + slab * (size_t)cap, comp + slab * (size_t)cap, nullptr,
                                         logit + slab * (size_t)G * cap, cap, n, n_old, sM, sf, (int)threadIdx.x, 128));
  __syncthreads();
  if (threadIdx.x == 0) rec[0] = 0;
}

}  // namespace dynts

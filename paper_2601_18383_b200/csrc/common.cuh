// Shared declarations of the sm_100a kernels: parameter blocks, small device helpers.
#pragma once

#include <cuda_runtime.h>
#include <cuda_bf16.h>
#include <cuda_fp16.h>
#include <stdint.h>

namespace dynts {

constexpr int kMaxGroup = 8;        // query heads per KV head handled by the kernels
constexpr int kHostLens = 64;       // batches up to this size get their lengths with the launch
constexpr int kErrTileOverflow = 1; // device status bits
constexpr int kErrLenOverflow = 2;
constexpr int kErrEvictSmem = 4;
constexpr int kErrTimeout = 8;           // a bounded wait on a shared-memory barrier gave up
constexpr int kErrStreamBounds = 16; // the streaming kernel's chunk list left the slab bounds

// One decode launch covers `n_layers` layers starting at `layer0`.
struct DecodeParams {
  const void* q;      // [n_layers, Nb, Hq, d] of this launch
  const void* k_new;  // [n_layers, Nb, Hkv, d]
  const void* v_new;
  void* out;          // [n_layers, Nb, Hq, d]
  float* delta_out;   // NULL or full [L, Nb, Hkv, cap]
  void* K;            // full [L, Nb, Hkv, cap, d]
  void* V;
  int* pos;           // full [L, Nb, Hkv, cap]
  float* score;       // full [L, Nb, Hkv, cap]
  float* comp;        // full [L, Nb, Hkv, cap]: rounding error of the score sums (compensated summation)
  int* len;           // [Nb] rows per slab of each sequence
  int* tot;           // [Nb] tokens seen so far (next position id)
  const int* active;  // [Nb]
  unsigned int* ticket;
  int* err;           // pinned host status word
  float* logit;       // streaming kernel: scaled logits of the step, [L, Nb, Hkv, G, cap]
  float* part;        // streaming kernel: per-CTA partials, [CTAs][2][O 8x128 | m 8 | l 8]
  int* arrive;        // streaming kernel: per-slab arrival counters, zero between launches
  int* dbg;           // streaming kernel: 32 ints describing the first failed self-check
  int layer0, n_layers, Nb, Hkv, G, d, cap;
  int advance;        // 1: the last CTA to finish increments len/tot of active sequences
  int tile_tokens;    // rows of logits a CTA can hold in shared memory
  int slabs_per_cta;  // streaming kernel: > 0 => every CTA takes this many whole slabs
  int accumulate;     // 1: add each row's attention mass to its score (Eq. 6); 0: scores come from the caller
  float scale_log2;   // log2(e) / sqrt(d); times k_scale when the slabs hold 8-bit rows
  float k_scale, v_scale;  // 8-bit slabs: a row is stored as e4m3(x / scale) and read as code value x scale
  float out_scale;    // factor of the output (v_scale for 8-bit slabs, else 1)
  // Streaming kernel: n_host > 0 => the rows per slab and the tokens seen so far of every sequence
  // come with the launch (the host's mirror; -1 = inactive sequence) instead of being read from
  // len / tot / active, and block 0 writes the advanced values back at once (no ticket at the end).
  int n_host;
  // Streaming kernel, whole-slab pieces: defer = 1 => the score pass of a CTA's last slab is not run
  // at the end of the launch (where nothing overlaps it) but recorded in pend[slab] = {n, n_old,
  // M[8], 1/L[8]} and run by the scorer warp of the next launch, beside its streaming, from the
  // other half of the logit scratch (logit_prev).  The host runs the recorded passes itself
  // (flush_pending_kernel) before anything else touches the scores.
  int defer;
  float* logit_prev;
  int* pend;          // [slabs][20]
  unsigned int spin_limit;  // streaming kernel: polls after which a wait on a shared-memory barrier gives up (kErrTimeout)
  int drop_item;            // streaming kernel, tests of the timeout path: CTA 0 omits the tile load of this item (-1: none)
  int len_host[kHostLens];
  int tot_host[kHostLens];
};

struct EvictParams {
  void* K;
  void* V;
  int* pos;
  float* score;
  float* comp;        // NULL, or the score sums' compensation terms (moved with the scores)
  const float* key;   // NULL, or [Nb, cap] selection keys shared by all slabs of a sequence (fused kernel only)
  int* src;           // [slabs, cap] gather list: src[dst] = surviving row index
  int* hdr;           // [slabs, 4]: {first moved dst, rows kept, old length, unused}
  int* len;           // [Nb]
  const int* pinned;  // [Nb]
  const int* target;  // [Nb]
  int* err;
  int L, Nb, Hkv, d, cap, window, elt_bytes;
  // Fused kernel: score passes the last streaming decode launch left recorded (DecodeParams::defer)
  // are applied by each slab's CTA before it reads the scores.  pend == NULL: nothing recorded.
  int* pend = nullptr;
  const float* logit_prev = nullptr;
  int G = 0;
};

__device__ __forceinline__ float fast_exp2(float x) {
  float y;
  asm("ex2.approx.ftz.f32 %0, %1;" : "=f"(y) : "f"(x));
  return y;
}

__device__ __forceinline__ float to_float(float x) { return x; }
__device__ __forceinline__ float to_float(__nv_bfloat16 x) { return __bfloat162float(x); }
__device__ __forceinline__ void from_float(float* p, float x) { *p = x; }
__device__ __forceinline__ void from_float(__nv_bfloat16* p, float x) { *p = __float2bfloat16_rn(x); }

// 8-bit floats (E4M3: 1 sign, 4 exponent bits with bias 7, 3 mantissa bits, largest finite 448).
// Two codes in a 16-bit word -> two halves (exact); low byte -> low half.
__device__ __forceinline__ uint32_t e4m3x2_to_half2(unsigned short v) {
  uint32_t h;
  asm("cvt.rn.f16x2.e4m3x2 %0, %1;" : "=r"(h) : "h"(v));
  return h;
}
__device__ __forceinline__ float e4m3_to_float(uint8_t v) {
  const uint32_t h = e4m3x2_to_half2((unsigned short)v);
  return __half2float(__ushort_as_half((unsigned short)(h & 0xffffu)));
}
// Codes of lo and hi (round to nearest even, magnitudes beyond 448 saturate): lo in the low byte.
__device__ __forceinline__ unsigned short float2_to_e4m3x2(float lo, float hi) {
  unsigned short r;
  asm("cvt.rn.satfinite.e4m3x2.f32 %0, %1, %2;" : "=h"(r) : "f"(hi), "f"(lo));
  return r;
}
__device__ __forceinline__ uint8_t float_to_e4m3(float x) { return (uint8_t)(float2_to_e4m3x2(x, 0.f) & 0xffu); }
// The code stored for a row element x of a slab with scale s (the division is IEEE fp32).
__device__ __forceinline__ uint8_t store_e4m3(float x, float s) { return float_to_e4m3(__fdiv_rn(x, s)); }

// Streaming 16-byte load that bypasses L1 allocation (each K/V byte is read once per step).
__device__ __forceinline__ uint4 ldg_stream(const void* p) {
  uint4 r;
  asm volatile("ld.global.nc.L1::no_allocate.v4.u32 {%0,%1,%2,%3}, [%4];"
               : "=r"(r.x), "=r"(r.y), "=r"(r.z), "=r"(r.w)
               : "l"(p));
  return r;
}

// Compensated (Kahan) addition of one step's mass x to a score s with running compensation c: the
// rounding error of each fp32 addition is carried into the next one, so a score accumulated over
// thousands of steps stays within about one ulp of the exact sum.  Pinned rows (score +inf) are
// left alone.
__device__ __forceinline__ void kahan_add(float& s, float& c, float x) {
  if (s > 3.0e38f) {  // +inf
    c = 0.f;
    return;
  }
  const float y = __fsub_rn(x, c);
  const float t = __fadd_rn(s, y);
  c = __fsub_rn(__fsub_rn(t, s), y);
  s = t;
}

// The last CTA of the grid to finish advances the per-sequence lengths: every other CTA has
// read them before taking its ticket, so the update cannot race with a read of this launch.
__device__ __forceinline__ void take_ticket(const DecodeParams& p) {  // one thread per CTA
  // (this CTA's reads of the lengths returned their values long ago; no fence is needed to
  // order them before the ticket)
  unsigned int t = atomicAdd(p.ticket, 1u);
  if (t == gridDim.x - 1) {
    *p.ticket = 0u;
    if (p.advance) {
      for (int b = 0; b < p.Nb; ++b) {
        if (p.active[b]) {
          p.len[b] += 1;
          p.tot[b] += 1;
        }
      }
    }
    __threadfence();
  }
}

__device__ __forceinline__ void finish_ticket(const DecodeParams& p) {
  __syncthreads();
  if (threadIdx.x == 0) take_ticket(p);
}

}  // namespace dynts

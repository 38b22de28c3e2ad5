// Prefill attention for sm_100a: every prompt position attends to the positions up to and
// including itself (Eq. 4-5 with t = 1..M), bf16, head_dim 128, grouped query heads.  This is the
// phase that fills the question window (Section 4.2); unlike the decode step it is a dense
// contraction (M x M x d per head), and it runs on the 5th-generation tensor path: tcgen05.mma with
// the accumulators in tensor memory, operands brought into shared memory by TMA tile loads.
//
// One CTA = 128 query rows of one query head.  It walks the key/value rows in tiles of 64 up to the
// diagonal; per tile
//     S  = Q K^T          M 128 x N 64 x K 128   (8 instructions of K = 16; Q and K tiles K-major)
//     P  = exp2(S * scale - rowmax)               (online softmax: running max and sum per row)
//     O += P V            M 128 x N 128 x K 64   (4 instructions; P from tensor memory, V MN-major)
// Seven warps.  Warps 0-3 are the softmax warps: thread r owns query row r, i.e. lane r of tensor
// memory -- it reads its row of S with tcgen05.ld, keeps the row's running max and sum, rescales
// its row of O in tensor memory when the max moves, and writes its row of P (bf16, two per column)
// back into tensor memory over the S tile it came from, where the second product reads it as its
// A operand: P never touches shared memory and the softmax of a tile does not wait for the product
// of the tile before (unless the row's reference maximum has to move).  One thread of
// warp 4 issues the TMA loads (Q once; K and V tiles into two stages each, requested as soon as the
// product that read the stage before has completed), one thread of warp 5 the second product and
// one of warp 6 the first, whose completion reaches the other warps through mbarriers
// (tcgen05.commit).  Each of those threads is a chain of waits and issues of a few hundred cycles
// apiece (a wait on a completed barrier about 300, an MMA about 90), which is why they are three:
// the chain of one never delays the others.  S is double
// buffered in tensor memory (columns 0-63 / 64-127; O in 128-255), so S of tile j + 1 is computed
// while the softmax of tile j runs; S of tile j + 2 overwrites the P of tile j and is issued once
// O += P V of tile j has completed.  96 KB of shared memory
// and 256 columns of tensor memory per CTA: two CTAs share an SM and fill each other's bubbles.
//
// Tiles above the diagonal are never loaded.  Rows and keys beyond the prompt come back from TMA
// as zeros (the tensor maps are [heads][T][128], so a box never reaches into the next head) and
// are masked like the keys above the diagonal.  No load uses cluster multicast.  Every wait is
// bounded: on expiry the CTA raises the timeout bit of the status word, every later wait returns
// at once, the CTA waits (bounded) for what it has in flight, frees its tensor memory and ends.
#pragma once

#include <cuda.h>
#include <math_constants.h>

#include "common.cuh"
#include "decode_stream.cuh"  // mbarrier wrappers, smem_u32
#include "tc5.cuh"

namespace dynts {

constexpr int kPfRows = 128;                      // query rows per CTA
constexpr int kPfKeys = 64;                       // key rows per tile
constexpr int kPfThreads = 224;                   // 4 softmax warps, one warp whose first lane issues the TMA loads, one warp each for O += P V and S = Q K^T
constexpr int kPfQBytes = kPfRows * 256;          // two boxes of 128 rows x 64 bf16
constexpr int kPfKvBytes = kPfKeys * 256;         // two boxes of 64 rows x 64 bf16
// Two CTAs must fit the 227 KB of an SM (each also costs 1 KB of system space), so there is no room
// for alignment slack: the dynamic shared memory is declared 1024-byte aligned (what the 128-byte
// swizzle needs) and the kernel checks that it is.
constexpr int kPfSmemBytes = kPfQBytes + 4 * kPfKvBytes + 128;
constexpr uint32_t kPfTmemCols = 256;             // S0 | S1 | O
constexpr uint32_t kPfSpinLimit = 1u << 21;

struct PrefillAttnParams {
  __nv_bfloat16* out;      // [L, Nb, Hq, T, 128]
  int* err;                // pinned host status word
  int* stop;               // device word: non-zero once a CTA of this cache's prefill launches has given up a wait
  int T, Hq, Hkv;
  float scale_log2;
};

__device__ __forceinline__ void pf_tma_load(uint32_t dst, const CUtensorMap* map, int x, int y, int z, uint32_t bar) {
  asm volatile(
      "cp.async.bulk.tensor.3d.shared::cluster.global.tile.mbarrier::complete_tx::bytes [%0], [%1, {%2, %3, %4}], [%5];"
      ::"r"(dst), "l"(reinterpret_cast<uint64_t>(map)), "r"(x), "r"(y), "r"(z), "r"(bar)
      : "memory");
}

__global__ void __launch_bounds__(kPfThreads, 2)
prefill_attn_kernel(const PrefillAttnParams p, const __grid_constant__ CUtensorMap tmQ, const __grid_constant__ CUtensorMap tmK,
                    const __grid_constant__ CUtensorMap tmV) {
  extern __shared__ __align__(1024) uint8_t pf_smem[];
  uint8_t* sm = pf_smem;
  const uint32_t sQ = smem_u32(sm);                       // [2 halves of head_dim][128 rows][128 B]
  const uint32_t sK = sQ + kPfQBytes;                     // [2 stages][2 halves][64 rows][128 B]
  const uint32_t sV = sK + 2 * kPfKvBytes;                // the same
  uint64_t* bars = reinterpret_cast<uint64_t*>(sm + kPfQBytes + 4 * kPfKvBytes);
  // barriers: 0 Q, 1-2 K stages landed, 3-4 V stages landed, 5-6 S buffers complete, 7 O += P V complete, 8-9 P written
  // (per S buffer), 10-11 V stages read, 12 the last O += P V complete, 13-14 drain.  Every barrier a thread waits on out of step with its producer is
  // one per buffer or stage: a parity wait tells a phase from the one before it, not from the one two before, and
  // with one barrier per buffer the phase after next cannot begin before the waiter has moved on.
  const uint32_t bar0 = smem_u32(bars);
  auto bar = [&](int i) { return bar0 + 8u * (uint32_t)i; };
  uint32_t* s_tmem = reinterpret_cast<uint32_t*>(bars + 15);
  volatile int* s_abort = reinterpret_cast<volatile int*>(s_tmem + 1);

  const int tid = threadIdx.x, warp = tid >> 5, lane = tid & 31;
  const int T = p.T;
  const int q0 = blockIdx.x * kPfRows;
  const int h = blockIdx.y, lb = blockIdx.z;
  const int zq = lb * p.Hq + h;
  const int zkv = lb * p.Hkv + h / (p.Hq / p.Hkv);
  const int q_last = min(T - 1, q0 + kPfRows - 1);
  const int n_kt = q_last / kPfKeys + 1;  // key tiles up to the diagonal

  // Set-up, spread over the warps so that the first tile loads are on their way as early as possible:
  // the loading thread initialises the barriers its loads complete on and issues Q, K_0, V_0 (K_1, V_1)
  // at once; thread 0 initialises the other barriers; warp 5 allocates the tensor memory.
  const bool lead4 = warp == 4 && lane == 0;
  auto load_k = [&](int j) {
    const uint32_t dst = sK + (uint32_t)(j & 1) * kPfKvBytes;
    mbar_arrive_expect_tx(bar(1 + (j & 1)), kPfKvBytes);
    pf_tma_load(dst, &tmK, 0, j * kPfKeys, zkv, bar(1 + (j & 1)));
    pf_tma_load(dst + kPfKvBytes / 2, &tmK, 64, j * kPfKeys, zkv, bar(1 + (j & 1)));
  };
  auto load_v = [&](int j) {
    const uint32_t dst = sV + (uint32_t)(j & 1) * kPfKvBytes;
    mbar_arrive_expect_tx(bar(3 + (j & 1)), kPfKvBytes);
    pf_tma_load(dst, &tmV, 0, j * kPfKeys, zkv, bar(3 + (j & 1)));
    pf_tma_load(dst + kPfKvBytes / 2, &tmV, 64, j * kPfKeys, zkv, bar(3 + (j & 1)));
  };
  if (lead4) {
    for (int i = 0; i < 5; ++i) mbar_init(bar(i), 1);
    asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory");
    asm volatile("fence.proxy.async.shared::cta;" ::: "memory");
    if ((smem_u32(sm) & 1023u) == 0u) {  // (else the tiles would not be where the swizzle expects them: see below)
      mbar_arrive_expect_tx(bar(0), kPfQBytes);
      pf_tma_load(sQ, &tmQ, 0, q0, zq, bar(0));
      pf_tma_load(sQ + kPfQBytes / 2, &tmQ, 64, q0, zq, bar(0));
      load_k(0);
      load_v(0);
      if (n_kt > 1) {
        load_k(1);
        load_v(1);
      }
    }
  }
  if (tid == 0) {
    for (int i = 5; i < 15; ++i) mbar_init(bar(i), (i == 8 || i == 9) ? kPfRows : 1);
    *s_abort = 0;
    if ((smem_u32(sm) & 1023u) != 0u) {
      atomicOr(p.err, kErrStreamBounds);
      *s_abort = 1;
    }
    asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory");
    asm volatile("fence.proxy.async.shared::cta;" ::: "memory");
  }
  if (warp == 5) {
    tc5::tmem_alloc(smem_u32(s_tmem), kPfTmemCols);
    tc5::tmem_relinquish();
  }
  tc5::fence_before_sync();
  __syncthreads();
  tc5::fence_after_sync();
  const uint32_t tmem = *s_tmem;
  const uint32_t tS0 = tmem, tO = tmem + 128;  // S buffer b at column 64 b

  if (warp == 4) {
    if (lane == 0) {
      // ================= the loading thread: TMA tile loads =================
      // (A launch whose waits run out must not take one time limit per CTA: the CTAs that start after the
      // first one gave up see the stop word here and skip the rest; their waits are bounded anyway.)
      if (*reinterpret_cast<volatile int*>(p.stop) != 0) *s_abort = 1;
      // A stage is requested again as soon as the product that read it has completed: K of tile j + 2
      // after S_j, V of tile j + 1 after O += P V of tile j - 1.  (Neither of these per-stage barriers
      // can run two phases ahead of this thread: the product that would complete the next phase needs
      // the very tile this thread loads after the wait.)
      for (int j = 0; j < n_kt && !*s_abort; ++j) {
        if (j + 2 < n_kt) {
          mbar_wait(bar(5 + (j & 1)), (uint32_t)((j >> 1) & 1), s_abort, p.err, kPfSpinLimit);
          if (!*s_abort) load_k(j + 2);
        }
        if (j >= 1 && j + 1 < n_kt) {
          mbar_wait(bar(10 + ((j - 1) & 1)), (uint32_t)(((j - 1) >> 1) & 1), s_abort, p.err, kPfSpinLimit);
          if (!*s_abort) load_v(j + 1);
        }
      }
      if (*s_abort) {
        // Something gave up.  Give the tile loads this thread started a bounded time to land before the
        // shared memory is released (every armed barrier completes its phase when its bytes are there).
        atomicOr(p.stop, 1);
        for (int i = 0; i < 5; ++i)
          for (uint32_t ph = 0; ph < 2; ++ph)
            for (uint32_t w = 0; w < (1u << 16); ++w)
              if (mbar_try_wait(bar(i), ph)) break;
      }
    }
  } else if (warp == 5) {
    // ================= the warp that issues O += P V =================
    // The whole warp runs the loop and polls the barriers (a warp of pollers notices a completed phase
    // sooner than one lane: 492 -> 468 us on config 3's prompt); one elected lane issues.  (Issued from code that only
    // one lane runs, an MMA cost about twice as long: its descriptors then live in ordinary registers
    // and have to be moved to uniform ones one by one.)
    // Operand descriptors differ only in their start-address field (bits 0-13, in units of 16 bytes):
    // one descriptor per tensor is built here, the per-instruction offsets are added to its low word.
    constexpr uint32_t idesc_o = tc5::idesc_bf16_f32(kPfRows, 128, 0, 1);       // P V: V is MN-major
    const uint64_t dV = tc5::smem_desc_sw128(sV, kPfKvBytes / 2, 1024);
    for (int j = 0; j < n_kt && !*s_abort; ++j) {
      const int st = j & 1;
      mbar_wait(bar(3 + st), (uint32_t)((j >> 1) & 1), s_abort, p.err, kPfSpinLimit);  // V_j has landed (asked for long ago)
      mbar_wait(bar(8 + st), (uint32_t)((j >> 1) & 1), s_abort, p.err, kPfSpinLimit);  // P_j written, O rescaled, S_j read
      __syncwarp();
      tc5::fence_after_sync();
      if (*s_abort) break;
      const uint64_t dVj = dV + (uint64_t)((uint32_t)st * (kPfKvBytes >> 4));
      if (tc5::elect_one()) {
#pragma unroll
        for (int kk = 0; kk < 4; ++kk)  // 16 keys per step: 8 columns of P (over S buffer j & 1), two 8-row groups (2048 bytes) of V
          tc5::mma_bf16_ts(tO, tS0 + 64u * (uint32_t)st + 8u * (uint32_t)kk, dVj + (uint64_t)(kk * 128), idesc_o,
                           (j > 0 || kk > 0) ? 1u : 0u);
        tc5::mma_commit(bar(7));
        tc5::mma_commit(bar(10 + st));  // P_j and the V stage of tile j have been read
        if (j == n_kt - 1) tc5::mma_commit(bar(12));  // O is final
      }
      __syncwarp();
    }
    if (*s_abort && tc5::elect_one()) {
      // give the MMAs already issued a bounded time to finish before the tensor memory is released
      atomicOr(p.stop, 1);
      tc5::mma_commit(bar(13));
      for (uint32_t w = 0; w < kPfSpinLimit; ++w)
        if (mbar_try_wait(bar(13), 0u)) break;
    }
  } else if (warp == 6) {
    // ================= the warp that issues S = Q K^T =================
    constexpr uint32_t idesc_s = tc5::idesc_bf16_f32(kPfRows, kPfKeys, 0, 0);   // both operands K-major
    const uint64_t dQ = tc5::smem_desc_sw128(sQ, 16, 1024);
    const uint64_t dK = tc5::smem_desc_sw128(sK, 16, 1024);
    auto mma_s = [&](int j) {  // S_j into S buffer j & 1
      const uint64_t dKj = dK + (uint64_t)((uint32_t)(j & 1) * (kPfKvBytes >> 4));
      if (tc5::elect_one()) {
#pragma unroll
        for (int kk = 0; kk < 8; ++kk)  // head_dim 16 kk .. 16 kk + 15: half kk >> 2 of the tile, 32 bytes per step inside a row
          tc5::mma_bf16_ss(tS0 + 64u * (uint32_t)(j & 1), dQ + (uint64_t)((kk >> 2) * (kPfQBytes >> 5) + (kk & 3) * 2),
                           dKj + (uint64_t)((kk >> 2) * (kPfKvBytes >> 5) + (kk & 3) * 2), idesc_s, kk > 0);
        tc5::mma_commit(bar(5 + (j & 1)));
      }
      __syncwarp();
    };
    mbar_wait(bar(0), 0u, s_abort, p.err, kPfSpinLimit);
    mbar_wait(bar(1), 0u, s_abort, p.err, kPfSpinLimit);
    __syncwarp();
    tc5::fence_after_sync();
    if (!*s_abort) mma_s(0);
    if (n_kt > 1) {
      mbar_wait(bar(2), 0u, s_abort, p.err, kPfSpinLimit);
      __syncwarp();
      tc5::fence_after_sync();
      if (!*s_abort) mma_s(1);
    }
    for (int j = 0; j + 2 < n_kt && !*s_abort; ++j) {
      const int st = j & 1;
      // S_{j+2} overwrites the columns P_j is read from, so O += P V of tile j must have completed (the
      // two products come from different warps and nothing but this barrier orders them); and its K
      // tile must have landed.
      mbar_wait(bar(1 + st), (uint32_t)(((j + 2) >> 1) & 1), s_abort, p.err, kPfSpinLimit);  // (lands first: asked for when S_j completed)
      mbar_wait(bar(10 + st), (uint32_t)((j >> 1) & 1), s_abort, p.err, kPfSpinLimit);
      __syncwarp();
      tc5::fence_after_sync();
      if (!*s_abort) mma_s(j + 2);
    }
    if (*s_abort && tc5::elect_one()) {
      atomicOr(p.stop, 1);
      tc5::mma_commit(bar(14));
      for (uint32_t w = 0; w < kPfSpinLimit; ++w)
        if (mbar_try_wait(bar(14), 0u)) break;
    }
  } else {
    // ================= softmax warps: thread = query row = tensor-memory lane =================
    const int qpos = q0 + tid;
    const uint32_t lane_base = (uint32_t)(warp * 32) << 16;
    float m = -CUDART_INF_F, l = 0.f;
    for (int j = 0; j < n_kt; ++j) {
      mbar_wait(bar(5 + (j & 1)), (uint32_t)((j >> 1) & 1), s_abort, p.err, kPfSpinLimit);  // S_j is complete
      tc5::fence_after_sync();
      uint32_t s_lo[32], s_hi[32];
      tc5::tmem_ld32(tS0 + lane_base + 64u * (uint32_t)(j & 1), s_lo);
      tc5::tmem_ld32(tS0 + lane_base + 64u * (uint32_t)(j & 1) + 32u, s_hi);
      tc5::tmem_wait_ld();
      const int key0 = j * kPfKeys;
      // Only the tiles that reach the diagonal need the mask (uniform over the CTA); the rest of the
      // row arithmetic works on the raw products: the scale is positive, so the maximum can be taken
      // before it is applied, and it is folded into the exponent's multiply-add.
      if (key0 + kPfKeys - 1 > q0) {
#pragma unroll
        for (int c = 0; c < 32; ++c) {
          if (key0 + c > qpos) s_lo[c] = 0xff800000u;       // -inf
          if (key0 + 32 + c > qpos) s_hi[c] = 0xff800000u;
        }
      }
      float mx4[4] = {-CUDART_INF_F, -CUDART_INF_F, -CUDART_INF_F, -CUDART_INF_F};
#pragma unroll
      for (int c = 0; c < 32; c += 4) {
#pragma unroll
        for (int u = 0; u < 4; ++u) mx4[u] = fmaxf(mx4[u], fmaxf(__uint_as_float(s_lo[c + u]), __uint_as_float(s_hi[c + u])));
      }
      const float mx = fmaxf(fmaxf(mx4[0], mx4[1]), fmaxf(mx4[2], mx4[3])) * p.scale_log2;
      // The reference maximum m of a row only has to keep exp2(x - m) in range, not to equal the true
      // maximum: it is moved (and O and l rescaled) only when the tile's maximum exceeds it by more
      // than 2^8, so P stays below 256 (bf16 and fp32 have the range) and most tiles rescale nothing.
      const bool move = mx > m + 8.0f;       // always at the first tile (m = -inf; key 0 is visible to every row)
      const float m_new = move ? mx : m;
      const float alpha = move ? fast_exp2(m - m_new) : 1.0f;  // 0 at the first tile, where l and O are empty
      const float neg_m = -m_new;
      float sum4[4] = {0.f, 0.f, 0.f, 0.f};
      uint32_t pk[32];  // the row's 64 weights as bf16 pairs
#pragma unroll
      for (int c = 0; c < 16; ++c) {
        const float a0 = fast_exp2(fmaf(__uint_as_float(s_lo[2 * c]), p.scale_log2, neg_m));
        const float a1 = fast_exp2(fmaf(__uint_as_float(s_lo[2 * c + 1]), p.scale_log2, neg_m));
        const float b0 = fast_exp2(fmaf(__uint_as_float(s_hi[2 * c]), p.scale_log2, neg_m));
        const float b1 = fast_exp2(fmaf(__uint_as_float(s_hi[2 * c + 1]), p.scale_log2, neg_m));
        sum4[c & 3] += (a0 + a1) + (b0 + b1);
        pk[c] = pack_bf16x2(a0, a1);
        pk[16 + c] = pack_bf16x2(b0, b1);
      }
      const float sum = (sum4[0] + sum4[1]) + (sum4[2] + sum4[3]);
      l = l * alpha + sum;
      m = m_new;
      if (j > 0 && __any_sync(0xffffffffu, move)) {  // warp-uniform: the tensor-memory accesses are collective
        // O += P V of the tile before must be complete before O is rescaled.  (That of the tile before it
        // is: S_j was issued after it had completed.  So the parity wait cannot mistake the phases.)
        mbar_wait(bar(7), (uint32_t)((j - 1) & 1), s_abort, p.err, kPfSpinLimit);
        tc5::fence_after_sync();
#pragma unroll
        for (int c0 = 0; c0 < 128; c0 += 32) {
          uint32_t o[32];
          tc5::tmem_ld32(tO + lane_base + (uint32_t)c0, o);
          tc5::tmem_wait_ld();
#pragma unroll
          for (int c = 0; c < 32; ++c) o[c] = __float_as_uint(__uint_as_float(o[c]) * alpha);
          tc5::tmem_st32(tO + lane_base + (uint32_t)c0, o);
        }
      }
      // the row of P over the first 32 columns of the S tile it was computed from (this thread has read
      // its row of S; nothing else reads that buffer before the product that follows)
      tc5::tmem_st32(tS0 + lane_base + 64u * (uint32_t)(j & 1), pk);
      tc5::tmem_wait_st();
      tc5::fence_before_sync();
      mbar_arrive(bar(8 + (j & 1)));
    }
    // epilogue: the row of O, normalised, rounded to bf16
    mbar_wait(bar(12), 0u, s_abort, p.err, kPfSpinLimit);  // (a barrier of its own: it has this one phase)
    tc5::fence_after_sync();
    const float inv_l = 1.0f / l;
    __nv_bfloat16* orow = p.out + ((size_t)zq * T + (size_t)min(qpos, T - 1)) * 128;
    const bool aborted = *s_abort != 0;  // (then tensor memory may not hold what this row expects: nothing is written)
#pragma unroll
    for (int c0 = 0; c0 < 128; c0 += 64) {
      uint32_t o[2][32];
      tc5::tmem_ld32(tO + lane_base + (uint32_t)c0, o[0]);
      tc5::tmem_ld32(tO + lane_base + (uint32_t)c0 + 32u, o[1]);
      tc5::tmem_wait_ld();
      if (qpos < T && !aborted) {
#pragma unroll
        for (int hh = 0; hh < 2; ++hh) {
#pragma unroll
          for (int c = 0; c < 32; c += 8) {
            uint4 w;
            w.x = pack_bf16x2(__uint_as_float(o[hh][c]) * inv_l, __uint_as_float(o[hh][c + 1]) * inv_l);
            w.y = pack_bf16x2(__uint_as_float(o[hh][c + 2]) * inv_l, __uint_as_float(o[hh][c + 3]) * inv_l);
            w.z = pack_bf16x2(__uint_as_float(o[hh][c + 4]) * inv_l, __uint_as_float(o[hh][c + 5]) * inv_l);
            w.w = pack_bf16x2(__uint_as_float(o[hh][c + 6]) * inv_l, __uint_as_float(o[hh][c + 7]) * inv_l);
            *reinterpret_cast<uint4*>(orow + c0 + 32 * hh + c) = w;
          }
        }
      }
    }
  }
  tc5::fence_before_sync();
  __syncthreads();
  if (warp == 5) tc5::tmem_dealloc(tmem, kPfTmemCols);
}

}  // namespace dynts

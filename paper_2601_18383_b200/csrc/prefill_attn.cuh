// Prefill attention for sm_100a: every prompt position attends to the positions up to and
// including itself (Eq. 4-5 with t = 1..M), bf16, head_dim 128, grouped query heads.  This is the
// phase that fills the question window (Section 4.2); unlike the decode step it is a dense
// contraction (M x M x d per head), and it runs on the 5th-generation tensor path: tcgen05.mma with
// the accumulators in tensor memory, operands brought into shared memory by TMA tile loads.
//
// A work item = 128 query rows of one query head.  The grid is two CTAs per SM, each working through
// its share of the items (heaviest first: see PfCursor) without tearing its pipeline down in
// between: the loads and the first product of the next item are issued while the last tiles of the
// current one are in the softmax, so the fill and drain of an item (about 4 us when each item was a
// CTA of its own, against 1.1 us per tile) overlap the neighbouring items.  An item walks the
// key/value rows in tiles of 64 up to the diagonal; per tile
//     S  = Q K^T          M 128 x N 64 x K 128   (8 instructions of K = 16; Q and K tiles K-major)
//     P  = exp2(S * scale - rowmax)               (online softmax: running max and sum per row)
//     O += P V            M 128 x N 128 x K 64   (4 instructions; P from tensor memory, V MN-major)
// Seven warps.  Warps 0-3 are the softmax warps: thread r owns query row r, i.e. lane r of tensor
// memory -- it reads its row of S with tcgen05.ld, keeps the row's running max and sum, rescales
// its row of O in tensor memory when the max moves, and writes its row of P (bf16, two per column)
// back into tensor memory over the S tile it came from, where the second product reads it as its
// A operand: P never touches shared memory and the softmax of a tile does not wait for the product
// of the tile before (unless the row's reference maximum has to move).  One thread of
// warp 4 issues the TMA loads (Q once per item; K and V tiles into two stages each, requested as soon as the
// product that read the stage before has completed), one lane of warp 5 the second product and
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
constexpr int kPfThreads = 256;                   // 4 softmax warps, the Q/K loading warp, one warp each for O += P V and S = Q K^T, the V loading warp
constexpr int kPfQBytes = kPfRows * 256;          // two boxes of 128 rows x 64 bf16
constexpr int kPfKvBytes = kPfKeys * 256;         // two boxes of 64 rows x 64 bf16
// Two CTAs must fit the 227 KB of an SM (each also costs 1 KB of system space), so there is no room
// for alignment slack: the dynamic shared memory is declared 1024-byte aligned (what the 128-byte
// swizzle needs) and the kernel checks that it is.
constexpr int kPfOutStageBytes = 4 * 32 * 128;    // per softmax warp: 32 rows x 64 bf16, the staging of half an output tile
constexpr int kPfSmemBytes = kPfQBytes + 4 * kPfKvBytes + kPfOutStageBytes + 128;
constexpr uint32_t kPfTmemCols = 256;             // S0 | S1 | O
constexpr uint32_t kPfSpinLimit = 1u << 21;

struct PrefillAttnParams {
  __nv_bfloat16* out;      // [L, Nb, Hq, T, 128]
  int* err;                // pinned host status word
  int* stop;               // device word: non-zero once a CTA of this cache's prefill launches has given up a wait
  int T, Hq, Hkv;
  int n_qt;                // query tiles of 128 rows per head
  int n_heads;             // layers x sequences x query heads of this launch
  float scale_log2;
};

// One work item = (query tile, query head).  The items are numbered heaviest first (the tile nearest
// the end of the prompt has the most key tiles below the diagonal), heads fastest, and CTA b takes
// the items b, b + gridDim.x, ...: every CTA gets its share of each weight class, and the CTAs
// running side by side work on the query heads of the same few KV heads, whose tiles they share in L2.
struct PfCursor {
  int it;    // index in this CTA's list of items
  int j;     // key tile within the item
  int nkt;   // key tiles of the item (up to the diagonal)
  int q0;    // first query row
  int zq;    // (layer, sequence, query head) flattened: the tensor maps' outer coordinate
  int zkv;   // the same for the KV head
};

__device__ __forceinline__ void pf_seek(PfCursor& c, int it, int n_items, const PrefillAttnParams& p) {
  c.it = it;
  c.j = 0;
  if (it >= n_items) return;
  // The second half of the grid takes its items lightest first: the two CTAs of an SM (one of each
  // half, when the CTAs are handed out SM by SM) then reach their item boundaries at different times,
  // and one fills the issue slots while the other drains and refills its pipeline.
  const int slot = 2 * (int)blockIdx.x >= (int)gridDim.x ? n_items - 1 - it : it;
  const int w = (int)blockIdx.x + slot * (int)gridDim.x;
  const int cls = w / p.n_heads;
  c.zq = w - cls * p.n_heads;
  c.q0 = (p.n_qt - 1 - cls) * kPfRows;
  c.nkt = min(p.T - 1, c.q0 + kPfRows - 1) / kPfKeys + 1;
  const int lb = c.zq / p.Hq, h = c.zq - lb * p.Hq;
  c.zkv = lb * p.Hkv + h / (p.Hq / p.Hkv);
}
__device__ __forceinline__ void pf_advance(PfCursor& c, int n_items, const PrefillAttnParams& p) {
  if (++c.j == c.nkt) pf_seek(c, c.it + 1, n_items, p);
}

__device__ __forceinline__ void pf_tma_load(uint32_t dst, const CUtensorMap* map, int x, int y, int z, uint32_t bar) {
  asm volatile(
      "cp.async.bulk.tensor.3d.shared::cluster.global.tile.mbarrier::complete_tx::bytes [%0], [%1, {%2, %3, %4}], [%5];"
      ::"r"(dst), "l"(reinterpret_cast<uint64_t>(map)), "r"(x), "r"(y), "r"(z), "r"(bar)
      : "memory");
}

// Asks the lines of a tile into L2 (no shared-memory destination, nothing to wait for).
__device__ __forceinline__ void pf_tma_prefetch(const CUtensorMap* map, int x, int y, int z) {
  asm volatile("cp.async.bulk.prefetch.tensor.3d.L2.global.tile [%0, {%1, %2, %3}];" ::"l"(reinterpret_cast<uint64_t>(map)), "r"(x),
               "r"(y), "r"(z)
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
  uint8_t* s_out = sm + kPfQBytes + 4 * kPfKvBytes;       // [4 softmax warps][32 rows][128 B], chunks of 16 B swizzled by row
  uint64_t* bars = reinterpret_cast<uint64_t*>(s_out + kPfOutStageBytes);
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
  const int n_work = p.n_qt * p.n_heads;
  const int n_items = (n_work - (int)blockIdx.x + (int)gridDim.x - 1) / (int)gridDim.x;  // >= 1: the grid is no larger than the work
  // Every role walks the same flat sequence of key tiles g = 0, 1, ... over the CTA's items; the S
  // buffer, the K and V stages and the phases of their barriers follow g, not the tile's index
  // within its item, so that the products and loads of the next item start while the last tiles of
  // the current one are still in the softmax.
  PfCursor first;
  pf_seek(first, 0, n_items, p);

  // Set-up, spread over the warps so that the first tile loads are on their way as early as possible:
  // the loading thread initialises the barriers its loads complete on and issues Q and the first two
  // K and V tiles at once; thread 0 initialises the other barriers; warp 5 allocates the tensor memory.
  const bool lead4 = warp == 4 && lane == 0;
  auto load_q = [&](const PfCursor& c) {
    mbar_arrive_expect_tx(bar(0), kPfQBytes);
    pf_tma_load(sQ, &tmQ, 0, c.q0, c.zq, bar(0));
    pf_tma_load(sQ + kPfQBytes / 2, &tmQ, 64, c.q0, c.zq, bar(0));
  };
  auto load_k = [&](const PfCursor& c, int g) {
    const uint32_t dst = sK + (uint32_t)(g & 1) * kPfKvBytes;
    mbar_arrive_expect_tx(bar(1 + (g & 1)), kPfKvBytes);
    pf_tma_load(dst, &tmK, 0, c.j * kPfKeys, c.zkv, bar(1 + (g & 1)));
    pf_tma_load(dst + kPfKvBytes / 2, &tmK, 64, c.j * kPfKeys, c.zkv, bar(1 + (g & 1)));
  };
  auto load_v = [&](const PfCursor& c, int g) {
    const uint32_t dst = sV + (uint32_t)(g & 1) * kPfKvBytes;
    mbar_arrive_expect_tx(bar(3 + (g & 1)), kPfKvBytes);
    pf_tma_load(dst, &tmV, 0, c.j * kPfKeys, c.zkv, bar(3 + (g & 1)));
    pf_tma_load(dst + kPfKvBytes / 2, &tmV, 64, c.j * kPfKeys, c.zkv, bar(3 + (g & 1)));
  };
  PfCursor second = first;          // flat tile 1
  pf_advance(second, n_items, p);
  PfCursor third = second;          // flat tile 2: the first one the loading warps ask for in their loops
  pf_advance(third, n_items, p);
  if (lead4) {
    for (int i = 0; i < 5; ++i) mbar_init(bar(i), 1);
    asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory");
    asm volatile("fence.proxy.async.shared::cta;" ::: "memory");
    if ((smem_u32(sm) & 1023u) == 0u) {  // (else the tiles would not be where the swizzle expects them: see below)
      load_q(first);
      load_k(first, 0);
      load_v(first, 0);
      if (second.it < n_items) {
        load_k(second, 1);
        load_v(second, 1);
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
    // ================= the warp that loads Q and K =================
    // Like the warps that issue the products, the whole warp runs the loop and polls (a single polling
    // lane saw a completed phase up to 1.4 us late, which delayed the next item's Q by as much); one
    // elected lane issues the loads.
    // (A launch whose waits run out must not take one time limit per CTA: the CTAs that start after the
    // first one gave up see the stop word here and skip the rest; their waits are bounded anyway.)
    if (lane == 0 && *reinterpret_cast<volatile int*>(p.stop) != 0) *s_abort = 1;
    __syncwarp();
    // A stage is requested again as soon as the product that read it has completed: K of tile g + 2
    // after S_g; the next item's Q after the last S of this one (its lines were asked into L2 when this
    // item began).  (Neither barrier can run two phases ahead of this warp: the product that would
    // complete the next phase needs the very tile this warp loads after the wait.)
    PfCursor cur = first, cK = third;
    for (int g = 0; cur.it < n_items && !*s_abort; ++g) {
      const bool next_q = cur.j == cur.nkt - 1 && cur.it + 1 < n_items;
      if (cur.j == 0 && cur.it + 1 < n_items && tc5::elect_one()) {
        PfCursor nq;
        pf_seek(nq, cur.it + 1, n_items, p);
        pf_tma_prefetch(&tmQ, 0, nq.q0, nq.zq);
        pf_tma_prefetch(&tmQ, 64, nq.q0, nq.zq);
      }
      if (cK.it < n_items || next_q) {
        mbar_wait(bar(5 + (g & 1)), (uint32_t)((g >> 1) & 1), s_abort, p.err, kPfSpinLimit);
        __syncwarp();
        if (!*s_abort && tc5::elect_one()) {
          if (next_q) {
            PfCursor nq;
            pf_seek(nq, cur.it + 1, n_items, p);
            load_q(nq);
          }
          if (cK.it < n_items) load_k(cK, g);  // tile g + 2: the stage S_g read
        }
        __syncwarp();
        if (cK.it < n_items) pf_advance(cK, n_items, p);
      }
      pf_advance(cur, n_items, p);
    }
    if (*s_abort && lane == 0) {
      // Something gave up.  Give the tile loads this warp started a bounded time to land before the
      // shared memory is released (every armed barrier completes its phase when its bytes are there).
      atomicOr(p.stop, 1);
      for (int i = 0; i < 3; ++i)
        for (uint32_t ph = 0; ph < 2; ++ph)
          for (uint32_t w = 0; w < (1u << 16); ++w)
            if (mbar_try_wait(bar(i), ph)) break;
    }
  } else if (warp == 7) {
    // ================= the warp that loads V =================
    // V of tile g + 1 after O += P V of tile g - 1 has completed (the stage it read).
    PfCursor cV = third;
    for (int g = 1; cV.it < n_items && !*s_abort; ++g) {
      mbar_wait(bar(10 + ((g - 1) & 1)), (uint32_t)(((g - 1) >> 1) & 1), s_abort, p.err, kPfSpinLimit);
      __syncwarp();
      if (!*s_abort && tc5::elect_one()) load_v(cV, g + 1);
      __syncwarp();
      pf_advance(cV, n_items, p);
    }
    if (*s_abort && lane == 0) {
      atomicOr(p.stop, 1);
      for (int i = 3; i < 5; ++i)
        for (uint32_t ph = 0; ph < 2; ++ph)
          for (uint32_t w = 0; w < (1u << 16); ++w)
            if (mbar_try_wait(bar(i), ph)) break;
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
    PfCursor cur = first;
    for (int g = 0; cur.it < n_items && !*s_abort; ++g) {
      const int st = g & 1;
      mbar_wait(bar(3 + st), (uint32_t)((g >> 1) & 1), s_abort, p.err, kPfSpinLimit);  // V of this tile has landed (asked for long ago)
      // P written, S read -- and, at the first tile of an item, the softmax warps have read the O of the item before
      mbar_wait(bar(8 + st), (uint32_t)((g >> 1) & 1), s_abort, p.err, kPfSpinLimit);
      __syncwarp();
      tc5::fence_after_sync();
      if (*s_abort) break;
      const uint64_t dVg = dV + (uint64_t)((uint32_t)st * (kPfKvBytes >> 4));
      if (tc5::elect_one()) {
#pragma unroll
        for (int kk = 0; kk < 4; ++kk)  // 16 keys per step: 8 columns of P (over S buffer g & 1), two 8-row groups (2048 bytes) of V
          tc5::mma_bf16_ts(tO, tS0 + 64u * (uint32_t)st + 8u * (uint32_t)kk, dVg + (uint64_t)(kk * 128), idesc_o,
                           (cur.j > 0 || kk > 0) ? 1u : 0u);
        tc5::mma_commit(bar(7));
        tc5::mma_commit(bar(10 + st));  // P and the V stage of this tile have been read
        if (cur.j == cur.nkt - 1) tc5::mma_commit(bar(12));  // the item's O is final
      }
      __syncwarp();
      pf_advance(cur, n_items, p);
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
    auto mma_s = [&](int g) {  // S of flat tile g into S buffer g & 1, from K stage g & 1
      const uint64_t dKg = dK + (uint64_t)((uint32_t)(g & 1) * (kPfKvBytes >> 4));
      if (tc5::elect_one()) {
#pragma unroll
        for (int kk = 0; kk < 8; ++kk)  // head_dim 16 kk .. 16 kk + 15: half kk >> 2 of the tile, 32 bytes per step inside a row
          tc5::mma_bf16_ss(tS0 + 64u * (uint32_t)(g & 1), dQ + (uint64_t)((kk >> 2) * (kPfQBytes >> 5) + (kk & 3) * 2),
                           dKg + (uint64_t)((kk >> 2) * (kPfKvBytes >> 5) + (kk & 3) * 2), idesc_s, kk > 0);
        tc5::mma_commit(bar(5 + (g & 1)));
      }
      __syncwarp();
    };
    PfCursor cur = first;
    for (int g = 0; cur.it < n_items && !*s_abort; ++g) {
      const int st = g & 1;
      mbar_wait(bar(1 + st), (uint32_t)((g >> 1) & 1), s_abort, p.err, kPfSpinLimit);  // the tile's K
      // S of tile g overwrites the columns P of tile g - 2 is read from, so O += P V of that tile must
      // have completed (the two products come from different warps and nothing but this barrier orders them).
      if (g >= 2) mbar_wait(bar(10 + st), (uint32_t)(((g - 2) >> 1) & 1), s_abort, p.err, kPfSpinLimit);
      // the item's Q: the last to arrive at the first tile of an item (asked for when the last S of the item before completed)
      if (cur.j == 0) mbar_wait(bar(0), (uint32_t)(cur.it & 1), s_abort, p.err, kPfSpinLimit);
      __syncwarp();
      tc5::fence_after_sync();
      if (!*s_abort) mma_s(g);
      pf_advance(cur, n_items, p);
    }
    if (*s_abort && tc5::elect_one()) {
      atomicOr(p.stop, 1);
      tc5::mma_commit(bar(14));
      for (uint32_t w = 0; w < kPfSpinLimit; ++w)
        if (mbar_try_wait(bar(14), 0u)) break;
    }
  } else {
    // ================= softmax warps: thread = query row = tensor-memory lane =================
    const uint32_t lane_base = (uint32_t)(warp * 32) << 16;
    // epilogue of an item: the row of O, normalised, rounded to bf16.  (A barrier of its own, one phase per
    // item: the next item's first O = P V, which would complete the phase after, waits for the P this
    // thread writes once it has read its row of O here.)
    auto epilogue = [&](float l, int q0, int zq, int it) {
    mbar_wait(bar(12), (uint32_t)(it & 1), s_abort, p.err, kPfSpinLimit);
    tc5::fence_after_sync();
    const float inv_l = 1.0f / l;
    const uint64_t inv2 = tc5::f2_pack(inv_l, inv_l);
    const bool aborted = *s_abort != 0;  // (then tensor memory may not hold what this row expects: nothing is written)
    // Half a row (64 columns, 128 bytes) at a time goes through the warp's staging tile so that the
    // global stores are whole 128-byte lines: a thread writes its half row as eight 16-byte chunks,
    // chunk c at position c ^ (row & 7) (conflict-free), then every eight lanes read one row back and
    // store it.  (Stored straight from the registers, a warp's store touched 32 different lines, and
    // the 16 of them took 1.4 us per item.)
    uint8_t* stage = s_out + warp * (32 * 128);
    __nv_bfloat16* obase = p.out + ((size_t)zq * T + (size_t)(q0 + warp * 32)) * 128;
    const int rows_here = T - (q0 + warp * 32);  // rows of this warp inside the prompt (may be <= 0 or > 32)
#pragma unroll
    for (int c0 = 0; c0 < 128; c0 += 64) {
      uint32_t o[2][32];
      tc5::tmem_ld32(tO + lane_base + (uint32_t)c0, o[0]);
      tc5::tmem_ld32(tO + lane_base + (uint32_t)c0 + 32u, o[1]);
      tc5::tmem_wait_ld();
#pragma unroll
      for (int hh = 0; hh < 2; ++hh) {
#pragma unroll
        for (int c = 0; c < 32; c += 8) {
          uint32_t w[4];
#pragma unroll
          for (int u = 0; u < 4; ++u) {
            float y0, y1;
            tc5::f2_unpack(tc5::f2_mul(tc5::f2_pack(__uint_as_float(o[hh][c + 2 * u]), __uint_as_float(o[hh][c + 2 * u + 1])), inv2), y0, y1);
            w[u] = pack_bf16x2(y0, y1);
          }
          const int chunk = 4 * hh + (c >> 3);
          *reinterpret_cast<uint4*>(stage + lane * 128 + ((chunk ^ (lane & 7)) << 4)) = make_uint4(w[0], w[1], w[2], w[3]);
        }
      }
      __syncwarp();
#pragma unroll
      for (int i = 0; i < 8; ++i) {
        const int row = 4 * i + (lane >> 3), chunk = lane & 7;
        const uint4 w = *reinterpret_cast<const uint4*>(stage + row * 128 + ((chunk ^ (row & 7)) << 4));
        if (row < rows_here && !aborted) *reinterpret_cast<uint4*>(obase + (size_t)row * 128 + c0 + chunk * 8) = w;
      }
      __syncwarp();
    }
    };
    bool ep_on = false;  // an item whose epilogue is still to run, and what it needs
    float ep_l = 0.f;
    int ep_q0 = 0, ep_zq = 0, ep_it = 0;
    PfCursor cur = first;
    int g = 0;  // flat tile index: S buffer g & 1
    while (cur.it < n_items) {
    const int it = cur.it, n_kt = cur.nkt, q0 = cur.q0, zq = cur.zq;
    const int qpos = q0 + tid;
    float m = -CUDART_INF_F, l = 0.f;
    for (int j = 0; j < n_kt; ++j, ++g) {
      mbar_wait(bar(5 + (g & 1)), (uint32_t)((g >> 1) & 1), s_abort, p.err, kPfSpinLimit);  // S of this tile is complete
      tc5::fence_after_sync();
      uint32_t s_lo[32], s_hi[32];
      tc5::tmem_ld32(tS0 + lane_base + 64u * (uint32_t)(g & 1), s_lo);
      tc5::tmem_ld32(tS0 + lane_base + 64u * (uint32_t)(g & 1) + 32u, s_hi);
      tc5::tmem_wait_ld();
      const int key0 = j * kPfKeys;
      // The causal mask, per warp (32 rows) and half tile (32 keys): the first row minus the first key
      // is a multiple of 32, so a half is either fully visible (>= 32), hidden (< 0) or the triangle
      // "key c <= lane" (0).  All of it is warp-uniform; only a triangle costs compares, and a hidden
      // half costs nothing (its weights are zero).  The rest of the row arithmetic works on the raw
      // products: the scale is positive, so the maximum can be taken before it is applied, and it is
      // folded into the exponent's multiply-add.
      const int d_lo = q0 + warp * 32 - key0, d_hi = d_lo - 32;
      const bool lo_live = d_lo >= 0, hi_live = d_hi >= 0;
      if (d_lo == 0) {
#pragma unroll
        for (int c = 1; c < 32; ++c)
          if (c > lane) s_lo[c] = 0xff800000u;  // -inf
      }
      if (d_hi == 0) {
#pragma unroll
        for (int c = 1; c < 32; ++c)
          if (c > lane) s_hi[c] = 0xff800000u;
      }
      auto max_half = [](const uint32_t (&sv)[32]) {  // four chains of three-input maxima
        float mx4[4] = {-CUDART_INF_F, -CUDART_INF_F, -CUDART_INF_F, -CUDART_INF_F};
#pragma unroll
        for (int c = 0; c < 32; c += 8) {
#pragma unroll
          for (int u = 0; u < 4; ++u) mx4[u] = tc5::f_max3(mx4[u], __uint_as_float(sv[c + u]), __uint_as_float(sv[c + 4 + u]));
        }
        return tc5::f_max3(fmaxf(mx4[0], mx4[1]), mx4[2], mx4[3]);
      };
      float mxr = -CUDART_INF_F;
      if (lo_live) mxr = max_half(s_lo);
      if (hi_live) mxr = fmaxf(mxr, max_half(s_hi));
      const float mx = mxr * p.scale_log2;
      // The reference maximum m of a row only has to keep exp2(x - m) in range, not to equal the true
      // maximum: it is moved (and O and l rescaled) only when the tile's maximum exceeds it by more
      // than 2^8, so P stays below 256 (bf16 and fp32 have the range) and most tiles rescale nothing.
      const bool move = mx > m + 8.0f;       // always at the first tile (m = -inf; key 0 is visible to every row)
      const float m_new = move ? mx : m;
      const float alpha = move ? fast_exp2(m - m_new) : 1.0f;  // 0 at the first tile, where l and O are empty
      const float neg_m = -m_new;
      const float scale_log2 = p.scale_log2;
      uint32_t pk[32];  // the row's 64 weights as bf16 pairs
      const uint64_t scale2 = tc5::f2_pack(scale_log2, scale_log2), negm2 = tc5::f2_pack(neg_m, neg_m);
      auto exp_half = [scale2, negm2](const uint32_t (&sv)[32], uint32_t* out) {
        uint64_t sum2[4] = {0ull, 0ull, 0ull, 0ull};  // four chains of (even, odd) column sums
#pragma unroll
        for (int c = 0; c < 16; ++c) {
          float x0, x1;
          tc5::f2_unpack(tc5::f2_fma(tc5::f2_pack(__uint_as_float(sv[2 * c]), __uint_as_float(sv[2 * c + 1])), scale2, negm2), x0, x1);
          const float a0 = fast_exp2(x0), a1 = fast_exp2(x1);
          sum2[c & 3] = tc5::f2_add(sum2[c & 3], tc5::f2_pack(a0, a1));
          out[c] = pack_bf16x2(a0, a1);
        }
        float e, o;
        tc5::f2_unpack(tc5::f2_add(tc5::f2_add(sum2[0], sum2[1]), tc5::f2_add(sum2[2], sum2[3])), e, o);
        return e + o;
      };
      float sum = 0.f;
      if (lo_live) {
        sum = exp_half(s_lo, pk);
      } else {
#pragma unroll
        for (int c = 0; c < 16; ++c) pk[c] = 0u;
      }
      if (hi_live) {
        sum += exp_half(s_hi, pk + 16);
      } else {
#pragma unroll
        for (int c = 0; c < 16; ++c) pk[16 + c] = 0u;
      }
      l = l * alpha + sum;
      m = m_new;
      if (j > 0 && __any_sync(0xffffffffu, move)) {  // warp-uniform: the tensor-memory accesses are collective
        // O += P V of the tile before must be complete before O is rescaled.  (That of the tile before it
        // is: this tile's S was issued after it had completed.  So the parity wait cannot mistake the phases.)
        mbar_wait(bar(7), (uint32_t)((g - 1) & 1), s_abort, p.err, kPfSpinLimit);
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
      // At the first tile of an item the epilogue of the item before is still to run: its last
      // O += P V has had the time of this tile's row arithmetic to complete, and the first O = P V of
      // this item, which overwrites O, cannot be issued before the P stored below.
      if (ep_on) {
        epilogue(ep_l, ep_q0, ep_zq, ep_it);
        ep_on = false;
      }
      // the row of P over the first 32 columns of the S tile it was computed from (this thread has read
      // its row of S; nothing else reads that buffer before the product that follows)
      tc5::tmem_st32(tS0 + lane_base + 64u * (uint32_t)(g & 1), pk);
      tc5::tmem_wait_st();
      tc5::fence_before_sync();
      mbar_arrive(bar(8 + (g & 1)));
    }
    // The item's epilogue is run inside the first tile of the next item (see above): the weights of
    // that tile are computed while the last O += P V of this item completes.
    ep_on = true;
    ep_l = l;
    ep_q0 = q0;
    ep_zq = zq;
    ep_it = it;
    pf_seek(cur, it + 1, n_items, p);
    }  // items
    if (ep_on) epilogue(ep_l, ep_q0, ep_zq, ep_it);
  }
  tc5::fence_before_sync();
  __syncthreads();
  if (warp == 5) tc5::tmem_dealloc(tmem, kPfTmemCols);
}

}  // namespace dynts

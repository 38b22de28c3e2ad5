// Budgeted eviction (Section 4.2) for sm_100a: selection, then in-place stable compaction.
//
//   evict_select_kernel   one CTA per slab.  Scores are compared through an order-preserving
//                         map of their fp32 bit patterns to uint32, so every decision is integer
//                         arithmetic.  A 4-pass, 8-bit radix select finds the k-th largest key T
//                         of the selection window; rows with key > T survive, and of the rows
//                         with key == T the lowest-indexed survive until k is reached (a prefix
//                         count gives each its rank).  A second prefix count over the survivor
//                         flags gives every survivor its destination row; the kernel writes the
//                         gather list src[dst] and compacts score and pos itself.
//   evict_compact_kernel  moves the K and V rows.  The gather is stable and only moves rows
//                         towards lower indices (src[dst] >= dst, both increasing), so a CTA that
//                         walks the destination rows in ascending chunks and, per chunk, loads
//                         every source row before storing any destination row never overwrites
//                         data it still needs.  CTAs split the row bytes into 64-byte column
//                         groups (and K from V), which makes them fully independent: no
//                         inter-CTA ordering, no second buffer.
#pragma once

#include "common.cuh"
#include "decode_stream.cuh"  // score_pass_lean, kStPendWords: recorded score passes are applied here

namespace dynts {

constexpr int kSelectThreads = 1024;
constexpr int kCompactThreads = 256;
constexpr int kCompactUnroll = 8;                                         // 16-byte loads in flight per thread
constexpr int kCompactRowsPerPass = kCompactThreads / 4;                  // 4 threads cover one 64-byte group
constexpr int kCompactChunkRows = kCompactRowsPerPass * kCompactUnroll;   // rows per load/store phase

// fp32 -> uint32 with the same order as the float comparison; -0 and +0 get the same key.
__device__ __forceinline__ uint32_t order_key(uint32_t raw_bits) {
  const float s = __fadd_rn(__uint_as_float(raw_bits), 0.0f);
  const uint32_t b = __float_as_uint(s);
  return (b & 0x80000000u) ? ~b : (b | 0x80000000u);
}

// Exclusive prefix count of a per-thread flag over the CTA, plus the CTA total.
__device__ __forceinline__ int block_prefix_count(bool flag, int* warp_tot /* [32] shared */, int& total) {
  const int lane = threadIdx.x & 31, warp = threadIdx.x >> 5;
  const unsigned bal = __ballot_sync(0xffffffffu, flag);
  const int in_warp = __popc(bal & ((1u << lane) - 1u));
  if (lane == 0) warp_tot[warp] = __popc(bal);
  __syncthreads();
  const int nwarps = blockDim.x >> 5;
  int before = 0, tot = 0;
  for (int w = 0; w < nwarps; ++w) {
    const int t = warp_tot[w];
    if (w < warp) before += t;
    tot += t;
  }
  __syncthreads();  // warp_tot may be reused right after
  total = tot;
  return before + in_warp;
}

__global__ void __launch_bounds__(kSelectThreads) evict_select_kernel(const EvictParams p) {
  const int slab = blockIdx.x;
  const int b = (slab / p.Hkv) % p.Nb;
  const int tid = threadIdx.x;
  const int n = p.len[b];
  const int tgt = p.target[b];
  int* hdr = p.hdr + (size_t)slab * 4;
  if (n <= tgt) {  // nothing to evict for this sequence
    if (tid == 0) {
      hdr[0] = n;
      hdr[1] = n;
      hdr[2] = n;
    }
    return;
  }
  const int M = p.pinned[b];
  const int lo = M, hi = n - p.window;  // selection window [lo, hi)
  const int k = tgt - M - p.window;     // survivors wanted from it (host guarantees 0 <= k < hi - lo)
  if (n > p.cap || M < 0 || k < 0 || hi < lo || k > hi - lo) {  // uniform over the CTA; the host's checks prevent it
    if (tid == 0) {
      atomicOr(p.err, kErrLenOverflow);  // recorded, and nothing moves
      hdr[0] = n;
      hdr[1] = n;
      hdr[2] = n;
    }
    return;
  }

  extern __shared__ __align__(16) uint32_t esm[];
  uint32_t* raw = esm;                                   // [cap] score bit patterns
  int* posbuf = reinterpret_cast<int*>(esm + p.cap);     // [cap]
  uint32_t* compbuf = esm + 2 * (size_t)p.cap;           // [cap], only with p.comp
  __shared__ unsigned int hist[256];
  __shared__ int warp_tot[32];
  __shared__ uint32_t s_prefix;
  __shared__ int s_krem, s_first;

  float* score = p.score + (size_t)slab * p.cap;
  int* pos = p.pos + (size_t)slab * p.cap;
  int* src = p.src + (size_t)slab * p.cap;
  float* comp = p.comp ? p.comp + (size_t)slab * p.cap : nullptr;
  // bit patterns the selection ranks by: the slab's own scores, or keys shared by all slabs of the
  // sequence (read from global memory: such slabs may leave no shared memory for a copy)
  const uint32_t* sel = p.key ? reinterpret_cast<const uint32_t*>(p.key + (size_t)b * p.cap) : raw;
  for (int j = tid; j < n; j += kSelectThreads) {
    raw[j] = __float_as_uint(score[j]);
    posbuf[j] = pos[j];
    if (comp) compbuf[j] = __float_as_uint(comp[j]);
  }
  if (tid == 0) {
    s_prefix = 0u;
    s_krem = k;
    s_first = n;
  }
  __syncthreads();

  // Radix select: after the pass for `shift`, s_prefix holds the top bits of the k-th largest
  // key and s_krem how many rows with exactly those top bits must still be taken.
  uint32_t mask = 0u;
  if (k > 0) {
    for (int shift = 24; shift >= 0; shift -= 8) {
      if (tid < 256) hist[tid] = 0u;
      __syncthreads();
      const uint32_t prefix = s_prefix;
      const int krem = s_krem;  // read by everyone before warp 0 updates it below
      for (int j = lo + tid; j < hi; j += kSelectThreads) {
        const uint32_t key = order_key(sel[j]);
        if ((key & mask) == prefix) atomicAdd(&hist[(key >> shift) & 255u], 1u);
      }
      __syncthreads();
      if (tid < 32) {
        // lane l owns bins 255-8l .. 248-8l (descending); find where the count from the top
        // reaches krem.
        unsigned int mine = 0;
        for (int i = 0; i < 8; ++i) mine += hist[255 - 8 * tid - i];
        unsigned int incl = mine;
        for (int o = 1; o < 32; o <<= 1) {
          const unsigned int v = __shfl_up_sync(0xffffffffu, incl, o);
          if (tid >= o) incl += v;
        }
        const unsigned int excl = incl - mine;
        if ((int)excl < krem && krem <= (int)incl) {
          unsigned int above = excl;
          for (int i = 0; i < 8; ++i) {
            const int bin = 255 - 8 * tid - i;
            const unsigned int c = hist[bin];
            if ((int)(above + c) >= krem) {
              s_prefix = prefix | ((uint32_t)bin << shift);
              s_krem = krem - (int)above;
              break;
            }
            above += c;
          }
        }
      }
      mask |= 0xFFu << shift;
      __syncthreads();
    }
  }
  const uint32_t T = s_prefix;   // key of the k-th largest candidate
  const int take_eq = s_krem;    // rows with key == T that survive (lowest indices first)

  int carry_eq = 0, carry_keep = 0;
  for (int base = 0; base < n; base += kSelectThreads) {
    const int j = base + tid;
    const bool in = j < n;
    const bool cand = in && j >= lo && j < hi;
    uint32_t key = 0u;
    if (cand) key = order_key(sel[j]);
    const bool gt = cand && k > 0 && key > T;
    const bool eq = cand && k > 0 && key == T;
    int tot_eq, tot_keep;
    const int eq_rank = carry_eq + block_prefix_count(eq, warp_tot, tot_eq);
    const bool keep = in && (!cand || gt || (eq && eq_rank < take_eq));
    const int dst = carry_keep + block_prefix_count(keep, warp_tot, tot_keep);
    if (keep) {
      src[dst] = j;
      score[dst] = __uint_as_float(raw[j]);
      pos[dst] = posbuf[j];
      if (comp) comp[dst] = __uint_as_float(compbuf[j]);
    } else if (in) {
      atomicMin(&s_first, j);
    }
    carry_eq += tot_eq;
    carry_keep += tot_keep;
  }
  __syncthreads();
  if (tid == 0) {
    hdr[0] = s_first;      // rows below the first evicted one do not move
    hdr[1] = carry_keep;   // == tgt
    hdr[2] = n;
  }
}

// grid.x = 2 * column groups (even: K, odd: V), grid.y = slabs.
__global__ void __launch_bounds__(kCompactThreads) evict_compact_kernel(const EvictParams p) {
  const int slab = blockIdx.y;
  const int which = blockIdx.x & 1;
  const int cgp = blockIdx.x >> 1;
  const int tid = threadIdx.x;
  const int* hdr = p.hdr + (size_t)slab * 4;
  const int lo = hdr[0], hi = hdr[1];
  // One designated CTA per sequence publishes the new length (no CTA of this launch reads len).
  if (blockIdx.x == 0 && tid == 0 && slab < p.Nb * p.Hkv && slab % p.Hkv == 0) p.len[slab / p.Hkv] = hi;
  if (lo >= hi) return;

  const size_t row_bytes = (size_t)p.d * p.elt_bytes;
  const int pieces = (int)(row_bytes >> 4);
  const int piece = cgp * 4 + (tid & 3);
  const bool col_ok = piece < pieces;
  char* base = reinterpret_cast<char*>(which ? p.V : p.K) + (size_t)slab * p.cap * row_bytes + (size_t)piece * 16;
  const int* src = p.src + (size_t)slab * p.cap;

  for (int c0 = lo; c0 < hi; c0 += kCompactChunkRows) {
    uint4 buf[kCompactUnroll];
#pragma unroll
    for (int uu = 0; uu < kCompactUnroll; ++uu) {
      const int dst = c0 + uu * kCompactRowsPerPass + (tid >> 2);
      if (col_ok && dst < hi) buf[uu] = *reinterpret_cast<const uint4*>(base + (size_t)src[dst] * row_bytes);
    }
    __syncthreads();  // every source row of the chunk is in registers before any row is overwritten
#pragma unroll
    for (int uu = 0; uu < kCompactUnroll; ++uu) {
      const int dst = c0 + uu * kCompactRowsPerPass + (tid >> 2);
      if (col_ok && dst < hi) *reinterpret_cast<uint4*>(base + (size_t)dst * row_bytes) = buf[uu];
    }
    // The next chunk reads rows src[dst'] >= dst' >= c0 + chunk, disjoint from the rows just
    // written, so no second barrier is needed.
  }
}

// ---------------------------------------------------------------------------------------------
// Fused eviction: one CTA per slab selects the survivors (same integer-only rule as
// evict_select_kernel) and then moves the slab's K and V rows itself, so the gather list never
// leaves shared memory and one launch does the whole event.  The CTA walks the destination rows in
// ascending blocks of whole rows; per block every source row is loaded into registers before any
// destination row is stored, and since src[dst] >= dst with both increasing, a later block never
// reads a row an earlier block has overwritten.  The new lengths are published by the last CTA of
// the grid to finish (every CTA reads the old length before it takes its ticket).
// ---------------------------------------------------------------------------------------------
constexpr int kFusedThreads = 256;
constexpr int kFusedUnroll = 8;  // 16-byte loads in flight per thread and tensor (K and V: 16 in total)

// Exclusive prefix sum of one int per thread over the CTA (256 threads), plus the total.
__device__ __forceinline__ int block_exclusive_scan(int v, int* warp_tot /* [8] shared */, int& total) {
  const int lane = threadIdx.x & 31, warp = threadIdx.x >> 5;
  int incl = v;
#pragma unroll
  for (int o = 1; o < 32; o <<= 1) {
    const int t = __shfl_up_sync(0xffffffffu, incl, o);
    if (lane >= o) incl += t;
  }
  if (lane == 31) warp_tot[warp] = incl;
  __syncthreads();
  int before = 0, tot = 0;
#pragma unroll
  for (int w = 0; w < kFusedThreads / 32; ++w) {
    const int t = warp_tot[w];
    if (w < warp) before += t;
    tot += t;
  }
  __syncthreads();  // warp_tot may be reused right after
  total = tot;
  return before + incl - v;
}

__global__ void __launch_bounds__(kFusedThreads) evict_fused_kernel(const EvictParams p, unsigned int* ticket) {
  const int slab = blockIdx.x;
  const int b = (slab / p.Hkv) % p.Nb;
  const int tid = threadIdx.x;
  // Launched with programmatic stream serialisation: wait here for the kernel before this one.
  asm volatile("griddepcontrol.wait;" ::: "memory");
  if (p.pend != nullptr) {
    // a score pass of this slab that the last decode launch recorded instead of running it
    int* rec = p.pend + (size_t)slab * kStPendWords;
    const int rn = rec[0];
    if (rn > 0 && rn <= p.cap) {  // uniform over the CTA
      __shared__ float s_recM[8], s_recf[8];
      if (tid < 8) {
        s_recM[tid] = reinterpret_cast<const float*>(rec)[2 + tid];
        s_recf[tid] = reinterpret_cast<const float*>(rec)[10 + tid];
      }
      const int rn_old = rec[1];
      __syncthreads();
      DYNTS_DISPATCH_GROUP(p.G, score_pass_lean<GG>(p.score + (size_t)slab * p.cap, p.comp + (size_t)slab * p.cap,
                                                    p.logit_prev + (size_t)slab * p.G * p.cap, p.cap, rn, rn_old, s_recM,
                                                    s_recf, tid, kFusedThreads));
      __syncthreads();  // the updated scores are read back below
      if (tid == 0) rec[0] = 0;
    }
  }
  const int n = p.len[b];
  const int tgt = p.target[b];
  int* hdr = p.hdr + (size_t)slab * 4;

  extern __shared__ __align__(16) uint32_t esm[];
  uint32_t* raw = esm;                                            // [cap] score bit patterns
  int* posbuf = reinterpret_cast<int*>(esm + p.cap);              // [cap]
  uint32_t* compbuf = esm + 2 * (size_t)p.cap;                    // [cap]
  int* srcbuf = reinterpret_cast<int*>(esm + 3 * (size_t)p.cap);  // [cap] gather list: srcbuf[dst] = surviving row
  uint32_t* sel = p.key ? esm + 4 * (size_t)p.cap : raw;          // [cap] bit patterns the selection ranks by
  __shared__ unsigned int hist[256];
  __shared__ int warp_tot[kFusedThreads / 32];
  __shared__ uint32_t s_prefix;
  __shared__ int s_krem, s_first;

  if (n > tgt) {  // uniform over the CTA
    const int M = p.pinned[b];
    const int lo = M, hi = n - p.window;  // selection window [lo, hi)
    const int k = tgt - M - p.window;     // survivors wanted from it (host guarantees 0 <= k < hi - lo)
    float* score = p.score + (size_t)slab * p.cap;
    int* pos = p.pos + (size_t)slab * p.cap;
    float* comp = p.comp ? p.comp + (size_t)slab * p.cap : nullptr;
    for (int j = tid; j < n; j += kFusedThreads) {
      raw[j] = __float_as_uint(score[j]);
      posbuf[j] = pos[j];
      compbuf[j] = comp ? __float_as_uint(comp[j]) : 0u;
      if (p.key) sel[j] = __float_as_uint(p.key[(size_t)b * p.cap + j]);
    }
    if (tid == 0) {
      s_prefix = 0u;
      s_krem = k;
      s_first = n;
    }
    __syncthreads();

    // Radix select of the k-th largest key of the selection window (8 bits per pass).
    uint32_t mask = 0u;
    if (k > 0) {
      for (int shift = 24; shift >= 0; shift -= 8) {
        hist[tid] = 0u;
        __syncthreads();
        const uint32_t prefix = s_prefix;
        const int krem = s_krem;
        // Scores of one slab mostly share their top bits, so most rows fall into one bin: the lanes
        // of a warp that hit the same bin add their count with a single atomic.
        for (int base = lo; base < hi; base += kFusedThreads) {
          const int j = base + tid;
          uint32_t bin = 0x100u;  // "no vote"
          if (j < hi) {
            const uint32_t key = order_key(sel[j]);
            if ((key & mask) == prefix) bin = (key >> shift) & 255u;
          }
          const unsigned peers = __match_any_sync(0xffffffffu, bin);
          if (bin < 0x100u && (int)(threadIdx.x & 31) == __ffs(peers) - 1) atomicAdd(&hist[bin], (unsigned)__popc(peers));
        }
        __syncthreads();
        if (tid < 32) {
          unsigned int mine = 0;
          for (int i = 0; i < 8; ++i) mine += hist[255 - 8 * tid - i];
          unsigned int incl = mine;
          for (int o = 1; o < 32; o <<= 1) {
            const unsigned int v = __shfl_up_sync(0xffffffffu, incl, o);
            if (tid >= o) incl += v;
          }
          const unsigned int excl = incl - mine;
          if ((int)excl < krem && krem <= (int)incl) {
            unsigned int above = excl;
            for (int i = 0; i < 8; ++i) {
              const int bin = 255 - 8 * tid - i;
              const unsigned int c = hist[bin];
              if ((int)(above + c) >= krem) {
                s_prefix = prefix | ((uint32_t)bin << shift);
                s_krem = krem - (int)above;
                break;
              }
              above += c;
            }
          }
        }
        mask |= 0xFFu << shift;
        __syncthreads();
      }
    }
    const uint32_t T = s_prefix;   // key of the k-th largest candidate
    const int take_eq = s_krem;    // rows with key == T that survive (lowest indices first)

    // Every thread owns a contiguous run of rows; two CTA-wide prefix sums give the rank of each
    // row among the ties and its destination.
    int run = (n + kFusedThreads - 1) / kFusedThreads;
    run |= 1;  // odd stride: conflict-free shared-memory walks
    const int j0 = min(tid * run, n), j1 = min(j0 + run, n);
    int my_eq = 0;
    for (int j = j0; j < j1; ++j)
      if (k > 0 && j >= lo && j < hi && order_key(sel[j]) == T) ++my_eq;
    int tot;
    int eq_rank = block_exclusive_scan(my_eq, warp_tot, tot);
    int my_keep = 0;
    unsigned long long keepbits = 0ull;  // run <= 64 rows (the host limits the capacity)
    int first_gone = n;
    for (int j = j0; j < j1; ++j) {
      const bool cand = j >= lo && j < hi;
      bool keep = true;
      if (cand) {
        const uint32_t key = order_key(sel[j]);
        keep = k > 0 && (key > T || (key == T && eq_rank < take_eq));
        if (k > 0 && key == T) ++eq_rank;
      }
      if (keep) {
        keepbits |= 1ull << (j - j0);
        ++my_keep;
      } else {
        first_gone = min(first_gone, j);
      }
    }
    int dst = block_exclusive_scan(my_keep, warp_tot, tot);
    for (int j = j0; j < j1; ++j)
      if ((keepbits >> (j - j0)) & 1ull) srcbuf[dst++] = j;
    if (first_gone < n) atomicMin(&s_first, first_gone);
    __syncthreads();
    const int first = s_first, kept = tot;  // rows below `first` stay where they are; kept == tgt
    if (tid == 0) {
      hdr[0] = first;
      hdr[1] = kept;
      hdr[2] = n;
    }
    // score, pos, compensation of the moved rows (sources are in shared memory: in place is safe)
    for (int dd = first + tid; dd < kept; dd += kFusedThreads) {
      const int j = srcbuf[dd];
      score[dd] = __uint_as_float(raw[j]);
      pos[dd] = posbuf[j];
      if (comp) comp[dd] = __uint_as_float(compbuf[j]);
    }
    // K and V rows
    const int row_bytes = p.d * p.elt_bytes;
    const int pieces = row_bytes >> 4;
    const int rpp = kFusedThreads / pieces;  // rows per pass
    const bool active = tid < rpp * pieces;
    const int r_in = tid / pieces, piece = tid - r_in * pieces;
    char* Kb = reinterpret_cast<char*>(p.K) + (size_t)slab * p.cap * row_bytes + (size_t)piece * 16;
    char* Vb = reinterpret_cast<char*>(p.V) + (size_t)slab * p.cap * row_bytes + (size_t)piece * 16;
    for (int c0 = first; c0 < kept; c0 += rpp * kFusedUnroll) {
      uint4 kb[kFusedUnroll], vb[kFusedUnroll];
#pragma unroll
      for (int uu = 0; uu < kFusedUnroll; ++uu) {
        const int dd = c0 + uu * rpp + r_in;
        if (active && dd < kept) {
          const size_t so = (size_t)srcbuf[dd] * row_bytes;
          kb[uu] = *reinterpret_cast<const uint4*>(Kb + so);
          vb[uu] = *reinterpret_cast<const uint4*>(Vb + so);
        }
      }
      __syncthreads();  // every source row of the block is in registers before any row is overwritten
#pragma unroll
      for (int uu = 0; uu < kFusedUnroll; ++uu) {
        const int dd = c0 + uu * rpp + r_in;
        if (active && dd < kept) {
          *reinterpret_cast<uint4*>(Kb + (size_t)dd * row_bytes) = kb[uu];
          *reinterpret_cast<uint4*>(Vb + (size_t)dd * row_bytes) = vb[uu];
        }
      }
    }
  } else if (tid == 0) {
    hdr[0] = n;
    hdr[1] = n;
    hdr[2] = n;
  }

  // The last CTA to finish publishes the new lengths.
  __syncthreads();
  if (tid == 0) {
    __threadfence();
    const unsigned int t = atomicAdd(ticket, 1u);
    if (t == gridDim.x - 1) {
      *ticket = 0u;
      for (int bb = 0; bb < p.Nb; ++bb) p.len[bb] = min(p.len[bb], p.target[bb]);
      __threadfence();
    }
  }
}

// ---------------------------------------------------------------------------------------------
// Split eviction (slabs of up to 256 * RPT rows): a cluster of S CTAs per slab.  Every CTA of the
// cluster takes the slab's selection decision for itself and then moves its own share of the
// columns of the K and V rows (16-byte pieces [rank * 2P / S, (rank + 1) * 2P / S) of the 2P pieces
// of a K row followed by a V row).  Column shares are disjoint, so the CTAs of a slab never wait
// for one another while rows move, and a slab whose first evicted row lies far from its end no
// longer keeps one CTA busy long after the rest of the grid has finished.
//
// Everything a thread knows about its rows lives in registers: row i * 256 + tid is the thread's
// row i, with its score, its compensation term and (where the selection ranks by keys shared
// across the sequence) its key.  A score pass that the last decode launch left recorded is applied
// right there -- new score = old score + the row's normalised mass, from the logit scratch -- so
// the pass costs no round trip through memory before the scores can be ranked.
//
// Selection, integer-only as above:
//   - the candidates' smallest and largest key give a shift s with (key - smallest) >> s < 2048;
//     that monotone map spreads the rows over the 2048 bins of one histogram according to their
//     values, so a bin rarely holds more than a few rows.  Walking the bins from the top finds the
//     bin of the k-th largest key; the search ends there if the bin must be taken whole ("key >=
//     the bin's lower bound" decides), else it repeats inside the bin with s - 11 (at most three
//     rounds resolve all 32 bits);
//   - only if the threshold key itself is shared by more rows than may survive do ranks among the
//     ties (by index, from warp ballots and one scan of the per-warp counts) come into play;
//   - destinations are the exclusive prefix count of the survivor flags in index order.
// Score and compensation are written to their destinations from the registers, positions are
// gathered; each of the three arrays by one CTA of the cluster.  One cluster barrier separates
// every CTA's read of the old scores from their being overwritten.
// ---------------------------------------------------------------------------------------------
constexpr int kSplitThreads = 256;
constexpr int kSplitBins = 2048;
// 16-byte loads in flight per thread while rows move, and CTAs per SM: short slabs leave room for
// four CTAs of 64 registers; longer ones hold more rows per thread and run as two CTAs of 128.
__host__ __device__ constexpr int split_unroll(int rpt) { return rpt <= 5 ? 8 : 16; }
__host__ __device__ constexpr int split_ctas_per_sm(int rpt) { return rpt <= 5 ? 4 : 2; }

__device__ __forceinline__ uint32_t cluster_cta_rank() {
  uint32_t r;
  asm volatile("mov.u32 %0, %%cluster_ctarank;" : "=r"(r));
  return r;
}
__device__ __forceinline__ uint32_t cluster_cta_count() {
  uint32_t r;
  asm volatile("mov.u32 %0, %%cluster_nctarank;" : "=r"(r));
  return r;
}
__device__ __forceinline__ void cluster_arrive() { asm volatile("barrier.cluster.arrive.release.aligned;" ::: "memory"); }
__device__ __forceinline__ void cluster_wait() { asm volatile("barrier.cluster.wait.acquire.aligned;" ::: "memory"); }

// Per-warp counts of a per-row flag (bit i of `flags` belongs to row i * 256 + tid): cnt[i * 8 + warp].
template <int RPT>
__device__ __forceinline__ void rows_count(uint32_t flags, int* cnt, int warp, int lane) {
#pragma unroll
  for (int i = 0; i < RPT; ++i) {
    const unsigned bal = __ballot_sync(0xffffffffu, (flags >> i) & 1u);
    if (lane == 0) cnt[i * 8 + warp] = __popc(bal);
  }
}
// One warp turns cnt[0 .. RPT * 8) into its exclusive prefix sums (index order of the rows) and
// leaves the total in cnt[RPT * 8].
template <int RPT>
__device__ __forceinline__ void rows_scan(int* cnt, int lane) {
  constexpr int N = RPT * 8, E = (N + 31) / 32;
  int v[E], sum = 0;
#pragma unroll
  for (int e = 0; e < E; ++e) {
    const int idx = lane * E + e;
    v[e] = idx < N ? cnt[idx] : 0;
    sum += v[e];
  }
  int incl = sum;
#pragma unroll
  for (int o = 1; o < 32; o <<= 1) {
    const int t = __shfl_up_sync(0xffffffffu, incl, o);
    if (lane >= o) incl += t;
  }
  int run = incl - sum;
#pragma unroll
  for (int e = 0; e < E; ++e) {
    const int idx = lane * E + e;
    if (idx < N) cnt[idx] = run;
    run += v[e];
  }
  if (lane == 31) cnt[N] = incl;
}

// The recorded score pass of a slab (see DecodeParams::defer) on the rows this thread holds: the
// same arithmetic, in the same order, as score_pass_vec.  The logits and the record's maxima and
// normalisers are requested before anyone knows whether the record is valid (the addresses always
// are), so that they travel together with the scores; `valid` decides whether they are used.
template <int RPT, int GG>
__device__ __forceinline__ void recorded_pass_rows(float (&sc)[RPT], float (&cc)[RPT], const float* __restrict__ lg, int cap,
                                                   const int* rec, bool valid, int n, int n_old, int tid) {
  float M[GG], f[GG];
#pragma unroll
  for (int g = 0; g < GG; ++g) {
    M[g] = __ldcg(reinterpret_cast<const float*>(rec) + 2 + g);
    f[g] = __ldcg(reinterpret_cast<const float*>(rec) + 10 + g);
  }
#pragma unroll
  for (int i = 0; i < RPT; ++i) {
    const int j = i * kSplitThreads + tid;
    float e[GG];
#pragma unroll
    for (int g = 0; g < GG; ++g) e[g] = j < cap ? __ldcg(lg + (size_t)g * cap + j) : 0.f;
    float dl = 0.f;
#pragma unroll
    for (int g = 0; g < GG; ++g) dl += fast_exp2(e[g] - M[g]) * f[g];
    if (valid && j < n) {
      if (j == n_old) sc[i] = cc[i] = 0.f;  // the appended row starts from zero
      kahan_add(sc[i], cc[i], dl);
    }
  }
}

// SHARED_KEYS: the selection ranks by p.key (one key per token, shared by all slabs of a sequence)
// instead of the slab's own scores.
template <int RPT, bool SHARED_KEYS>
__global__ void __launch_bounds__(kSplitThreads, split_ctas_per_sm(RPT)) evict_split_kernel(const EvictParams p, unsigned int* ticket) {
  constexpr int kSplitUnroll = split_unroll(RPT);
  const uint32_t S = cluster_cta_count(), rank = cluster_cta_rank();
  const int slab = (int)(blockIdx.x / S);
  const int b = (slab / p.Hkv) % p.Nb;
  const int tid = threadIdx.x, lane = tid & 31, warp = tid >> 5;

  extern __shared__ __align__(16) int split_src[];  // [cap] gather list: split_src[dst] = surviving row
  __shared__ __align__(16) unsigned int hist[kSplitBins];
  __shared__ int s_cnt_eq[RPT * 8 + 1], s_cnt_keep[RPT * 8 + 1];
  __shared__ int s_wtot[kSplitThreads / 32];
  __shared__ uint32_t s_wmin[kSplitThreads / 32], s_wmax[kSplitThreads / 32];
  __shared__ uint32_t s_base;
  __shared__ int s_krem, s_bin_cnt;
  __shared__ int s_wfirst[kSplitThreads / 32];

  // nothing here touches global memory: it may overlap the tail of the kernel before this one
#pragma unroll
  for (int i = 0; i < kSplitBins / 4 / kSplitThreads; ++i)
    reinterpret_cast<uint4*>(hist)[i * kSplitThreads + tid] = make_uint4(0u, 0u, 0u, 0u);
  asm volatile("griddepcontrol.wait;" ::: "memory");  // launched with programmatic stream serialisation

  // One round trip: the lengths, the record of a score pass the last decode launch may have left,
  // and this thread's rows (score, compensation, position; the logits of the recorded pass).
  float* score = p.score + (size_t)slab * p.cap;
  float* comp = p.comp ? p.comp + (size_t)slab * p.cap : nullptr;
  int* pos = p.pos + (size_t)slab * p.cap;
  const bool have_rec = !SHARED_KEYS && p.pend != nullptr;
  const int* rec = have_rec ? p.pend + (size_t)slab * kStPendWords : nullptr;
  const int n = p.len[b];
  const int tgt = p.target[b];
  const int M = p.pinned[b];
  const int rn = have_rec ? rec[0] : 0, rn_old = have_rec ? rec[1] : 0;
  // Owners of the per-row arrays within the cluster.
  const bool own_score = rank == 0, own_comp = rank == (2u % S), own_pos = rank == (1u % S);
  float sc[RPT], cc[RPT];
  int posv[RPT];
#pragma unroll
  for (int i = 0; i < RPT; ++i) {
    const int j = i * kSplitThreads + tid;
    sc[i] = j < p.cap ? score[j] : 0.f;
    cc[i] = (j < p.cap && comp) ? comp[j] : 0.f;
    posv[i] = (j < p.cap && own_pos) ? pos[j] : 0;
  }
  int* hdr = p.hdr + (size_t)slab * 4;
  const bool fits = n <= p.cap && n <= RPT * kSplitThreads;
  if (!fits && tid == 0) atomicOr(p.err, kErrEvictSmem);  // (the host chooses RPT from the capacity)
  const bool evicting = fits && n > tgt;                        // uniform over the cluster
  bool applied = false;
  if constexpr (!SHARED_KEYS) {
    if (have_rec) {
      applied = fits && rn > 0 && rn == n;                      // uniform over the cluster
      DYNTS_DISPATCH_GROUP(p.G, (recorded_pass_rows<RPT, GG>(sc, cc, p.logit_prev + (size_t)slab * p.G * p.cap, p.cap, rec, applied, n,
                                                            rn_old, tid)));
      if (rn > 0 && !applied && tid == 0) atomicOr(p.err, kErrLenOverflow);  // a record that does not match the slab: the host mirror prevents it
    }
  }
  __syncthreads();  // hist, s_first

  if (evicting) {
    const int lo = M, hi = n - p.window;  // selection window [lo, hi)
    const int k = tgt - M - p.window;     // survivors wanted from it (host guarantees 0 <= k < hi - lo)

    // keys of the selection window
    uint32_t key[RPT];
    uint32_t candm = 0u;
    uint32_t tmin = 0xffffffffu, tmax = 0u;
#pragma unroll
    for (int i = 0; i < RPT; ++i) {
      const int j = i * kSplitThreads + tid;
      const bool cand = j >= lo && j < hi;
      uint32_t bits = __float_as_uint(sc[i]);
      if constexpr (SHARED_KEYS) bits = cand ? __float_as_uint(p.key[(size_t)b * p.cap + j]) : 0u;
      key[i] = cand ? order_key(bits) : 0u;
      candm |= (cand ? 1u : 0u) << i;
      if (cand) {
        tmin = min(tmin, key[i]);
        tmax = max(tmax, key[i]);
      }
    }
    cluster_arrive();  // this CTA has read the old scores (paired with the wait before any of them is overwritten)

    uint32_t T = 0u;
    int take_eq = 0;
    bool whole_bin = true;  // every row with key >= T survives (no tie is split)
    if (k > 0) {
      tmin = __reduce_min_sync(0xffffffffu, tmin);
      tmax = __reduce_max_sync(0xffffffffu, tmax);
      if (lane == 0) {
        s_wmin[warp] = tmin;
        s_wmax[warp] = tmax;
      }
      __syncthreads();
      uint32_t kmin = s_wmin[0], kmax = s_wmax[0];
#pragma unroll
      for (int w = 1; w < kSplitThreads / 32; ++w) {
        kmin = min(kmin, s_wmin[w]);
        kmax = max(kmax, s_wmax[w]);
      }
      // keys in [base, base + width): bin = (key - base) >> s, with width >> s <= 2048
      uint32_t base = kmin;
      int s = max(0, 32 - __clz(kmax - kmin) - 11);  // (kmax == kmin: clz = 32, s = 0, every row in bin 0)
      uint32_t width_m1 = kmax - kmin;                // width - 1 of the current interval
      int krem = k;
      whole_bin = false;
      for (int round = 0; round < 3; ++round) {  // s: <= 21, <= 10, 0
#pragma unroll
        for (int i = 0; i < RPT; ++i) {
          const uint32_t off = key[i] - base;
          if (((candm >> i) & 1u) && key[i] >= base && off <= width_m1) atomicAdd(&hist[off >> s], 1u);
        }
        __syncthreads();
        // thread t owns bins 2040 - 8t .. 2047 - 8t; walking t upwards walks the bins downwards
        const int hb = kSplitBins - 8 - 8 * tid;
        unsigned int hv[8];
        {
          const uint4 h0 = reinterpret_cast<const uint4*>(hist)[hb >> 2], h1 = reinterpret_cast<const uint4*>(hist)[(hb >> 2) + 1];
          hv[0] = h0.x; hv[1] = h0.y; hv[2] = h0.z; hv[3] = h0.w;
          hv[4] = h1.x; hv[5] = h1.y; hv[6] = h1.z; hv[7] = h1.w;
          reinterpret_cast<uint4*>(hist)[hb >> 2] = make_uint4(0u, 0u, 0u, 0u);  // clear for the next round
          reinterpret_cast<uint4*>(hist)[(hb >> 2) + 1] = make_uint4(0u, 0u, 0u, 0u);
        }
        const int mine = (int)(hv[0] + hv[1] + hv[2] + hv[3] + hv[4] + hv[5] + hv[6] + hv[7]);
        int incl = mine;
#pragma unroll
        for (int o = 1; o < 32; o <<= 1) {
          const int t = __shfl_up_sync(0xffffffffu, incl, o);
          if (lane >= o) incl += t;
        }
        if (lane == 31) s_wtot[warp] = incl;
        __syncthreads();
#pragma unroll
        for (int w = 0; w < kSplitThreads / 32; ++w)
          if (w < warp) incl += s_wtot[w];
        const int excl = incl - mine;
        if (excl < krem && krem <= incl) {  // exactly one thread: its bins hold the krem-th largest remaining key
          int above = excl;
#pragma unroll
          for (int i = 7; i >= 0; --i) {
            const int c = (int)hv[i];
            if (above < krem && krem <= above + c) {
              s_base = base + ((uint32_t)(hb + i) << s);
              s_krem = krem - above;
              s_bin_cnt = c;
            }
            above += c;
          }
        }
        __syncthreads();
        base = s_base;
        krem = s_krem;
        T = base;
        take_eq = krem;
        if (krem == s_bin_cnt) {  // the whole bin survives: nothing finer needs to be known
          whole_bin = true;
          break;
        }
        if (s == 0) break;        // the bin is one key value, shared by more rows than may survive
        width_m1 = (1u << s) - 1u;
        s = max(0, s - 11);
      }
    }

    // survivor flags
    uint32_t keepm = 0u;
    if (whole_bin) {
#pragma unroll
      for (int i = 0; i < RPT; ++i) {
        const int j = i * kSplitThreads + tid;
        const bool cand = (candm >> i) & 1u;
        const bool keep = cand ? (k > 0 && key[i] >= T) : (j < n);
        keepm |= (keep ? 1u : 0u) << i;
      }
    } else {
      // more rows share the threshold key than may survive: the lowest-indexed take_eq of them do
      uint32_t eqm = 0u;
#pragma unroll
      for (int i = 0; i < RPT; ++i) eqm |= ((((candm >> i) & 1u) && key[i] == T) ? 1u : 0u) << i;
      rows_count<RPT>(eqm, s_cnt_eq, warp, lane);
      __syncthreads();
      if (warp == 0) rows_scan<RPT>(s_cnt_eq, lane);
      __syncthreads();
#pragma unroll
      for (int i = 0; i < RPT; ++i) {
        const int j = i * kSplitThreads + tid;
        const bool cand = (candm >> i) & 1u;
        const bool eq = (eqm >> i) & 1u;
        const unsigned bal = __ballot_sync(0xffffffffu, eq);
        const int eq_rank = s_cnt_eq[i * 8 + warp] + __popc(bal & ((1u << lane) - 1u));
        const bool keep = cand ? (key[i] > T || (eq && eq_rank < take_eq)) : (j < n);
        keepm |= (keep ? 1u : 0u) << i;
      }
    }
    // destinations and the gather list
    rows_count<RPT>(keepm, s_cnt_keep, warp, lane);
    __syncthreads();
    if (warp == 0) rows_scan<RPT>(s_cnt_keep, lane);
    __syncthreads();
    int dstv[RPT];  // destination of this thread's surviving rows
    int wfirst = 0x7fffffff;  // first row of this warp's rows that leaves (the same value in every lane)
#pragma unroll
    for (int i = 0; i < RPT; ++i) {
      const int j = i * kSplitThreads + tid;
      const bool keep = (keepm >> i) & 1u;
      const unsigned bal = __ballot_sync(0xffffffffu, keep);
      dstv[i] = s_cnt_keep[i * 8 + warp] + __popc(bal & ((1u << lane) - 1u));
      if (keep) split_src[dstv[i]] = j;
      const unsigned gone = __ballot_sync(0xffffffffu, !keep && j < n);
      if (gone != 0u) wfirst = min(wfirst, i * kSplitThreads + warp * 32 + __ffs(gone) - 1);
    }
    if (lane == 0) s_wfirst[warp] = wfirst;
    __syncthreads();
    int first = s_wfirst[0];  // rows below `first` stay where they are
#pragma unroll
    for (int w = 1; w < kSplitThreads / 32; ++w) first = min(first, s_wfirst[w]);
    const int kept = s_cnt_keep[RPT * 8];  // == tgt
    if (rank == 0 && tid == 0) {
      hdr[0] = first;
      hdr[1] = kept;
      hdr[2] = n;
    }
    cluster_wait();  // every CTA of the cluster has read the old scores: they may be overwritten now
    if (applied && rank == S - 1 && (p.cap & 31) == 0) {
      // ... and the logits of the recorded pass, which are dead now: drop their L2 lines (32 rows of one
      // head each) instead of letting them be written back
      const float* lg = p.logit_prev + (size_t)slab * p.G * p.cap;
      const int lines = (n + 31) >> 5;
      for (int x = tid; x < p.G * lines; x += kSplitThreads) {
        const int g = x / lines, ln = x - g * lines;
        asm volatile("discard.global.L2 [%0], 128;" ::"l"(lg + (size_t)g * p.cap + 32 * ln) : "memory");
      }
    }
#pragma unroll
    for (int i = 0; i < RPT; ++i) {
      const bool keep = (keepm >> i) & 1u;
      const bool moved = keep && dstv[i] >= first;
      if (own_score && keep && (moved || applied)) score[dstv[i]] = sc[i];
      if (own_comp && comp && keep && (moved || applied)) comp[dstv[i]] = cc[i];
      if (own_pos && moved) pos[dstv[i]] = posv[i];
    }

    // K and V rows: this CTA's share of the 16-byte pieces of (K row | V row).  Ascending blocks; all
    // sources of a block are in registers before any destination of it is written (src >= dst).
    const int row_bytes = p.d * p.elt_bytes;
    const int P = row_bytes >> 4;               // pieces per row and tensor
    const int ppc = (2 * P) / (int)S;            // pieces per CTA and row (the host makes S divide 2P)
    const int rpp = kSplitThreads / ppc;         // rows per pass
    const bool active = tid < rpp * ppc;
    const int r_in = tid / ppc;
    const int q = (int)rank * ppc + (tid - r_in * ppc);
    const int isv = q >= P ? 1 : 0;
    char* kvbase = reinterpret_cast<char*>(isv ? p.V : p.K) + (size_t)slab * p.cap * row_bytes + (size_t)(q - isv * P) * 16;
    for (int c0 = first; c0 < kept; c0 += rpp * kSplitUnroll) {
      uint4 buf[kSplitUnroll];
#pragma unroll
      for (int uu = 0; uu < kSplitUnroll; ++uu) {
        const int dd = c0 + uu * rpp + r_in;
        if (active && dd < kept) buf[uu] = *reinterpret_cast<const uint4*>(kvbase + (size_t)split_src[dd] * row_bytes);
      }
      __syncthreads();  // every source row of the block is in registers before any row is overwritten
#pragma unroll
      for (int uu = 0; uu < kSplitUnroll; ++uu) {
        const int dd = c0 + uu * rpp + r_in;
        if (active && dd < kept) *reinterpret_cast<uint4*>(kvbase + (size_t)dd * row_bytes) = buf[uu];
      }
    }
  } else {
    if (rank == 0 && tid == 0) {
      hdr[0] = n;
      hdr[1] = n;
      hdr[2] = n;
    }
    if (applied) {  // no row leaves, but the recorded pass has changed the scores (this launch's CTAs are the only readers)
#pragma unroll
      for (int i = 0; i < RPT; ++i) {
        const int j = i * kSplitThreads + tid;
        if (j < n && own_score) score[j] = sc[i];
        if (j < n && own_comp && comp) comp[j] = cc[i];
      }
    }
  }
  if (applied && rank == 0 && tid == 0) p.pend[(size_t)slab * kStPendWords] = 0;

  // The last CTA to finish publishes the new lengths.
  __syncthreads();
  if (tid == 0) {
    __threadfence();
    const unsigned int t = atomicAdd(ticket, 1u);
    if (t == gridDim.x - 1) {
      *ticket = 0u;
      for (int bb = 0; bb < p.Nb; ++bb) p.len[bb] = min(p.len[bb], p.target[bb]);
      __threadfence();
    }
  }
}

// ---------------------------------------------------------------------------------------------
// One importance score per token, aggregated across all layers and KV heads (Appendix B.1):
// agg[b][j] = sum over (layer, head) of score[layer][b][head][j].  The fp32 slab scores are added
// in double precision and the sum is rounded to fp32 once, so the key a ranking is decided by is
// within half an ulp of the exact sum whatever the number of slabs.  grid = (row blocks, sequences).
// ---------------------------------------------------------------------------------------------
__global__ void __launch_bounds__(256) aggregate_scores_kernel(const float* score, float* agg, const int* len,
                                                               const int* active, int L, int Nb, int Hkv, int cap) {
  const int b = blockIdx.y;
  const int j = blockIdx.x * blockDim.x + threadIdx.x;
  if (!active[b] || j >= len[b] || j >= cap) return;
  double acc = 0.0;
  for (int l = 0; l < L; ++l)
    for (int h = 0; h < Hkv; ++h) acc += (double)score[(((size_t)l * Nb + b) * Hkv + h) * cap + j];
  agg[(size_t)b * cap + j] = (float)acc;
}

// ---------------------------------------------------------------------------------------------
// Predictor scores (Section 4.1, Eq. 7; Section 4.2: a new token's score is appended beside its
// KV): the row appended by the latest decode step gets s_new[b] in every slab of sequence b.
// ---------------------------------------------------------------------------------------------
__global__ void __launch_bounds__(256) append_scores_kernel(float* score, float* comp, const int* len, const int* active,
                                                            const float* s_new, int n_slabs, int Nb, int Hkv, int cap) {
  const int slab = blockIdx.x * blockDim.x + threadIdx.x;
  if (slab >= n_slabs) return;
  const int b = (slab / Hkv) % Nb;
  const int n = len[b];
  if (!active[b] || n < 1 || n > cap) return;
  score[(size_t)slab * cap + n - 1] = s_new[b];
  comp[(size_t)slab * cap + n - 1] = 0.f;
}

// ---------------------------------------------------------------------------------------------
// Prompt load (question window, Section 4.2).  grid.x = row blocks, grid.y = slabs touched.
// ---------------------------------------------------------------------------------------------
struct PrefillParams {
  const void* k;   // [L, Nb, Hkv, T, d] (seq < 0) or [L, Hkv, T, d] (one sequence)
  const void* v;
  void* K;
  void* V;
  int* pos;
  float* score;
  float* comp;
  int* len;
  int* tot;
  int* pinned;
  int* active;
  int L, Nb, Hkv, d, cap, elt_bytes, T, n_pinned, seq;
  int layer0;              // the source tensors hold the layers layer0 .. (as many as the grid covers)
  int set_len;             // 1: this launch also publishes length, position counter, pins and the active flag
  int kv8;                 // 1: k, v are bf16 and the slabs take their E4M3 codes (elt_bytes = 1)
  float k_scale, v_scale;
};

__global__ void __launch_bounds__(256) prefill_kernel(const PrefillParams p) {
  const int sl = blockIdx.y;  // index over the slabs of the source tensor
  int l, b, h;
  if (p.seq < 0) {
    h = sl % p.Hkv;
    b = (sl / p.Hkv) % p.Nb;
    l = p.layer0 + sl / (p.Hkv * p.Nb);
  } else {
    h = sl % p.Hkv;
    l = p.layer0 + sl / p.Hkv;
    b = p.seq;
  }
  const size_t slab = ((size_t)l * p.Nb + b) * p.Hkv + h;
  const size_t row_bytes = (size_t)p.d * p.elt_bytes;
  char* Kd = reinterpret_cast<char*>(p.K) + slab * p.cap * row_bytes;
  char* Vd = reinterpret_cast<char*>(p.V) + slab * p.cap * row_bytes;
  if (p.kv8) {
    // 8 bf16 elements (16 bytes) in, 8 codes out per thread and step; rows are contiguous on both sides
    const __nv_bfloat16* ks = reinterpret_cast<const __nv_bfloat16*>(p.k) + (size_t)sl * p.T * p.d;
    const __nv_bfloat16* vs = reinterpret_cast<const __nv_bfloat16*>(p.v) + (size_t)sl * p.T * p.d;
    const size_t total = (size_t)p.T * p.d / 8;
    for (size_t e = (size_t)blockIdx.x * blockDim.x + threadIdx.x; e < total; e += (size_t)gridDim.x * blockDim.x) {
      const uint4 kin = reinterpret_cast<const uint4*>(ks)[e], vin = reinterpret_cast<const uint4*>(vs)[e];
      const __nv_bfloat16* kb = reinterpret_cast<const __nv_bfloat16*>(&kin);
      const __nv_bfloat16* vb = reinterpret_cast<const __nv_bfloat16*>(&vin);
      uint32_t ko[2] = {0u, 0u}, vo[2] = {0u, 0u};
#pragma unroll
      for (int i = 0; i < 8; ++i) {
        ko[i >> 2] |= (uint32_t)store_e4m3(__bfloat162float(kb[i]), p.k_scale) << (8 * (i & 3));
        vo[i >> 2] |= (uint32_t)store_e4m3(__bfloat162float(vb[i]), p.v_scale) << (8 * (i & 3));
      }
      reinterpret_cast<uint2*>(Kd)[e] = make_uint2(ko[0], ko[1]);
      reinterpret_cast<uint2*>(Vd)[e] = make_uint2(vo[0], vo[1]);
    }
  } else {
    const int pieces = (int)(row_bytes >> 4);
    const char* ks = reinterpret_cast<const char*>(p.k) + (size_t)sl * p.T * row_bytes;
    const char* vs = reinterpret_cast<const char*>(p.v) + (size_t)sl * p.T * row_bytes;
    const size_t total = (size_t)p.T * pieces;
    for (size_t e = (size_t)blockIdx.x * blockDim.x + threadIdx.x; e < total; e += (size_t)gridDim.x * blockDim.x) {
      reinterpret_cast<uint4*>(Kd)[e] = reinterpret_cast<const uint4*>(ks)[e];
      reinterpret_cast<uint4*>(Vd)[e] = reinterpret_cast<const uint4*>(vs)[e];
    }
  }
  for (int t = blockIdx.x * blockDim.x + threadIdx.x; t < p.T; t += gridDim.x * blockDim.x) {
    p.pos[slab * p.cap + t] = t;
    p.score[slab * p.cap + t] = t < p.n_pinned ? __int_as_float(0x7f800000) : 0.f;
    p.comp[slab * p.cap + t] = 0.f;
  }
  if (p.set_len && blockIdx.x == 0 && threadIdx.x == 0 && l == p.layer0 && h == 0) {
    p.len[b] = p.T;
    p.tot[b] = p.T;
    p.pinned[b] = p.n_pinned;
    p.active[b] = 1;
  }
}

}  // namespace dynts

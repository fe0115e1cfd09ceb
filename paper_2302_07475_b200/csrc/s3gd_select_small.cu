// Selection of a row whose filtered candidates fit one SM's shared memory: one CTA per
// row lays the candidates out in index order on chip, then does the three radix passes
// and the ordered emission as flat sweeps over that array without leaving the chip, so the chain of dependent global round trips that
// a sequence of small launches pays per pass is paid once.
//
// Same arithmetic as the general passes in s3gd_select.cu: MSB-first radix select on the
// 31 magnitude bits (11 + 10 + 10), then index-ordered emission tile by tile with the
// lowest-index rule for entries equal to the K-th magnitude (Eq. (3)-(4) plus the tie
// reading).  Rows it cannot take (no valid candidate list, or too many candidates) are
// left untouched for the general passes; rows it finishes are marked done.
#include <cooperative_groups.h>

#include "s3gd_common.cuh"

namespace s3gd {
namespace {

constexpr int kSmallThreads = 1024;
constexpr int kSmallWarps = kSmallThreads / 32;
static_assert(kSmallWarps == 32, "the block scan below folds 32 warp totals in one warp");

__device__ __forceinline__ uint32_t block_scan_excl_1024(uint32_t v, uint32_t* s_warp, uint32_t* total) {
  const uint32_t lane = threadIdx.x & 31, warp = threadIdx.x >> 5;
  uint32_t inc = v;
#pragma unroll
  for (int s = 1; s < 32; s <<= 1) {
    const uint32_t o = __shfl_up_sync(0xFFFFFFFFu, inc, s);
    if (lane >= (uint32_t)s) inc += o;
  }
  __syncthreads();                               // earlier readers of s_warp are done
  if (lane == 31) s_warp[warp] = inc;
  __syncthreads();
  const uint32_t mine = s_warp[lane];            // 32 warp totals, one per lane
  uint32_t winc = mine;
#pragma unroll
  for (int s = 1; s < 32; s <<= 1) {
    const uint32_t o = __shfl_up_sync(0xFFFFFFFFu, winc, s);
    if (lane >= (uint32_t)s) winc += o;
  }
  *total = __shfl_sync(0xFFFFFFFFu, winc, 31);
  const uint32_t woff = __shfl_sync(0xFFFFFFFFu, winc - mine, warp);
  return woff + inc - v;
}


// ---- a bin list too long for shared memory (votes only, band form of the filter pass): the same
// decisions taken over the list where it lies, in L2 / device memory, by the row's one CTA.  The
// entries share their upper 21 magnitude bits; one sweep counts the low 10, and if the entries
// equal to the K-th magnitude are not all kept, three more sweeps find the index up to which they
// are (a radix select on the index: the lowest indices win).  A last sweep lets the kept ones vote.
// Rare for smooth data (a bin is 1024 keys wide); the rule for coarsely quantised gradients with
// tens of thousands of equal magnitudes at the threshold.
__device__ __forceinline__ void warp_hist_add(uint32_t* s_hist, bool on, uint32_t digit) {
  const uint32_t act = __ballot_sync(0xFFFFFFFFu, on);
  if (act == 0u) return;                             // warp-uniform
  const uint32_t lead = (uint32_t)__ffs((int)act) - 1u;
  const uint32_t d0 = __shfl_sync(0xFFFFFFFFu, digit, lead);
  if (__all_sync(0xFFFFFFFFu, !on || digit == d0)) {   // equal magnitudes: one add for the warp
    if ((threadIdx.x & 31u) == lead) atomicAdd(&s_hist[d0], (uint32_t)__popc(act));
  } else if (on) {
    atomicAdd(&s_hist[digit], 1u);
  }
}

// The bin among `nbins` (a power of two, at most 2048) that holds the want-th entry counted from the
// top (descending) or from the bottom; *before = entries in the bins passed on the way.  Block-wide.
__device__ __forceinline__ uint32_t pick_bin_1024(const uint32_t* s_hist, int nbins, bool from_top, uint32_t want,
                                                  uint32_t* before, uint32_t* s_warp, uint32_t* s_sel) {
  const uint32_t tid = threadIdx.x;
  const int per = nbins > kSmallThreads ? nbins / kSmallThreads : 1;
  uint32_t mine = 0, cbin[2] = {0u, 0u};
  if ((int)tid * per < nbins) {
#pragma unroll
    for (int i = 0; i < 2; ++i)
      if (i < per) {
        const int pos = (int)tid * per + i;
        cbin[i] = s_hist[from_top ? nbins - 1 - pos : pos];
        mine += cbin[i];
      }
  }
  uint32_t total;
  const uint32_t earlier = block_scan_excl_1024(mine, s_warp, &total);
  if (tid == 0) s_sel[0] = 0xFFFFFFFFu;
  __syncthreads();
  if (earlier < want && earlier + mine >= want) {              // exactly one thread
    uint32_t a = earlier;
#pragma unroll
    for (int i = 0; i < 2; ++i) {
      if (i < per) {
        if (a + cbin[i] >= want) {
          const int pos = (int)tid * per + i;
          s_sel[0] = (uint32_t)(from_top ? nbins - 1 - pos : pos);
          s_sel[1] = a;
          break;
        }
        a += cbin[i];
      }
    }
  }
  __syncthreads();
  *before = s_sel[1];
  return s_sel[0];                                             // 0xFFFFFFFF: fewer than `want` entries
}

__device__ __forceinline__ void select_bin_in_place(RowState* __restrict__ rows, uint32_t row, const RowState& rs,
                                                    const uint2* __restrict__ c, uint32_t n, uint32_t* __restrict__ hdr,
                                                    const EmitOut& o, uint32_t* s_hist, uint32_t* s_warp,
                                                    uint32_t* s_sel, bool overflowed) {
  const uint32_t tid = threadIdx.x;
  constexpr int kLoads = 4;                                    // list entries a thread has in flight
  const uint32_t k_want = rs.k_rem;
  bool bad = overflowed;
  // ---- low 10 bits of the magnitude
  for (int b = tid; b < 1024; b += kSmallThreads) s_hist[b] = 0u;
  __syncthreads();
  for (uint32_t base = 0; base < n; base += kSmallThreads * kLoads) {
    uint32_t key[kLoads];
    bool on[kLoads];
#pragma unroll
    for (int u = 0; u < kLoads; ++u) {
      const uint32_t i = base + u * kSmallThreads + tid;
      on[u] = i < n;
      key[u] = on[u] ? (c[i].x & kAbsMask) : 0u;
    }
#pragma unroll
    for (int u = 0; u < kLoads; ++u) warp_hist_add(s_hist, on[u], key[u] & 1023u);
  }
  __syncthreads();
  uint32_t above = 0;
  uint32_t digit = pick_bin_1024(s_hist, 1024, true, k_want, &above, s_warp, s_sel);
  if (digit == 0xFFFFFFFFu) { bad = true; digit = 0u; above = 0u; }     // cannot happen for a valid row
  const uint32_t tau = (rs.prefix << pass_bits(kNumPasses - 1)) | digit, take = k_want - above;
  const uint32_t n_equal = s_hist[digit];
  __syncthreads();
  // ---- entries equal to tau: all kept, or those with the `take` lowest indices
  uint32_t idx_limit = 0xFFFFFFFFu;
  if (n_equal > take) {
    uint32_t iprefix = 0, t_rem = take;
#pragma unroll 1
    for (int pass = 0; pass < 3; ++pass) {
      const int shift = pass == 0 ? 21 : (pass == 1 ? 10 : 0);
      const int prev_shift = pass == 1 ? 21 : 10;
      const int nbins = pass == 2 ? 1024 : 2048;
      const uint32_t mask = (uint32_t)(nbins - 1);
      for (int b = tid; b < nbins; b += kSmallThreads) s_hist[b] = 0u;
      __syncthreads();
      for (uint32_t base = 0; base < n; base += kSmallThreads * kLoads) {
        uint2 e[kLoads];
#pragma unroll
        for (int u = 0; u < kLoads; ++u) {
          const uint32_t i = base + u * kSmallThreads + tid;
          e[u] = i < n ? c[i] : make_uint2(0u, 0u);
        }
#pragma unroll
        for (int u = 0; u < kLoads; ++u) {
          const bool in = base + u * kSmallThreads + tid < n;
          if (in && (e[u].x & kAbsMask) == tau && (pass == 0 || (e[u].y >> prev_shift) == iprefix))
            atomicAdd(&s_hist[(e[u].y >> shift) & mask], 1u);
        }
      }
      __syncthreads();
      uint32_t a = 0;
      uint32_t idigit = pick_bin_1024(s_hist, nbins, false, t_rem, &a, s_warp, s_sel);
      if (idigit == 0xFFFFFFFFu) { bad = true; idigit = 0u; a = 0u; }   // cannot happen: take <= n_equal
      t_rem -= a;
      iprefix = (iprefix << (pass == 2 ? 10 : 11)) | idigit;
      __syncthreads();
    }
    idx_limit = iprefix;
  }
  // ---- votes
  for (uint32_t base = 0; base < n; base += kSmallThreads * kLoads) {
    uint2 e[kLoads];
#pragma unroll
    for (int u = 0; u < kLoads; ++u) {
      const uint32_t i = base + u * kSmallThreads + tid;
      e[u] = i < n ? c[i] : make_uint2(0u, 0u);
    }
#pragma unroll
    for (int u = 0; u < kLoads; ++u) {
      const uint32_t key = e[u].x & kAbsMask;
      if (base + u * kSmallThreads + tid < n && (key > tau || (key == tau && e[u].y <= idx_limit)))
        add_vote(o.counter, o.packed, e[u].y, e[u].x >> 31);
    }
  }
  if (tid == 0) {
    rows[row].tau = tau;
    rows[row].take_ties = take;
    rows[row].n_emitted = bad ? 0xFFFFFFFFu : o.K;
    if (bad) {
      atomicAdd(hdr + kHdrBadCount, 1u);
      atomicOr(hdr + kHdrStatus, (uint32_t)kFlagInternal);
    }
    atomicMax(hdr + kHdrMaxCand, rs.n_cand);
  }
}

// kOrdered: the message (indices, sign bits) is wanted, so the candidates are laid out in index
// order and emitted with their output positions.  Otherwise only the votes are wanted, whose
// order does not matter: the candidates are copied as they lie, every entry above tau votes at
// once, and only the entries equal to tau are ranked by index among themselves: pairwise up to
// kMaxTiesUnordered of them, beyond that by a radix select on the index.
constexpr uint32_t kMaxTiesUnordered = 1024;

// kBin (votes only): the list is the row's bin list of the two-pass form (s3gd_select.cu) instead of
// its candidates -- the entries that share the upper 21 bits of the K-th magnitude -- of which the
// k_rem largest are kept; everything above them has voted already and the row is counted as finished.
template <bool kOrdered, bool kBin = false>
__global__ void __launch_bounds__(kSmallThreads, 1)
select_small_kernel(RowState* __restrict__ rows, const uint2* __restrict__ cand, uint32_t cap,
                    const uint2* __restrict__ seg, uint32_t n_tiles, uint32_t* __restrict__ hdr, EmitOut o) {
  static_assert(!(kOrdered && kBin), "bin lists are unordered");
  extern __shared__ __align__(16) unsigned char smem_raw[];
  __shared__ uint32_t s_hist[kHistBins];
  __shared__ uint32_t s_warp[kSmallWarps];
  __shared__ uint32_t s_sel[2];
  __shared__ uint32_t s_first[kOrdered ? kSmallThreads : 1];   // first chunk of each tile of a layout round
  const uint32_t row = blockIdx.x, tid = threadIdx.x, lane = tid & 31, lt = lanemask_lt();
  grid_dependency_wait();                            // (launched with launch_after)
  const RowState rs = rows[row];
  if (kBin ? rs.done != kRowBin : !row_uses_candidates(rs, o.K, cap)) return;
  if (!kBin && !fits_single_cta(rs.n_cand)) {
    // An unordered list (band form of the filter pass) cannot go through the general passes, which
    // count and emit in index order: such a row is redone over the whole row.
    if (o.unordered && tid == 0) rows[row].exact = 1u;
    return;
  }
  const uint32_t n = kBin ? (rs.n_bin < cap ? rs.n_bin : cap) : rs.n_cand;
  if (kBin && !fits_single_cta(n)) {                 // longer than this CTA's shared memory: select it where it lies
    select_bin_in_place(rows, row, rs, cand + (uint64_t)row * cap, n, hdr, o, s_hist, s_warp, s_sel, rs.n_bin > cap);
    return;
  }
  // entries to keep out of the n (whatever voted during the filter pass is no longer looked for; n_hi is 0
  // unless that pass took its band form)
  const uint32_t k_want = kBin ? rs.k_rem : o.K - rs.n_hi;
  uint32_t* s_bits = reinterpret_cast<uint32_t*>(smem_raw);   // [n] bit patterns, in ascending index order
  uint32_t* s_idx = s_bits + n;                               // [n] their indices
  const uint2* c = cand + (uint64_t)row * cap;

  if (!kOrdered) {
#pragma unroll 8
    for (uint32_t i = tid; i < n; i += kSmallThreads) {
      const uint2 e = c[i];
      s_bits[i] = e.x;
      s_idx[i] = e.y;
    }
  } else {
    // ---- bring the candidates on chip in index order: the filter stored them tile by tile, each
    // tile's segment wherever its claim landed; laying the segments out in tile order sorts them.
    // 1024 tiles per round (one per thread for the bookkeeping).  The round's segments are cut into
    // chunks of up to 32 entries -- a tile with c entries has ceil(c / 32), an empty one none -- and the
    // chunks are dealt to the warps in turn, eight chunks' loads in flight per warp before the first
    // store: gradients with layer-wise scales put hundreds of candidates into the tiles of a few layers
    // and none into most, and a division by tiles left most warps waiting for a few.
    {
      static_assert(kHistBins >= 2 * kSmallThreads, "two tables of the layout live in the histogram's words");
      uint32_t* s_src = s_hist;                      // (the histogram is not in use yet)
      uint32_t* s_dst = s_hist + kSmallThreads;
      const uint32_t warp = tid >> 5;
      uint32_t carry = 0;
      for (uint32_t base = 0; base < n_tiles; base += kSmallThreads) {
        const uint32_t t = base + tid;
        const uint2 sg = t < n_tiles ? seg[(uint64_t)row * n_tiles + t] : make_uint2(0u, 0u);
        uint32_t total, total_chunks;
        const uint32_t dst = carry + block_scan_excl_1024(sg.y, s_warp, &total);
        const uint32_t first_chunk = block_scan_excl_1024((sg.y + 31u) >> 5, s_warp, &total_chunks);
        const uint32_t end = carry + total;          // where the round's last segment ends
        carry = end;
        s_src[tid] = sg.x;
        s_dst[tid] = dst;
        s_first[tid] = first_chunk;
        __syncthreads();
        // a warp takes 32 chunks at a time, one per lane for the lookup: the chunk's tile is the last one whose
        // first chunk is <= k (first_chunk does not decrease; an empty tile shares its value with the next one)
        constexpr int kBatch = 8;
#pragma unroll 1
        for (uint32_t k0 = warp * 32u; k0 < total_chunks; k0 += kSmallWarps * 32u) {   // warp-uniform
          const uint32_t k = k0 + lane;
          uint32_t my_d0 = 0, my_cnt = 0, my_src = 0, my_off = 0;
          if (k < total_chunks) {
            uint32_t lo = 0, len = kSmallThreads;        // invariant: s_first[lo] <= k
#pragma unroll
            for (int it = 0; it < 10; ++it) {
              len >>= 1;
              if (s_first[lo + len] <= k) lo += len;
            }
            my_d0 = s_dst[lo];
            my_cnt = (lo + 1u < (uint32_t)kSmallThreads ? s_dst[lo + 1u] : end) - my_d0;
            my_src = s_src[lo];
            my_off = (k - s_first[lo]) * 32u;
          }
          const uint32_t n_here = total_chunks - k0 < 32u ? total_chunks - k0 : 32u;
#pragma unroll 1
          for (uint32_t j0 = 0; j0 < n_here; j0 += kBatch) {
            uint2 e[kBatch];
            uint32_t at[kBatch];
#pragma unroll
            for (int j = 0; j < kBatch; ++j) {
              const uint32_t jj = j0 + j;                  // (a lane beyond n_here holds zeros: nothing to copy)
              const uint32_t d0 = __shfl_sync(0xFFFFFFFFu, my_d0, jj & 31u), cnt = __shfl_sync(0xFFFFFFFFu, my_cnt, jj & 31u);
              const uint32_t src = __shfl_sync(0xFFFFFFFFu, my_src, jj & 31u);
              const uint32_t i = __shfl_sync(0xFFFFFFFFu, my_off, jj & 31u) + lane;
              at[j] = 0xFFFFFFFFu;
              if (jj < n_here && i < cnt) {
                at[j] = d0 + i;
                e[j] = c[src + i];
              }
            }
#pragma unroll
            for (int j = 0; j < kBatch; ++j)
              if (at[j] != 0xFFFFFFFFu) { s_bits[at[j]] = e[j].x; s_idx[at[j]] = e[j].y; }
          }
        }
        __syncthreads();                             // the three tables are rewritten by the next round
      }
    }
  }

  // ---- radix select: tau = K-th largest magnitude, take = how many entries equal to tau are kept
  // (the entries of a bin list share their upper 21 bits, which the first sweep fixed: last pass only)
  uint32_t prefix = kBin ? rs.prefix : 0u, k_rem = k_want, n_equal = 0;
  for (int pass = kBin ? kNumPasses - 1 : 0; pass < kNumPasses; ++pass) {
    const int nbins = 1 << pass_bits(pass);
    const uint32_t mask = (uint32_t)(nbins - 1);
    for (int b = tid; b < nbins; b += kSmallThreads) s_hist[b] = 0u;
    __syncthreads();                             // also: the candidate arrays are complete (first pass)
    if (pass == 0) {
      // Every candidate is >= tau_lo, and most sit within a few leading-digit values of it
      // (gradient magnitudes fall off fast).  Warp-wide votes and shuffles are scarce on one
      // SM, so each thread counts the first eight values above tau_lo's in registers over
      // all its entries; one warp reduction per value at the end.  The rest: plain atomics.
      const uint32_t d_lo = (rs.tau_lo >> pass_shift(0)) & mask;
      uint32_t cnt8[8] = {0u, 0u, 0u, 0u, 0u, 0u, 0u, 0u};
      for (uint32_t i = tid; i < n; i += kSmallThreads) {
        const uint32_t digit = ((s_bits[i] & kAbsMask) >> pass_shift(0)) & mask;
        const uint32_t rel = digit - d_lo;                      // >= 0 for every candidate
#pragma unroll
        for (uint32_t b = 0; b < 8; ++b) cnt8[b] += (uint32_t)(rel == b);
        if (rel >= 8u) atomicAdd(&s_hist[digit], 1u);
      }
#pragma unroll
      for (uint32_t b = 0; b < 8; ++b) {
        const uint32_t v = __reduce_add_sync(0xFFFFFFFFu, cnt8[b]);
        if (lane == b && v != 0u) atomicAdd(&s_hist[(d_lo + b) & mask], v);
      }
    } else {
      // later digits are spread out: plain shared-memory atomics of the few entries still in play
      for (uint32_t i = tid; i < n; i += kSmallThreads) {
        const uint32_t key = s_bits[i] & kAbsMask;
        if ((key >> pass_shift(pass - 1)) == prefix) atomicAdd(&s_hist[(key >> pass_shift(pass)) & mask], 1u);
      }
    }
    __syncthreads();
    // thread t owns bins [t*per, t*per+per) counted from the TOP (descending magnitude)
    const int per = nbins > kSmallThreads ? nbins / kSmallThreads : 1;
    uint32_t mine = 0;
    uint32_t cbin[2] = {0u, 0u};
    if ((int)tid * per < nbins) {
#pragma unroll
      for (int i = 0; i < 2; ++i)
        if (i < per) { cbin[i] = s_hist[nbins - 1 - ((int)tid * per + i)]; mine += cbin[i]; }
    }
    uint32_t total;
    const uint32_t above = block_scan_excl_1024(mine, s_warp, &total);   // entries in higher bins
    if (tid == 0) s_sel[0] = 0xFFFFFFFFu;
    __syncthreads();
    if (above < k_rem && above + mine >= k_rem) {        // exactly one thread
      uint32_t a = above;
#pragma unroll
      for (int i = 0; i < 2; ++i) {
        if (i < per) {
          if (a + cbin[i] >= k_rem) { s_sel[0] = (uint32_t)(nbins - 1 - ((int)tid * per + i)); s_sel[1] = a; break; }
          a += cbin[i];
        }
      }
    }
    __syncthreads();
    uint32_t digit = s_sel[0], a = s_sel[1];
    n_equal = digit == 0xFFFFFFFFu ? 0u : s_hist[digit];        // after the last pass: entries equal to tau
    if (digit == 0xFFFFFFFFu) {                          // fewer than k_rem entries: cannot happen for a valid row
      if (tid == 0) atomicOr(hdr + kHdrStatus, (uint32_t)kFlagInternal);
      digit = 0u; a = 0u;
    }
    prefix = (prefix << pass_bits(pass)) | digit;
    k_rem -= a;
    __syncthreads();                             // s_sel and s_hist are reused by the next pass
  }
  const uint32_t tau = prefix, take = k_rem;

  if (!kOrdered) {
    // ---- votes only.  Entries equal to tau are few as a rule; they are kept by ascending index
    // until `take` are taken, which needs their rank among themselves only.
    bool rank_ties = n_equal > take;                             // otherwise every one of them is kept
    uint32_t idx_limit = 0xFFFFFFFFu;                            // entries equal to tau are kept up to this index
    if (rank_ties && n_equal > kMaxTiesUnordered) {
      // Too many to rank pairwise: a second radix select, on the index, finds the take-th smallest
      // index among the entries equal to tau (indices are distinct, so exactly `take` lie at or below it).
      uint32_t iprefix = 0, t_rem = take;
#pragma unroll 1
      for (int pass = 0; pass < 3; ++pass) {
        const int shift = pass == 0 ? 21 : (pass == 1 ? 10 : 0);
        const int prev_shift = pass == 1 ? 21 : 10;
        const int nbins = pass == 2 ? 1024 : 2048;
        const uint32_t mask = (uint32_t)(nbins - 1);
        for (int b = tid; b < nbins; b += kSmallThreads) s_hist[b] = 0u;
        __syncthreads();
        for (uint32_t i = tid; i < n; i += kSmallThreads) {
          if ((s_bits[i] & kAbsMask) != tau) continue;
          const uint32_t idx = s_idx[i];
          if (pass == 0 || (idx >> prev_shift) == iprefix) atomicAdd(&s_hist[(idx >> shift) & mask], 1u);
        }
        __syncthreads();
        const int per = nbins / kSmallThreads;                   // 2 or 1 bins per thread, ascending
        uint32_t cb[2] = {0u, 0u}, mine = 0;
#pragma unroll
        for (int i = 0; i < 2; ++i)
          if (i < per) { cb[i] = s_hist[(int)tid * per + i]; mine += cb[i]; }
        uint32_t total;
        const uint32_t below = block_scan_excl_1024(mine, s_warp, &total);
        if (tid == 0) s_sel[0] = 0xFFFFFFFFu;
        __syncthreads();
        if (below < t_rem && below + mine >= t_rem) {            // exactly one thread
          uint32_t a = below;
#pragma unroll
          for (int i = 0; i < 2; ++i) {
            if (i < per) {
              if (a + cb[i] >= t_rem) { s_sel[0] = (uint32_t)((int)tid * per + i); s_sel[1] = a; break; }
              a += cb[i];
            }
          }
        }
        __syncthreads();
        uint32_t digit = s_sel[0];
        const uint32_t a = s_sel[1];
        if (digit == 0xFFFFFFFFu) {                              // cannot happen: take <= n_equal
          if (tid == 0) atomicOr(hdr + kHdrStatus, (uint32_t)kFlagInternal);
          digit = 0u;
        } else {
          t_rem -= a;
        }
        iprefix = (iprefix << (pass == 2 ? 10 : 11)) | digit;
        __syncthreads();
      }
      idx_limit = iprefix;
      rank_ties = false;                                         // decided by idx_limit instead
    }
    uint32_t* s_tie_idx = s_hist;                                // the histogram is no longer needed
    uint32_t* s_tie_neg = s_hist + kMaxTiesUnordered;
    if (tid == 0) s_sel[0] = 0u;
    __syncthreads();
#pragma unroll 4
    for (uint32_t i = tid; i < n; i += kSmallThreads) {
      const uint32_t bits = s_bits[i], key = bits & kAbsMask;
      if (key > tau || (key == tau && !rank_ties && s_idx[i] <= idx_limit)) {
        const uint32_t idx = s_idx[i];
        add_vote(o.counter, o.packed, idx, bits >> 31);
        if (o.err) o.err[(uint64_t)row * o.d + idx] = 0.f;
      } else if (rank_ties && key == tau) {
        const uint32_t slot = atomicAdd(&s_sel[0], 1u);
        s_tie_idx[slot] = s_idx[i];
        s_tie_neg[slot] = bits >> 31;
      }
    }
    uint32_t n_kept = k_want;
    if (rank_ties) {
      __syncthreads();
      const uint32_t e = s_sel[0];                               // == n_equal
      if (tid < e) {
        const uint32_t mine = s_tie_idx[tid];
        uint32_t before = 0;
        for (uint32_t j = 0; j < e; ++j) before += (uint32_t)(s_tie_idx[j] < mine);
        if (before < take) {
          add_vote(o.counter, o.packed, mine, s_tie_neg[tid]);
          if (o.err) o.err[(uint64_t)row * o.d + mine] = 0.f;
        }
      }
      if (e != n_equal) n_kept = 0xFFFFFFFFu;                    // cannot happen
    }
    if (tid == 0) {
      rows[row].tau = tau;
      rows[row].take_ties = take;
      rows[row].n_emitted = n_kept == k_want ? o.K : n_kept;
      if (!kBin) {                                               // a kRowBin row was counted when it was marked
        rows[row].done = 1u;
        atomicAdd(hdr + kHdrRowsDone, 1u);
      }
      if (n_kept != k_want || (kBin && rs.n_bin > cap)) {
        atomicAdd(hdr + kHdrBadCount, 1u);
        atomicOr(hdr + kHdrStatus, (uint32_t)kFlagInternal);
      }
      atomicMax(hdr + kHdrMaxCand, kBin ? rs.n_cand : n);
    }
    return;
  }

  // ---- ordered emission, kPer consecutive candidates per thread and round: an entry is kept if
  // it is above tau, or equal to tau with fewer than `take` equal entries before it; its
  // output position is the number of kept entries before it.  (Many entries per thread keep
  // the number of block-wide scans, and with it of warp shuffles, small.)
  constexpr int kPer = 16;
  uint32_t carry_eq = 0, carry_out = 0;
  // the row's sign words are put together in shared memory (the histogram's words are free again;
  // K <= n <= 27k entries are at most 848 words) and written out whole at the end
  const bool sign_on_chip = o.signbits != nullptr && o.words <= (uint32_t)kHistBins;
  if (sign_on_chip) {
    for (uint32_t w = tid; w < o.words; w += kSmallThreads) s_hist[w] = 0u;
    __syncthreads();
  }
  for (uint32_t base = 0; base < n; base += kSmallThreads * kPer) {
    const uint32_t i0 = base + tid * kPer;
    uint32_t bits[kPer], eqf = 0, inf = 0;
#pragma unroll
    for (int q = 0; q < kPer; ++q) {
      const bool in = i0 + q < n;
      bits[q] = in ? s_bits[i0 + q] : 0u;
      inf |= (uint32_t)in << q;
      eqf |= (uint32_t)(in && (bits[q] & kAbsMask) == tau) << q;
    }
    uint32_t tot_eq, tot_sel;
    const uint32_t tie0 = carry_eq + block_scan_excl_1024(__popc(eqf), s_warp, &tot_eq);
    uint32_t self = 0, tie = tie0;
#pragma unroll
    for (int q = 0; q < kPer; ++q) {
      const uint32_t key = bits[q] & kAbsMask;
      const uint32_t is_eq = eqf >> q & 1u;
      const bool keep = (inf >> q & 1u) && (key > tau || (is_eq && tie < take));
      tie += is_eq;
      self |= (uint32_t)keep << q;
    }
    uint32_t pos = carry_out + block_scan_excl_1024(__popc(self), s_warp, &tot_sel);
#pragma unroll
    for (int q = 0; q < kPer; ++q) {
      if (self >> q & 1u) {
        if (pos < o.K) {
          const uint32_t idx = s_idx[i0 + q];
          const uint32_t neg = bits[q] >> 31;
          if (o.idx) o.idx[(uint64_t)row * o.K + pos] = idx;
          if (o.counter) add_vote(o.counter, o.packed, idx, neg);
          if (o.err) o.err[(uint64_t)row * o.d + idx] = 0.f;
          // sign bits only when the message is asked for: one atomic per negative entry
          if (neg) {
            if (sign_on_chip) atomicOr(&s_hist[pos >> 5], 1u << (pos & 31));
            else if (o.signbits) atomicOr(o.signbits + (uint64_t)row * o.words + (pos >> 5), 1u << (pos & 31));
          }
        }
        ++pos;
      }
    }
    carry_eq += tot_eq;
    carry_out += tot_sel;
  }
  if (sign_on_chip) {
    __syncthreads();
    for (uint32_t w = tid; w < o.words; w += kSmallThreads) o.signbits[(uint64_t)row * o.words + w] = s_hist[w];
  }
  if (tid == 0) {
    rows[row].tau = tau;
    rows[row].take_ties = take;
    rows[row].n_emitted = carry_out;
    rows[row].done = 1u;
    atomicAdd(hdr + kHdrRowsDone, 1u);
    if (carry_out != o.K) {
      atomicAdd(hdr + kHdrBadCount, 1u);
      atomicOr(hdr + kHdrStatus, (uint32_t)kFlagInternal);
    }
    atomicMax(hdr + kHdrMaxCand, n);
  }
}


// ---- votes only, for a row whose candidates need the shared memory of several SMs: a
// thread-block cluster of C CTAs per row.  CTA r keeps the r-th slice of the row's candidate
// list in its own shared memory and counts its own histogram; after a cluster barrier every
// CTA adds up the C histograms through distributed shared memory and takes the same decision,
// so nothing is broadcast.  Entries equal to tau, if not all of them are kept, are cut by a
// second radix select on the index (the lowest indices win).  Every CTA then votes for its slice.
template <uint32_t C>
__global__ void __launch_bounds__(kSmallThreads, 1)
select_cluster_kernel(RowState* __restrict__ rows, const uint2* __restrict__ cand, uint32_t cap,
                      uint32_t* __restrict__ hdr, EmitOut o) {
  namespace cg = cooperative_groups;
  cg::cluster_group cluster = cg::this_cluster();
  extern __shared__ __align__(16) unsigned char smem_raw[];
  __shared__ uint32_t s_hist[kHistBins];
  __shared__ uint32_t s_warp[kSmallWarps];
  __shared__ uint32_t s_sel[2];
  const uint32_t rank = cluster.block_rank();             // the launch gives the cluster C CTAs
  const uint32_t row = blockIdx.x / C, tid = threadIdx.x, lane = tid & 31;
  grid_dependency_wait();                                 // (the launch allows an early start, as launch_after() does)
  const RowState rs = rows[row];
  const uint32_t n = rs.n_cand;
  const uint32_t per_cta = (n + C - 1) / C;
  // the same for every CTA of the cluster: either all go on or all leave
  if (!row_uses_candidates(rs, o.K, cap)) return;
  if ((uint64_t)per_cta * 8u > (uint64_t)kSmallSelectBytes) {
    if (o.unordered && rank == 0 && tid == 0) rows[row].exact = 1u;   // see select_small_kernel
    return;
  }
  const uint32_t lo = rank * per_cta < n ? rank * per_cta : n;
  const uint32_t hi = lo + per_cta < n ? lo + per_cta : n;
  const uint32_t m = hi - lo;                                  // entries of this CTA
  uint32_t* s_bits = reinterpret_cast<uint32_t*>(smem_raw);
  uint32_t* s_idx = s_bits + per_cta;
  const uint2* c = cand + (uint64_t)row * cap + lo;
#pragma unroll 8
  for (uint32_t i = tid; i < m; i += kSmallThreads) {
    const uint2 e = c[i];
    s_bits[i] = e.x;
    s_idx[i] = e.y;
  }
  // bin `b` summed over the cluster (C is a template argument so that the remote loads are all
  // issued before the first one is used)
  auto combined = [&](uint32_t b) {
    uint32_t part[C];
#pragma unroll
    for (uint32_t q = 0; q < C; ++q) part[q] = cluster.map_shared_rank(s_hist, q)[b];
    uint32_t v = 0;
#pragma unroll
    for (uint32_t q = 0; q < C; ++q) v += part[q];
    return v;
  };
  // One radix pass over a 2048- or 1024-bin histogram that every CTA has filled for its slice:
  // finds the bin holding the want-th entry counted from the top (descending) or from the bottom,
  // returns it and the number of entries before it; *in_bin = entries in that bin.
  auto pick = [&](int nbins, bool from_top, uint32_t want, uint32_t* before, uint32_t* in_bin) -> uint32_t {
    cluster.sync();                                            // all C histograms are complete
    const int per = nbins > kSmallThreads ? nbins / kSmallThreads : 1;
    uint32_t mine = 0, cbin[2] = {0u, 0u};
    if ((int)tid * per < nbins) {
#pragma unroll
      for (int i = 0; i < 2; ++i)
        if (i < per) {
          const int pos = (int)tid * per + i;
          cbin[i] = combined((uint32_t)(from_top ? nbins - 1 - pos : pos));
          mine += cbin[i];
        }
    }
    uint32_t total;
    const uint32_t earlier = block_scan_excl_1024(mine, s_warp, &total);
    if (tid == 0) s_sel[0] = 0xFFFFFFFFu;
    __syncthreads();
    if (earlier < want && earlier + mine >= want) {            // exactly one thread
      uint32_t a = earlier;
#pragma unroll
      for (int i = 0; i < 2; ++i) {
        if (i < per) {
          if (a + cbin[i] >= want) {
            const int pos = (int)tid * per + i;
            s_sel[0] = (uint32_t)(from_top ? nbins - 1 - pos : pos);
            s_sel[1] = a;
            break;
          }
          a += cbin[i];
        }
      }
    }
    __syncthreads();
    uint32_t digit = s_sel[0];
    *before = s_sel[1];
    if (digit == 0xFFFFFFFFu) {                                // fewer than `want` entries: cannot happen for a valid row
      if (tid == 0) atomicOr(hdr + kHdrStatus, (uint32_t)kFlagInternal);
      digit = 0u;
      *before = 0u;
    }
    *in_bin = combined(digit);
    cluster.sync();                                            // everyone has read before anyone clears
    return digit;
  };

  // ---- tau = K-th largest magnitude of the row, take = how many entries equal to tau are kept
  uint32_t prefix = 0, k_rem = o.K - rs.n_hi, n_equal = 0;
  for (int pass = 0; pass < kNumPasses; ++pass) {
    const int nbins = 1 << pass_bits(pass);
    const uint32_t mask = (uint32_t)(nbins - 1);
    for (int b = tid; b < nbins; b += kSmallThreads) s_hist[b] = 0u;
    __syncthreads();                                           // also: the slice is on chip (first pass)
    if (pass == 0) {
      const uint32_t d_lo = (rs.tau_lo >> pass_shift(0)) & mask;
      uint32_t cnt8[8] = {0u, 0u, 0u, 0u, 0u, 0u, 0u, 0u};
      for (uint32_t i = tid; i < m; i += kSmallThreads) {
        const uint32_t digit = ((s_bits[i] & kAbsMask) >> pass_shift(0)) & mask;
        const uint32_t rel = digit - d_lo;
#pragma unroll
        for (uint32_t b = 0; b < 8; ++b) cnt8[b] += (uint32_t)(rel == b);
        if (rel >= 8u) atomicAdd(&s_hist[digit], 1u);
      }
#pragma unroll
      for (uint32_t b = 0; b < 8; ++b) {
        const uint32_t v = __reduce_add_sync(0xFFFFFFFFu, cnt8[b]);
        if (lane == b && v != 0u) atomicAdd(&s_hist[(d_lo + b) & mask], v);
      }
    } else {
      for (uint32_t i = tid; i < m; i += kSmallThreads) {
        const uint32_t key = s_bits[i] & kAbsMask;
        if ((key >> pass_shift(pass - 1)) == prefix) atomicAdd(&s_hist[(key >> pass_shift(pass)) & mask], 1u);
      }
    }
    uint32_t a;
    const uint32_t digit = pick(nbins, true, k_rem, &a, &n_equal);
    prefix = (prefix << pass_bits(pass)) | digit;
    k_rem -= a;
  }
  const uint32_t tau = prefix, take = k_rem;

  // ---- entries equal to tau: all kept, or the `take` lowest indices
  uint32_t idx_limit = 0xFFFFFFFFu;
  if (n_equal > take) {
    uint32_t iprefix = 0, t_rem = take;
#pragma unroll 1
    for (int pass = 0; pass < 3; ++pass) {
      const int shift = pass == 0 ? 21 : (pass == 1 ? 10 : 0);
      const int prev_shift = pass == 1 ? 21 : 10;
      const int nbins = pass == 2 ? 1024 : 2048;
      const uint32_t mask = (uint32_t)(nbins - 1);
      for (int b = tid; b < nbins; b += kSmallThreads) s_hist[b] = 0u;
      __syncthreads();
      for (uint32_t i = tid; i < m; i += kSmallThreads) {
        if ((s_bits[i] & kAbsMask) != tau) continue;
        const uint32_t idx = s_idx[i];
        if (pass == 0 || (idx >> prev_shift) == iprefix) atomicAdd(&s_hist[(idx >> shift) & mask], 1u);
      }
      uint32_t a, unused;
      const uint32_t digit = pick(nbins, false, t_rem, &a, &unused);
      t_rem -= a;
      iprefix = (iprefix << (pass == 2 ? 10 : 11)) | digit;
    }
    idx_limit = iprefix;
  }

  // ---- votes of this slice
#pragma unroll 4
  for (uint32_t i = tid; i < m; i += kSmallThreads) {
    const uint32_t bits = s_bits[i], key = bits & kAbsMask;
    if (key > tau || (key == tau && s_idx[i] <= idx_limit)) {
      const uint32_t idx = s_idx[i];
      add_vote(o.counter, o.packed, idx, bits >> 31);
      if (o.err) o.err[(uint64_t)row * o.d + idx] = 0.f;
    }
  }
  if (rank == 0 && tid == 0) {
    rows[row].tau = tau;
    rows[row].take_ties = take;
    rows[row].n_emitted = o.K;
    rows[row].done = 1u;
    atomicAdd(hdr + kHdrRowsDone, 1u);
    atomicMax(hdr + kHdrMaxCand, n);
  }
}

}  // namespace

cudaError_t launch_select_small(const Layout& L, RowState* rows, const uint2* cand, const uint2* seg, uint32_t* hdr,
                                const EmitOut& o, cudaStream_t st) {
  // enough dynamic shared memory for the largest row this kernel accepts
  uint64_t need = (uint64_t)L.cap * 8u;
  if (need > kSmallSelectBytes) need = kSmallSelectBytes;
  const bool ordered = o.idx != nullptr || o.signbits != nullptr || o.counter == nullptr;
  auto kernel = ordered ? select_small_kernel<true> : select_small_kernel<false>;
  static int opted[2][kMaxDevices];
  cudaError_t e = opt_in_dynamic_smem(reinterpret_cast<const void*>(kernel), (int)kSmallSelectBytes, opted[ordered ? 1 : 0]);
  if (e != cudaSuccess) return e;
  e = launch_after(kernel, dim3(L.M), dim3(kSmallThreads), (size_t)need, st, rows, cand, L.cap, seg, L.n_tiles, hdr, o);
  if (e == cudaSuccess) count_launch();
  return e;
}

cudaError_t launch_select_bin(const Layout& L, RowState* rows, const uint2* bin, uint32_t bin_cap, uint32_t* hdr,
                              const EmitOut& o, cudaStream_t st) {
  auto kernel = select_small_kernel<false, true>;
  static int opted[kMaxDevices];
  cudaError_t e = opt_in_dynamic_smem(reinterpret_cast<const void*>(kernel), (int)kSmallSelectBytes, opted);
  if (e != cudaSuccess) return e;
  uint64_t need = (uint64_t)bin_cap * 8u;
  if (need > kSmallSelectBytes) need = kSmallSelectBytes;
  e = launch_after(kernel, dim3(L.M), dim3(kSmallThreads), (size_t)need, st, rows, bin, bin_cap,
                   static_cast<const uint2*>(nullptr), 0u, hdr, o);
  if (e == cudaSuccess) count_launch();
  return e;
}

}  // namespace s3gd

namespace s3gd {

// Smallest cluster (2 or 4 CTAs) whose shared memory holds a row of `n_cand` candidates; 0 if none does.
// (Eight CTAs per row measured slower than the general passes: 0.895 against 0.876 ms at 159k candidates.)
uint32_t cluster_size_for(uint32_t n_cand) {
  for (uint32_t c = 2; c <= 4; c *= 2)
    if ((uint64_t)((n_cand + c - 1) / c) * 8u <= (uint64_t)kSmallSelectBytes) return c;
  return 0u;
}

cudaError_t launch_select_cluster(const Layout& L, RowState* rows, const uint2* cand, uint32_t* hdr, const EmitOut& o,
                                  uint32_t cluster, cudaStream_t st) {
  auto kernel = cluster == 2u ? select_cluster_kernel<2> : (cluster == 4u ? select_cluster_kernel<4> : select_cluster_kernel<8>);
  if (cluster != 2u && cluster != 4u && cluster != 8u) return cudaErrorInvalidValue;
  static int opted[3][kMaxDevices];
  cudaError_t e = opt_in_dynamic_smem(reinterpret_cast<const void*>(kernel), (int)kSmallSelectBytes,
                                      opted[cluster == 2u ? 0 : (cluster == 4u ? 1 : 2)]);
  if (e != cudaSuccess) return e;
  uint64_t need = (uint64_t)((L.cap + cluster - 1) / cluster) * 8u;
  if (need > kSmallSelectBytes) need = kSmallSelectBytes;
  cudaLaunchConfig_t cfg = {};
  cfg.gridDim = dim3((unsigned)L.M * cluster);
  cfg.blockDim = dim3(kSmallThreads);
  cfg.dynamicSmemBytes = (size_t)need;
  cfg.stream = st;
  cudaLaunchAttribute attr[2];
  attr[0].id = cudaLaunchAttributeClusterDimension;
  attr[0].val.clusterDim.x = cluster;
  attr[0].val.clusterDim.y = 1;
  attr[0].val.clusterDim.z = 1;
  attr[1].id = cudaLaunchAttributeProgrammaticStreamSerialization;    // as launch_after()
  attr[1].val.programmaticStreamSerializationAllowed = 1;
  cfg.attrs = attr;
  cfg.numAttrs = 2;
  e = cudaLaunchKernelEx(&cfg, kernel, rows, cand, L.cap, hdr, o);
  if (e == cudaSuccess) count_launch();
  return e;
}

}  // namespace s3gd

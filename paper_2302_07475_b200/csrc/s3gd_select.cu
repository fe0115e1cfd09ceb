// Exact top-K of every row by a most-significant-digit radix select on the
// magnitude bits (11 + 10 + 10), followed by a stable, index-ordered emission
// with the lowest-index rule for entries equal to the K-th magnitude
// (Eq. (3)-(4); the tie rule is this library's reading).
//
// Two sources feed the same passes:
//   * candidates: the filtered list of a row (few entries, L2 resident) -- normal case;
//   * whole row:  every entry of the row -- for large K, and for rows whose filter
//                 produced fewer than K or more than `cap` survivors.
// Each launch carries blocks for both sources; a block looks at its row's state and
// works only if its source is the live one (row_uses_candidates), so the host never
// has to look at device state.  The per-row follow-up of a pass (choosing the digit,
// scanning the per-tile counts) is done by whichever block finishes that row last.
#include <cooperative_groups.h>

#include "s3gd_tile.cuh"

namespace s3gd {

namespace {

constexpr int kSelThreads = 256;
static_assert(kSelThreads == kTileThreads, "row-source blocks load tiles with kTileThreads threads");

// ---------------------------------------------------------------- init
__global__ void init_kernel(uint32_t* __restrict__ hdr, RowState* __restrict__ rows, uint32_t* __restrict__ hist,
                            int M, uint32_t K, uint32_t force_exact) {
  const uint32_t tid = blockIdx.x * blockDim.x + threadIdx.x, nthr = gridDim.x * blockDim.x;
  if (tid < (uint32_t)kHdrWords) hdr[tid] = 0u;
  for (uint32_t m = tid; m < (uint32_t)M; m += nthr) {
    RowState rs = {};
    rs.k_rem = K;
    rs.exact = force_exact;
    rs.tau_hi = kNoPrevote;
    rows[m] = rs;
  }
  for (uint64_t i = tid; i < (uint64_t)M * kHistBins; i += nthr) hist[i] = 0u;
}

// A row's state.  kFromL2: in the single-launch form the passes are separated by grid-wide
// barriers and the state is rewritten between them by other SMs, so the fields that change are
// taken from L2; a launch of its own starts with a clean L1 and reads them the ordinary way,
// which measured faster.
template <bool kFromL2>
__device__ __forceinline__ RowState load_row_state(const RowState* p) {
  if (!kFromL2) return *p;
  RowState rs = {};
  rs.tau_lo = p->tau_lo;
  rs.n_cand = p->n_cand;
  rs.done = p->done;
  rs.tau_hi = p->tau_hi;
  rs.n_hi = p->n_hi;
  rs.exact = __ldcg(&p->exact);              // the first pass of the two-pass form may set it
  rs.prefix = __ldcg(&p->prefix);
  rs.k_rem = __ldcg(&p->k_rem);
  rs.tau = __ldcg(&p->tau);
  rs.take_ties = __ldcg(&p->take_ties);
  rs.n_emitted = __ldcg(&p->n_emitted);
  return rs;
}

// True in exactly one block per row: the one that arrives after all others of that row have
// published their global writes.  Every block of the row must call it exactly once.
__device__ __forceinline__ bool last_block_of_row(uint32_t* ticket, uint32_t n_blocks, uint32_t* s_flag) {
  __threadfence();
  __syncthreads();
  if (threadIdx.x == 0) {
    const uint32_t t = atomicAdd(ticket, 1u);
    *s_flag = (t == n_blocks - 1u) ? 1u : 0u;
    if (t == n_blocks - 1u) atomicExch(ticket, 0u);      // ready for the next pass
  }
  __syncthreads();
  const bool last = *s_flag != 0u;
  if (last) __threadfence();
  return last;
}

// ------------------------------------------------------- histogram passes
// Shared-memory histogram.  Gradient magnitudes cluster: in a coarse pass, or in any pass over
// quantised gradients, a whole warp often holds one digit value, and 32 atomics on one word
// would serialise.  So a warp first checks whether its active lanes agree (a ballot, a shuffle
// and a vote); if so one lane adds their count.  Otherwise every lane adds for itself: the
// digits are then spread out, and plain atomics measured faster than grouping equal digits
// with __match_any_sync (two histogram passes over 10.8 M candidates: 77 against 87 us).
__device__ __forceinline__ void hist_add(uint32_t* s_hist, bool on, uint32_t digit) {
  const uint32_t act = __ballot_sync(0xFFFFFFFFu, on);
  if (act == 0u) return;                             // warp-uniform
  const uint32_t lead = (uint32_t)__ffs((int)act) - 1u;
  const uint32_t d0 = __shfl_sync(0xFFFFFFFFu, digit, lead);
  if (__all_sync(0xFFFFFFFFu, !on || digit == d0)) {
    if ((threadIdx.x & 31u) == lead) atomicAdd(&s_hist[d0], (uint32_t)__popc(act));
  } else if (on) {
    atomicAdd(&s_hist[digit], 1u);
  }
}

__device__ __forceinline__ bool in_prefix(uint32_t key, uint32_t prefix, int pass) {
  return pass == 0 || (key >> pass_shift(pass - 1)) == prefix;
}

// Two-pass form for rows that select from their candidates.  Every candidate is at or above
// tau_lo, and the K-th magnitude is normally within a few percent of it, so the first two
// digits of the three-pass form carry almost no information: all candidates share them.  The
// first pass here takes the 11-bit digit from (key >> 10) - (tau_lo >> 10) instead -- 2047 bins
// of 1024 keys, a quarter of an octave above tau_lo, and one bin for everything beyond -- and
// thereby fixes the upper 21 bits at once; the second pass is the ordinary last pass over the
// low 10 bits.  RowState::done == kRowTwoPass marks a row whose first pass found its bin; its
// remaining passes run in launches that look only at such rows, and the general launch after
// them skips it like any finished row.
// If only the votes are wanted the rest is shorter still: everything above the bin is in the top K
// whatever the low bits say, so it votes in the second sweep, which also copies the entries of the
// bin itself -- a few thousand as a rule -- to the row's bin list; one CTA then selects the k_rem
// largest of those on chip (ties to the lower index) and lets them vote.  No count, no ordered
// emission.  The first pass knows how many entries the bin holds and marks the row kRowBin only
// if the list fits one CTA's shared memory.
constexpr uint32_t kJointClamp = (uint32_t)kHistBins - 1u;
__device__ __forceinline__ uint32_t joint_digit(uint32_t key, uint32_t tau_lo) {
  const uint32_t rel = (key >> pass_shift(1)) - (tau_lo >> pass_shift(1));
  return rel < kJointClamp ? rel : kJointClamp;
}

// Find the digit in which the k_rem-th largest entry lies, fix it, and clear the
// histogram for the next pass.  One block of kSelThreads threads.
__device__ __forceinline__ void pick_digit(RowState* __restrict__ rows, uint32_t row, uint32_t* __restrict__ h,
                                           uint32_t* __restrict__ hdr, int pass, uint32_t* s_sum, uint32_t* s_sel,
                                           bool joint = false, uint32_t bin_limit = 0u, bool band = false) {
  const uint32_t tid = threadIdx.x;
  const int nbins = 1 << pass_bits(pass);
  const int per = nbins / kSelThreads;               // 8 or 4 bins per thread, ascending
  uint32_t c[8];
  uint32_t mine = 0;
#pragma unroll
  for (int i = 0; i < 8; ++i) {
    c[i] = (i < per) ? __ldcg(h + tid * per + i) : 0u;
    mine += c[i];
  }
  s_sum[tid] = mine;
  if (tid == 0) { s_sel[0] = 0xFFFFFFFFu; s_sel[1] = 0u; }
  __syncthreads();
  // (first pass of the two-pass form: whatever voted during the filter pass is no longer looked for)
  const uint32_t k_rem = __ldcg(&rows[row].k_rem) - (joint ? rows[row].n_hi : 0u);
  uint32_t above = 0;                                // entries in bins owned by higher threads
  for (int t = kSelThreads - 1; t > (int)tid; --t) above += s_sum[t];
  if (above < k_rem && above + mine >= k_rem) {      // exactly one thread
    uint32_t a = above;
    for (int i = per - 1; i >= 0; --i) {
      if (a + c[i] >= k_rem) { s_sel[0] = tid * per + i; s_sel[1] = a; s_sel[2] = c[i]; break; }
      a += c[i];
    }
  }
  __syncthreads();
  for (int i = 0; i < per; ++i) h[tid * per + i] = 0u;
  if (tid == 0 && joint) {
    // first pass of the two-pass form: the digit counts 1024-key steps above tau_lo.  The top bin
    // collects everything further up; if the k_rem-th entry lies there the row stays untouched
    // (prefix 0, k_rem K, histogram cleared) and the launch that follows the fast passes does it.
    const uint32_t digit = s_sel[0], a = s_sel[1];
    if (digit < kJointClamp) {
      rows[row].prefix = (rows[row].tau_lo >> pass_shift(1)) + digit;
      rows[row].k_rem = k_rem - a;
      rows[row].done = s_sel[2] <= bin_limit ? kRowBin : kRowTwoPass;
      atomicAdd(hdr + kHdrRowsDone, 1u);
    } else if (band) {
      rows[row].exact = 1u;       // an unordered list cannot go through count and emission: redo the whole row
    }
  } else if (tid == 0) {
    uint32_t digit = s_sel[0], a = s_sel[1];
    if (digit == 0xFFFFFFFFu) {                      // fewer than k_rem entries: cannot happen for a valid row
      atomicOr(hdr + kHdrStatus, (uint32_t)kFlagInternal);
      digit = 0u; a = 0u;
    }
    const uint32_t prefix = (__ldcg(&rows[row].prefix) << pass_bits(pass)) | digit;
    rows[row].prefix = prefix;
    rows[row].k_rem = k_rem - a;
    if (pass == kNumPasses - 1) {
      rows[row].tau = prefix;
      rows[row].take_ties = k_rem - a;
    }
  }
}

// One (virtual) block of a histogram pass.  A row has gx blocks: the first gx_c walk its
// candidates, the others its tiles; bx is the block's number within the row.
template <bool kFromL2>
__device__ __forceinline__ void hist_pick_block(const uint32_t* __restrict__ gbits, uint64_t d, uint32_t n_tiles,
                                                const uint2* __restrict__ cand, uint32_t cap,
                                                RowState* __restrict__ rows, uint32_t K, uint32_t* __restrict__ hist,
                                                uint32_t* __restrict__ hdr, int pass, uint32_t gx_c, uint32_t bx,
                                                uint32_t row, uint32_t gx) {
  __shared__ uint32_t s_hist[kHistBins];
  __shared__ uint32_t s_sum[kSelThreads];
  __shared__ uint32_t s_sel[3];
  __shared__ uint32_t s_flag;
  const RowState rs = load_row_state<kFromL2>(rows + row);
  if (rs.done) return;                               // finished by the single-CTA selection (all blocks of the row agree)
  const bool use_c = row_uses_candidates(rs, K, cap);
  const bool is_c = bx < gx_c;
  const int nbins = 1 << pass_bits(pass);
  const uint32_t mask = (uint32_t)(nbins - 1);
  uint32_t* g_hist = hist + (uint64_t)row * kHistBins;
  bool worked = false;
  if (is_c && use_c && (uint64_t)bx * kSelThreads * 4 < rs.n_cand) {
    worked = true;
    for (int b = threadIdx.x; b < nbins; b += kSelThreads) s_hist[b] = 0u;
    __syncthreads();
    const uint2* c = cand + (uint64_t)row * cap;
    // four entries per thread and round, all four loads issued before the first is used
    const uint32_t n = rs.n_cand, step = gx_c * kSelThreads * 4;
    for (uint32_t base = bx * kSelThreads * 4; base < n; base += step) {
      uint32_t key[4];
      bool on[4];
#pragma unroll
      for (int u = 0; u < 4; ++u) {
        const uint32_t i = base + u * kSelThreads + threadIdx.x;
        on[u] = i < n;
        key[u] = on[u] ? (c[i].x & kAbsMask) : 0u;
      }
#pragma unroll
      for (int u = 0; u < 4; ++u)
        hist_add(s_hist, on[u] && in_prefix(key[u], rs.prefix, pass), (key[u] >> pass_shift(pass)) & mask);
    }
  } else if (!is_c && !use_c) {
    worked = true;
    for (int b = threadIdx.x; b < nbins; b += kSelThreads) s_hist[b] = 0u;
    __syncthreads();
    const uint32_t* rowp = gbits + (uint64_t)row * d;
    const uint32_t head = row_head(rowp, d);
    const uint32_t gx_r = gx - gx_c;
    for (uint32_t t = bx - gx_c; t < n_tiles; t += gx_r) {
      Tile T;
      load_tile(T, rowp, d, head, t);
      if (t == 0 && threadIdx.x < 32) {
        const uint32_t key = T.head_bits & kAbsMask;
        hist_add(s_hist, T.head_valid && in_prefix(key, rs.prefix, pass), (key >> pass_shift(pass)) & mask);
      }
#pragma unroll
      for (int it = 0; it < kTileIters; ++it) {
#pragma unroll
        for (int q = 0; q < 4; ++q) {
          const uint32_t key = T.bits[it][q] & kAbsMask;
          const bool on = (T.valid[it] >> q & 1u) && in_prefix(key, rs.prefix, pass);
          hist_add(s_hist, on, (key >> pass_shift(pass)) & mask);
        }
      }
    }
  }
  if (worked) {
    __syncthreads();
    for (int b = threadIdx.x; b < nbins; b += kSelThreads) {
      const uint32_t c = s_hist[b];
      if (c) atomicAdd(&g_hist[b], c);
    }
  }
  if (last_block_of_row(&rows[row].ticket_hist, gx, &s_flag))
    pick_digit(rows, row, g_hist, hdr, pass, s_sum, s_sel);
}

// One block of a histogram pass of the two-pass form (pass 0: the joint digit; pass 2: the low
// 10 bits).  Candidate rows only; a row has gx blocks.
// The second sweep of a kRowBin row: entries above the bin vote, entries of the bin go to the list
// (in any order).  Each warp stages its bin entries in shared memory and claims room in the list
// for 64 or more of them at once: one claim per warp and step queued 8,000 atomics per row on the
// one list counter (125 us for this sweep), and staging per block cost a barrier per round (61 us).
constexpr int kTwoPassLoads = 4;                    // candidate entries a thread of a two-pass sweep has in flight
constexpr uint32_t kBinFlush = 64;                   // a warp flushes once it holds more than this
constexpr uint32_t kBinStage = kBinFlush + kTwoPassLoads * 32;   // ... so that a round of loads always fits
__device__ __forceinline__ void collect_bin_block(const uint2* __restrict__ c, const RowState& rs, RowState* rowp,
                                                  uint2* __restrict__ bin, uint32_t bin_cap, const EmitOut& o,
                                                  uint32_t bx, uint32_t gx) {
  __shared__ uint2 s_stage[kSelThreads / 32][kBinStage];
  const uint32_t lane = threadIdx.x & 31, warp = threadIdx.x >> 5, lt = lanemask_lt();
  const uint32_t n = rs.n_cand, step = gx * kSelThreads * kTwoPassLoads;
  uint32_t staged = 0;                               // warp-uniform
  for (uint32_t base = bx * kSelThreads * kTwoPassLoads; base < n; base += step) {
    uint2 e[kTwoPassLoads];
    bool on[kTwoPassLoads];
#pragma unroll
    for (int u = 0; u < kTwoPassLoads; ++u) {
      const uint32_t i = base + u * kSelThreads + threadIdx.x;
      on[u] = i < n;
      e[u] = on[u] ? c[i] : make_uint2(0u, 0u);
    }
#pragma unroll
    for (int u = 0; u < kTwoPassLoads; ++u) {
      const uint32_t p = (e[u].x & kAbsMask) >> pass_shift(1);
      if (on[u] && p > rs.prefix) add_vote(o.counter, o.packed, e[u].y, e[u].x >> 31);
      const bool in_bin = on[u] && p == rs.prefix;
      const uint32_t b = __ballot_sync(0xFFFFFFFFu, in_bin);
      if (b == 0u) continue;                           // warp-uniform
      if (in_bin) s_stage[warp][staged + __popc(b & lt)] = e[u];
      staged += (uint32_t)__popc(b);
    }
    if (staged > kBinFlush || (staged != 0u && base + step >= n)) {     // warp-uniform
      __syncwarp();
      uint32_t at0 = 0;
      if (lane == 0) at0 = atomicAdd(&rowp->n_bin, staged);
      at0 = __shfl_sync(0xFFFFFFFFu, at0, 0);
      for (uint32_t i = lane; i < staged; i += 32)
        if (at0 + i < bin_cap) bin[at0 + i] = s_stage[warp][i];
      __syncwarp();
      staged = 0;
    }
  }
}

__device__ __forceinline__ void hist_two_pass_block(const uint2* __restrict__ cand, uint32_t cap,
                                                    RowState* __restrict__ rows, uint32_t K,
                                                    uint32_t* __restrict__ hist, uint32_t* __restrict__ hdr, int pass,
                                                    uint32_t bx, uint32_t row, uint32_t gx, uint2* __restrict__ bin,
                                                    uint32_t bin_cap, const EmitOut& o, bool band) {
  __shared__ uint32_t s_hist[kHistBins];
  __shared__ uint32_t s_sum[kSelThreads];
  __shared__ uint32_t s_sel[3];
  __shared__ uint32_t s_flag;
  const RowState rs = rows[row];
  const bool joint = pass == 0;
  if (!joint && rs.done == kRowBin) {
    collect_bin_block(cand + (uint64_t)row * cap, rs, rows + row, bin + (uint64_t)row * bin_cap, bin_cap, o, bx, gx);
    return;
  }
  if (joint ? (rs.done != 0u || !row_uses_candidates(rs, K, cap)) : rs.done != kRowTwoPass) return;
  const int nbins = 1 << pass_bits(pass);
  const uint32_t mask = (uint32_t)(nbins - 1);
  uint32_t* g_hist = hist + (uint64_t)row * kHistBins;
  if ((uint64_t)bx * kSelThreads * kTwoPassLoads < rs.n_cand) {
    for (int b = threadIdx.x; b < nbins; b += kSelThreads) s_hist[b] = 0u;
    __syncthreads();
    const uint2* c = cand + (uint64_t)row * cap;
    const uint32_t n = rs.n_cand, step = gx * kSelThreads * kTwoPassLoads;
    for (uint32_t base = bx * kSelThreads * kTwoPassLoads; base < n; base += step) {
      uint32_t key[kTwoPassLoads];
      bool on[kTwoPassLoads];
#pragma unroll
      for (int u = 0; u < kTwoPassLoads; ++u) {
        const uint32_t i = base + u * kSelThreads + threadIdx.x;
        on[u] = i < n;
        key[u] = on[u] ? (c[i].x & kAbsMask) : 0u;
      }
#pragma unroll
      for (int u = 0; u < kTwoPassLoads; ++u) {
        if (joint) hist_add(s_hist, on[u], joint_digit(key[u], rs.tau_lo));
        else hist_add(s_hist, on[u] && in_prefix(key[u], rs.prefix, pass), key[u] & mask);
      }
    }
    __syncthreads();
    for (int b = threadIdx.x; b < nbins; b += kSelThreads) {
      const uint32_t cnt = s_hist[b];
      if (cnt) atomicAdd(&g_hist[b], cnt);
    }
  }
  if (last_block_of_row(&rows[row].ticket_hist, gx, &s_flag))
    pick_digit(rows, row, g_hist, hdr, pass, s_sum, s_sel, joint, o.counter != nullptr && o.idx == nullptr ? bin_cap : 0u,
               band);
}

}  // namespace
}  // namespace s3gd

#include "s3gd_select_emit.inl"

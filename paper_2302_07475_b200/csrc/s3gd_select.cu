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
  rs.exact = p->exact;
  rs.done = p->done;
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
// Shared-memory histogram with warp-aggregated increments: lanes that hit the same
// bin elect a leader which adds their count once (gradient magnitudes cluster in a
// few bins, and quantised gradients do so in every pass, so plain atomics would
// serialise on those bins).
__device__ __forceinline__ void hist_add(uint32_t* s_hist, bool on, uint32_t digit) {
  const uint32_t peers = __match_any_sync(0xFFFFFFFFu, on ? digit : 0xFFFFFFFFu);
  if (on && (peers & lanemask_lt()) == 0u) atomicAdd(&s_hist[digit], (uint32_t)__popc(peers));
}

__device__ __forceinline__ bool in_prefix(uint32_t key, uint32_t prefix, int pass) {
  return pass == 0 || (key >> pass_shift(pass - 1)) == prefix;
}

// Find the digit in which the k_rem-th largest entry lies, fix it, and clear the
// histogram for the next pass.  One block of kSelThreads threads.
__device__ __forceinline__ void pick_digit(RowState* __restrict__ rows, uint32_t row, uint32_t* __restrict__ h,
                                           uint32_t* __restrict__ hdr, int pass, uint32_t* s_sum, uint32_t* s_sel) {
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
  const uint32_t k_rem = __ldcg(&rows[row].k_rem);
  uint32_t above = 0;                                // entries in bins owned by higher threads
  for (int t = kSelThreads - 1; t > (int)tid; --t) above += s_sum[t];
  if (above < k_rem && above + mine >= k_rem) {      // exactly one thread
    uint32_t a = above;
    for (int i = per - 1; i >= 0; --i) {
      if (a + c[i] >= k_rem) { s_sel[0] = tid * per + i; s_sel[1] = a; break; }
      a += c[i];
    }
  }
  __syncthreads();
  for (int i = 0; i < per; ++i) h[tid * per + i] = 0u;
  if (tid == 0) {
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
  __shared__ uint32_t s_sel[2];
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

}  // namespace
}  // namespace s3gd

#include "s3gd_select_emit.inl"

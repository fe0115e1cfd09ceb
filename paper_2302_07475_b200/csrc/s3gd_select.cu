// Exact top-K of every row by a most-significant-digit radix select on the
// magnitude bits (11 + 10 + 10), followed by a stable, index-ordered emission
// with the lowest-index rule for entries equal to the K-th magnitude
// (Eq. (3)-(4); the tie rule is this library's reading).
//
// Two sources feed the same passes:
//   * candidates: the filtered list of a row (few entries, L2 resident) -- normal case;
//   * whole row:  every entry of the row -- for large K, and for rows whose filter
//                 produced fewer than K or more than `cap` survivors.
// Each kernel decides per row which source is live (row_uses_candidates), so the
// host never has to look at device state.
#include "s3gd_tile.cuh"

namespace s3gd {

namespace {

constexpr int kHistThreads = 256;

// ---------------------------------------------------------------- init
__global__ void init_kernel(uint32_t* __restrict__ hdr, RowState* __restrict__ rows, uint32_t* __restrict__ hist,
                            int M, uint32_t K, uint32_t force_exact) {
  const uint32_t tid = blockIdx.x * blockDim.x + threadIdx.x, nthr = gridDim.x * blockDim.x;
  if (tid < (uint32_t)kHdrWords) hdr[tid] = 0u;
  for (uint32_t m = tid; m < (uint32_t)M; m += nthr) {
    RowState rs;
    rs.tau_lo = 0u; rs.n_cand = 0u; rs.prefix = 0u; rs.k_rem = K;
    rs.tau = 0u; rs.take_ties = 0u; rs.n_emitted = 0u; rs.exact = force_exact;
    rows[m] = rs;
  }
  for (uint64_t i = tid; i < (uint64_t)M * kHistBins; i += nthr) hist[i] = 0u;
}

// ------------------------------------------------------- histogram passes
// Shared-memory histogram with warp-aggregated increments: lanes that hit the same
// bin elect a leader which adds their count once.
__device__ __forceinline__ void hist_add(uint32_t* s_hist, bool on, uint32_t digit) {
  uint32_t peers = __match_any_sync(0xFFFFFFFFu, on ? digit : 0xFFFFFFFFu);
  if (on && (peers & lanemask_lt()) == 0u) atomicAdd(&s_hist[digit], (uint32_t)__popc(peers));
}

__device__ __forceinline__ bool in_prefix(uint32_t key, uint32_t prefix, int pass) {
  return pass == 0 || (key >> pass_shift(pass - 1)) == prefix;
}

__device__ __forceinline__ void hist_flush(const uint32_t* s_hist, uint32_t* __restrict__ g_hist, int nbins) {
  for (int b = threadIdx.x; b < nbins; b += blockDim.x) {
    uint32_t c = s_hist[b];
    if (c) atomicAdd(&g_hist[b], c);
  }
}

// grid (blocks per row, M)
__global__ void __launch_bounds__(kHistThreads) hist_cand_kernel(const uint2* __restrict__ cand, uint32_t cap,
                                                                 const RowState* __restrict__ rows, uint32_t K,
                                                                 uint32_t* __restrict__ hist, int pass) {
  __shared__ uint32_t s_hist[kHistBins];
  const uint32_t row = blockIdx.y;
  const RowState rs = rows[row];
  if (!row_uses_candidates(rs, K, cap)) return;
  const uint32_t n = rs.n_cand;
  if ((uint64_t)blockIdx.x * kHistThreads >= n) return;
  const int nbins = 1 << pass_bits(pass);
  for (int b = threadIdx.x; b < nbins; b += kHistThreads) s_hist[b] = 0u;
  __syncthreads();
  const uint2* c = cand + (uint64_t)row * cap;
  const uint32_t step = gridDim.x * kHistThreads;
  const uint32_t n_round = (n + 31u) & ~31u;          // whole warps stay in the loop together
  for (uint32_t i = blockIdx.x * kHistThreads + threadIdx.x; i < n_round; i += step) {
    bool on = i < n;
    uint32_t key = on ? (c[i].x & kAbsMask) : 0u;
    on = on && in_prefix(key, rs.prefix, pass);
    hist_add(s_hist, on, (key >> pass_shift(pass)) & (uint32_t)(nbins - 1));
  }
  __syncthreads();
  hist_flush(s_hist, hist + (uint64_t)row * kHistBins, nbins);
}

// grid (blocks per row, M); each block walks tiles of its row
__global__ void __launch_bounds__(kTileThreads) hist_row_kernel(const uint32_t* __restrict__ gbits, uint64_t d,
                                                                uint32_t n_tiles, uint32_t cap,
                                                                const RowState* __restrict__ rows, uint32_t K,
                                                                uint32_t* __restrict__ hist, int pass) {
  __shared__ uint32_t s_hist[kHistBins];
  const uint32_t row = blockIdx.y;
  const RowState rs = rows[row];
  if (row_uses_candidates(rs, K, cap)) return;
  const int nbins = 1 << pass_bits(pass);
  for (int b = threadIdx.x; b < nbins; b += kTileThreads) s_hist[b] = 0u;
  __syncthreads();
  const uint32_t* rowp = gbits + (uint64_t)row * d;
  const uint32_t head = row_head(rowp, d);
  const uint32_t mask = (uint32_t)(nbins - 1);
  for (uint32_t t = blockIdx.x; t < n_tiles; t += gridDim.x) {
    Tile T;
    load_tile(T, rowp, d, head, t);
    if (t == 0 && threadIdx.x < 32) {
      uint32_t key = T.head_bits & kAbsMask;
      hist_add(s_hist, T.head_valid && in_prefix(key, rs.prefix, pass), (key >> pass_shift(pass)) & mask);
    }
#pragma unroll
    for (int it = 0; it < kTileIters; ++it) {
#pragma unroll
      for (int q = 0; q < 4; ++q) {
        uint32_t key = T.bits[it][q] & kAbsMask;
        bool on = (T.valid[it] >> q & 1u) && in_prefix(key, rs.prefix, pass);
        hist_add(s_hist, on, (key >> pass_shift(pass)) & mask);
      }
    }
  }
  __syncthreads();
  hist_flush(s_hist, hist + (uint64_t)row * kHistBins, nbins);
}

// One CTA per row: find the digit in which the k_rem-th largest entry lies, fix it,
// and clear the histogram for the next pass.
__global__ void __launch_bounds__(256) pick_kernel(RowState* __restrict__ rows, uint32_t* __restrict__ hist,
                                                   uint32_t* __restrict__ hdr, int pass) {
  __shared__ uint32_t s_sum[256];
  __shared__ uint32_t s_sel[2];
  const uint32_t row = blockIdx.x, tid = threadIdx.x;
  const int nbins = 1 << pass_bits(pass);
  const int per = nbins / 256;                       // 8 or 4 bins per thread, ascending
  uint32_t* h = hist + (uint64_t)row * kHistBins;
  uint32_t c[8];
  uint32_t mine = 0;
#pragma unroll
  for (int i = 0; i < 8; ++i) {
    c[i] = (i < per) ? h[tid * per + i] : 0u;
    mine += c[i];
  }
  s_sum[tid] = mine;
  if (tid == 0) { s_sel[0] = 0xFFFFFFFFu; s_sel[1] = 0u; }
  __syncthreads();
  const uint32_t k_rem = rows[row].k_rem;
  // entries in bins owned by higher threads
  uint32_t above = 0;
  for (int t = 255; t > (int)tid; --t) above += s_sum[t];
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
    RowState rs = rows[row];
    if (digit == 0xFFFFFFFFu) {                      // fewer than k_rem entries: cannot happen for a valid row
      atomicOr(hdr + kHdrStatus, (uint32_t)kFlagInternal);
      digit = 0u; a = 0u;
    }
    rs.prefix = (rs.prefix << pass_bits(pass)) | digit;
    rs.k_rem = k_rem - a;
    if (pass == kNumPasses - 1) {
      rs.tau = rs.prefix;
      rs.take_ties = rs.k_rem;
    }
    rows[row] = rs;
  }
}

}  // namespace
}  // namespace s3gd

#include "s3gd_select_emit.inl"

// The single read of the gradients: a sampled, conservative magnitude threshold
// per row, then one streaming pass that keeps every entry at or above it.
//
// Why this is exact: the true top-K of a row (Eq. (3), ties to the lower index)
// consists of entries with magnitude >= the K-th largest magnitude.  If the
// filter threshold tau_lo is <= that magnitude, all of them survive the filter,
// and "survivors >= K" proves tau_lo was low enough.  The sample only decides how
// many extra survivors there are; a bad sample costs a second route, never a wrong
// answer (rows with too few or too many survivors take the exact multi-pass route).
#include "s3gd_tile.cuh"

namespace s3gd {

namespace {

__device__ __forceinline__ uint32_t mix32(uint32_t v) {   // integer finaliser, spreads group numbers
  v ^= v >> 16; v *= 0x7FEB352Du;
  v ^= v >> 15; v *= 0x846CA68Bu;
  v ^= v >> 16;
  return v;
}

// One CTA per row.  Histogram of magnitude >> 16 over n_sample entries taken as
// chunks of 32 neighbours (one 128-byte line, so the sample costs its own bytes and
// no more) spread evenly over the row with a hashed offset inside each stride, then
// tau_lo = lower edge of the highest bin b with (#sampled >= b) >= j_rank.
constexpr int kChunk = 32;
constexpr int kSampleUnroll = 8;

// The kernel also resets the row's selection state, its radix histogram and (block 0) the
// status words, so that no separate initialisation launch is needed on this route.
__global__ void __launch_bounds__(1024) sample_threshold_kernel(const uint32_t* __restrict__ gbits, uint64_t d,
                                                                RowState* __restrict__ rows, uint32_t n_sample,
                                                                uint32_t stride, uint32_t j_rank, uint32_t K,
                                                                uint32_t* __restrict__ hdr,
                                                                uint32_t* __restrict__ hist) {
  extern __shared__ uint32_t s_hist[];            // kSampleBins counters
  __shared__ uint32_t s_wsum[32];
  __shared__ uint32_t s_pick[2];
  const uint32_t tid = threadIdx.x, warp = tid >> 5, lane = tid & 31;
  const uint32_t row = blockIdx.x;
  const uint32_t* rowp = gbits + (uint64_t)row * d;

  if (blockIdx.x == 0 && tid < (uint32_t)kHdrWords) hdr[tid] = 0u;
  if (tid == 0) {
    RowState rs = {};
    rs.k_rem = K;
    rows[row] = rs;                                // tau_lo is filled in at the end
  }
  for (uint32_t b = tid; b < (uint32_t)kHistBins; b += 1024) hist[(uint64_t)row * kHistBins + b] = 0u;
  for (uint32_t b = tid; b < (uint32_t)kSampleBins; b += 1024) s_hist[b] = 0u;
  __syncthreads();
  if (stride == 0) {                              // short row: every entry is inspected
    for (uint32_t e = tid; e < n_sample; e += 1024) atomicAdd(&s_hist[(rowp[e] & kAbsMask) >> 16], 1u);
  } else {
    const uint32_t n_chunks = n_sample / kChunk;  // chunk c starts in [c*stride, (c+1)*stride - 32]
    for (uint32_t c0 = warp; c0 < n_chunks; c0 += 32 * kSampleUnroll) {
      uint32_t v[kSampleUnroll];
#pragma unroll
      for (int u = 0; u < kSampleUnroll; ++u) {
        const uint32_t c = c0 + 32 * u;
        if (c < n_chunks) {
          const uint64_t pos = (uint64_t)c * stride + (mix32(c) % (stride - (kChunk - 1))) + lane;
          v[u] = __ldg(rowp + pos);
        }
      }
#pragma unroll
      for (int u = 0; u < kSampleUnroll; ++u)
        if (c0 + 32 * u < n_chunks) atomicAdd(&s_hist[(v[u] & kAbsMask) >> 16], 1u);
    }
  }
  __syncthreads();

  // warp w owns bins [1024 w, 1024 w + 1024): conflict-free strided reads
  uint32_t part = 0;
#pragma unroll 8
  for (int i = 0; i < 32; ++i) part += s_hist[warp * 1024 + i * 32 + lane];
#pragma unroll
  for (int s = 16; s > 0; s >>= 1) part += __shfl_xor_sync(0xFFFFFFFFu, part, s);
  if (lane == 0) s_wsum[warp] = part;
  if (tid == 0) { s_pick[0] = 0xFFFFFFFFu; s_pick[1] = 0u; }
  __syncthreads();
  if (tid == 0) {
    // highest warp range in which the count from the top reaches j_rank
    uint32_t above = 0;
    for (int w = 31; w >= 0; --w) {
      if (above + s_wsum[w] >= j_rank) { s_pick[0] = (uint32_t)w; s_pick[1] = above; break; }
      above += s_wsum[w];
    }
  }
  __syncthreads();
  const uint32_t wsel = s_pick[0];
  if (wsel == 0xFFFFFFFFu) {                     // fewer than j_rank samples in total: keep everything
    if (tid == 0) rows[row].tau_lo = 0u;
    return;
  }
  if (warp != wsel) return;
  // inside the chosen 1024 bins: 32 groups of 32 bins, from the top
  uint32_t above = s_pick[1];
  uint32_t result = 0;
  bool found = false;
  for (int g = 31; g >= 0 && !found; --g) {
    uint32_t c = s_hist[wsel * 1024 + g * 32 + lane];
    uint32_t suffix = c;                         // inclusive count of this bin and higher bins of the group
#pragma unroll
    for (int s = 1; s < 32; s <<= 1) {
      uint32_t o = __shfl_down_sync(0xFFFFFFFFu, suffix, s);
      if (lane + s < 32) suffix += o;
    }
    uint32_t gtot = __shfl_sync(0xFFFFFFFFu, suffix, 0);
    if (above + gtot >= j_rank) {
      uint32_t ok = __ballot_sync(0xFFFFFFFFu, above + suffix >= j_rank);   // lanes 0..L satisfy it
      int top = 31 - __clz(ok);                  // highest bin of the group that still reaches j_rank
      result = wsel * 1024 + g * 32 + (uint32_t)top;
      found = true;
    } else {
      above += gtot;
    }
  }
  if (lane == 0) rows[row].tau_lo = result << 16;
}

// Persistent CTAs over (row, tile).  Survivors of a tile are appended to the row's
// candidate list in ascending index order; the list position of a tile is claimed
// with one atomic, and (position, count) is recorded per tile so that later passes
// can walk a row's candidates in index order without sorting.
//
// One block barrier per tile and no wait on the claim: the survivors of tile k are
// first staged in shared memory at their rank; the atomic that claims their list
// position is issued and left in flight; after the barrier of tile k+1 -- a whole
// tile of loads and compares later -- its result is there and the staged survivors
// are copied out, coalesced.  Tiles with more survivors than the staging buffer holds
// (dense regions) claim and store directly, with one more barrier.
constexpr int kStageCap = 512;                 // survivors staged per tile (8 bytes each, two buffers)

// magnitude >= tau_lo, decided on the float value: |x| < tau is false for NaN, whose bit
// pattern is above every threshold, so !(|x| < tau) agrees with the unsigned compare of the
// sign-less bit patterns for every input (denormals are not flushed in this build).
__device__ __forceinline__ uint32_t hit(uint32_t b, float tau) { return (uint32_t)!(fabsf(__uint_as_float(b)) < tau); }

__global__ void __launch_bounds__(kTileThreads, 4) filter_kernel(const uint32_t* __restrict__ gbits, int M, uint64_t d,
                                                              RowState* __restrict__ rows, uint2* __restrict__ cand,
                                                              uint32_t cap, uint2* __restrict__ seg,
                                                              uint32_t n_tiles) {
  __shared__ uint2 s_stage[2][kStageCap];
  __shared__ uint32_t s_wtot[2][kWarpsPerTile + 1];
  __shared__ uint32_t s_base[2];
  __shared__ uint32_t s_direct_base;
  const uint32_t tid = threadIdx.x, lane = tid & 31;
  const uint64_t n_work = (uint64_t)M * n_tiles;
  uint32_t pend_n = 0, pend_row = 0, pend_t = 0;   // staged survivors of the previous tile (uniform)
  uint32_t pend_base = 0;                          // thread 0: the claim made for them (may still be in flight)
  int par = 0;
  for (uint64_t w = blockIdx.x; w < n_work; w += gridDim.x, par ^= 1) {
    const uint32_t row = (uint32_t)(w / n_tiles), t = (uint32_t)(w - (uint64_t)row * n_tiles);
    const uint32_t* rowp = gbits + (uint64_t)row * d;
    const uint32_t head = row_head(rowp, d);
    const float tau = __uint_as_float(rows[row].tau_lo);
    Tile T;
    load_tile(T, rowp, d, head, t);
    uint32_t flags[kTileIters];
#pragma unroll
    for (int it = 0; it < kTileIters; ++it)
      flags[it] = (hit(T.bits[it][0], tau) | (hit(T.bits[it][1], tau) << 1) | (hit(T.bits[it][2], tau) << 2) |
                   (hit(T.bits[it][3], tau) << 3)) & T.valid[it];
    const bool head_flag = T.head_valid && hit(T.head_bits, tau);
    TileRanks R;
    tile_ranks_publish(R, flags, head_flag, s_wtot[par]);
    if (tid == 0 && pend_n) {                      // the claim of the previous tile has had a tile's time to return
      s_base[par ^ 1] = pend_base;
      seg[(uint64_t)pend_row * n_tiles + pend_t] = make_uint2(pend_base, pend_n);
    }
    __syncthreads();
    if (pend_n) {                                  // copy out the previous tile's survivors
      const uint32_t base = s_base[par ^ 1];
      uint2* out = cand + (uint64_t)pend_row * cap;
      for (uint32_t i = tid; i < pend_n; i += kTileThreads)
        if (base + i < cap) out[base + i] = s_stage[par ^ 1][i];
    }
    tile_ranks_collect(R, s_wtot[par]);
    const uint32_t total = R.tile_total;
    if (total == 0u) {
      if (tid == 0) seg[(uint64_t)row * n_tiles + t] = make_uint2(0u, 0u);
      pend_n = 0;
      continue;
    }
    if (total <= (uint32_t)kStageCap) {
      if (head_flag) s_stage[par][R.head_rank] = make_uint2(T.head_bits, lane);
#pragma unroll
      for (int it = 0; it < kTileIters; ++it) {
        if (flags[it] == 0u) continue;
#pragma unroll
        for (int q = 0; q < 4; ++q)
          if (flags[it] >> q & 1u)
            s_stage[par][rank_of(R, flags, it, q)] = make_uint2(T.bits[it][q], (uint32_t)(T.first(it) + q));
      }
      if (tid == 0) pend_base = atomicAdd(&rows[row].n_cand, total);
      pend_n = total; pend_row = row; pend_t = t;
    } else {                                       // dense tile: claim now, store from registers
      if (tid == 0) {
        const uint32_t b = atomicAdd(&rows[row].n_cand, total);
        s_direct_base = b;
        seg[(uint64_t)row * n_tiles + t] = make_uint2(b, total);
      }
      __syncthreads();
      const uint32_t base = s_direct_base;
      uint2* out = cand + (uint64_t)row * cap;
      if (head_flag && base + R.head_rank < cap) out[base + R.head_rank] = make_uint2(T.head_bits, lane);
#pragma unroll
      for (int it = 0; it < kTileIters; ++it) {
        if (flags[it] == 0u) continue;
#pragma unroll
        for (int q = 0; q < 4; ++q) {
          if (flags[it] >> q & 1u) {
            const uint32_t pos = base + rank_of(R, flags, it, q);
            if (pos < cap) out[pos] = make_uint2(T.bits[it][q], (uint32_t)(T.first(it) + q));
          }
        }
      }
      pend_n = 0;
    }
  }
  if (pend_n) {                                    // the last tile's survivors
    if (tid == 0) {
      s_base[par ^ 1] = pend_base;
      seg[(uint64_t)pend_row * n_tiles + pend_t] = make_uint2(pend_base, pend_n);
    }
    __syncthreads();
    const uint32_t base = s_base[par ^ 1];
    uint2* out = cand + (uint64_t)pend_row * cap;
    for (uint32_t i = tid; i < pend_n; i += kTileThreads)
      if (base + i < cap) out[base + i] = s_stage[par ^ 1][i];
  }
}

}  // namespace

cudaError_t launch_sample_and_filter(const uint32_t* gbits, const Layout& L, RowState* rows, uint2* cand, uint2* seg,
                                     uint32_t* hdr, uint32_t* hist, cudaStream_t st) {
  // 128 KB of dynamic shared memory needs the opt-in on every device this runs on
  const size_t smem = (size_t)kSampleBins * sizeof(uint32_t);
  cudaError_t e = cudaFuncSetAttribute(sample_threshold_kernel, cudaFuncAttributeMaxDynamicSharedMemorySize,
                                       (int)smem);
  if (e != cudaSuccess) return e;
  sample_threshold_kernel<<<L.M, 1024, smem, st>>>(gbits, L.d, rows, L.n_sample, L.sample_stride, L.j_rank,
                                                   (uint32_t)L.K, hdr, hist);
  e = cudaGetLastError();
  if (e != cudaSuccess) return e;
  prof_mark(kPhaseSampled, st);
  count_launch(2);
  uint64_t n_work = (uint64_t)L.M * L.n_tiles;
  uint64_t blocks = n_work < (uint64_t)kSMs * 8 ? n_work : (uint64_t)kSMs * 8;
  filter_kernel<<<(unsigned)blocks, kTileThreads, 0, st>>>(gbits, L.M, L.d, rows, cand, L.cap, seg, L.n_tiles);
  return cudaGetLastError();
}

}  // namespace s3gd

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

// The kernel also resets the row's selection state, its radix histogram and (block 0) the
// status words, so that no separate initialisation launch is needed on this route.
// kEF: the row to sample is g = g~ + eta * e, formed on the fly from the gradients and the
// error memory (which still holds e at this point).
// Blocks beyond the M sampling blocks clear the vote counters (if asked to): sampling is
// latency-bound and leaves SMs idle, so the clearing costs no time of its own.
template <bool kEF>
__global__ void __launch_bounds__(1024) sample_threshold_kernel(const uint32_t* __restrict__ gbits, uint64_t d,
                                                                RowState* __restrict__ rows, uint32_t n_sample,
                                                                uint32_t stride, uint32_t j_rank, uint32_t j_hi,
                                                                uint32_t K,
                                                                uint32_t* __restrict__ hdr,
                                                                uint32_t* __restrict__ hist,
                                                                const float* __restrict__ err, float eta, uint32_t M,
                                                                int32_t* __restrict__ zero, uint64_t n_zero,
                                                                uint32_t zero_word) {
  extern __shared__ uint32_t s_hist[];            // kSampleBins counters
  __shared__ uint32_t s_wsum[32];
  const uint32_t tid = threadIdx.x, warp = tid >> 5, lane = tid & 31;
  grid_dependency_wait();                         // (launched with launch_after: whatever ran before on the stream is done)
  if (blockIdx.x >= M) {                          // a clearing block; `zero` is 16-byte aligned, n_zero words
    const uint64_t n4 = n_zero / 4, nthr = (uint64_t)(gridDim.x - M) * 1024;
    uint4* z4 = reinterpret_cast<uint4*>(zero);
    for (uint64_t i = (uint64_t)(blockIdx.x - M) * 1024 + tid; i < n4; i += nthr)
      z4[i] = make_uint4(zero_word, zero_word, zero_word, zero_word);
    if (blockIdx.x == M && tid < (uint32_t)(n_zero - n4 * 4)) zero[n4 * 4 + tid] = (int32_t)zero_word;
    return;
  }
  const uint32_t row = blockIdx.x;
  const uint32_t* rowp = gbits + (uint64_t)row * d;
  const float* errp = kEF ? err + (uint64_t)row * d : nullptr;

  if (blockIdx.x == 0 && tid < (uint32_t)kHdrWords) hdr[tid] = 0u;
  if (tid == 0) {
    RowState rs = {};
    rs.k_rem = K;
    rs.tau_hi = kNoPrevote;
    rows[row] = rs;                                // tau_lo (and tau_hi, if j_hi != 0) are filled in at the end
  }
  for (uint32_t b = tid; b < (uint32_t)kHistBins; b += 1024) hist[(uint64_t)row * kHistBins + b] = 0u;
  for (uint32_t b = tid; b < (uint32_t)kSampleBins; b += 1024) s_hist[b] = 0u;
  __syncthreads();
  // every sampled entry of the row; with error memory the row is formed on the fly from the two buffers.
  // A short row is inspected whole:
  auto visit_samples = [&](auto&& visit) {
    for (uint32_t e = tid; e < n_sample; e += 1024) visit(kEF ? ef_value(rowp[e], errp[e], eta) : rowp[e]);
  };
  // The long-row form: chunk c is 32 neighbours starting in [c*stride, (c+1)*stride - 32], on a 16-byte boundary
  // so that a lane reads four of them at once; eight lanes per chunk, four chunks per warp and load.  (The
  // error memory's rows have the gradient rows' phase within 16 bytes: the host checks.)
  auto visit_samples_vec = [&](auto&& visit) {
    const uint32_t n_chunks = n_sample / kChunk;
    const uint32_t a4 = (uint32_t)(reinterpret_cast<uintptr_t>(rowp) >> 2) & 3u;     // the row's phase within 16 bytes
    constexpr int kVecUnroll = kEF ? 4 : 8;
    for (uint32_t c0 = warp * 4 + (lane >> 3); c0 < n_chunks; c0 += 32 * 4 * kVecUnroll) {
      uint4 v[kVecUnroll];
      float4 e[kEF ? kVecUnroll : 1];
#pragma unroll
      for (int u = 0; u < kVecUnroll; ++u) {
        const uint32_t c = c0 + 32 * 4 * u;
        if (c < n_chunks) {
          // offset inside the stride: hash scaled into [0, stride - 34) by a multiply-high (no division),
          // then up to the next position that is 16-byte aligned in memory (at most 3 further)
          const uint64_t p = (uint64_t)c * stride + __umulhi(mix32(c), stride - (kChunk + 2));
          const uint64_t pos = ((p + a4 + 3u) & ~(uint64_t)3u) - a4 + (lane & 7u) * 4u;
          v[u] = ld_stream_v4(rowp + pos);
          if (kEF) e[u] = __ldg(reinterpret_cast<const float4*>(errp + pos));
        }
      }
#pragma unroll
      for (int u = 0; u < kVecUnroll; ++u) {
        if (c0 + 32 * 4 * u < n_chunks) {
          if (kEF) {
            v[u].x = ef_value(v[u].x, e[u].x, eta); v[u].y = ef_value(v[u].y, e[u].y, eta);
            v[u].z = ef_value(v[u].z, e[u].z, eta); v[u].w = ef_value(v[u].w, e[u].w, eta);
          }
          visit(v[u].x); visit(v[u].y); visit(v[u].z); visit(v[u].w);
        }
      }
    }
  };
  auto visit_all = [&](auto&& visit) {
    if (stride == 0) visit_samples(visit);
    else visit_samples_vec(visit);
  };
  visit_all([&](uint32_t b) { atomicAdd(&s_hist[(b & kAbsMask) >> 16], 1u); });
  __syncthreads();

  // warp w owns bins [1024 w, 1024 w + 1024): conflict-free strided reads
  uint32_t part = 0;
#pragma unroll 8
  for (int i = 0; i < 32; ++i) part += s_hist[warp * 1024 + i * 32 + lane];
#pragma unroll
  for (int s = 16; s > 0; s >>= 1) part += __shfl_xor_sync(0xFFFFFFFFu, part, s);
  if (lane == 0) s_wsum[warp] = part;
  __syncthreads();
  // Two searches for "the highest bin b such that at least `want` sampled entries lie in bins >= b":
  // warp 0 with want = j_rank (tau_lo is that bin's lower edge), warp 1 with want = j_hi + 1 (the bin above
  // it is the lowest one with at most j_hi sampled entries at or above its lower edge: tau_hi).
  __shared__ uint32_t s_res[2];
  __shared__ uint32_t s_fine[2];                  // the bin of tau_lo and the number of sampled entries above it
  const bool searching = warp == 0 || (warp == 1 && j_hi != 0u);
  const uint32_t want = warp == 0 ? j_rank : j_hi + 1u;
  uint32_t wsel = 0xFFFFFFFFu, above = 0;
  if (searching) {
    const uint32_t mine = s_wsum[lane];           // one 1024-bin range per lane
    uint32_t suffix = mine;                        // entries in this range and all higher ones
#pragma unroll
    for (int s = 1; s < 32; s <<= 1) {
      const uint32_t o = __shfl_down_sync(0xFFFFFFFFu, suffix, s);
      if (lane + s < 32) suffix += o;
    }
    const uint32_t ok = __ballot_sync(0xFFFFFFFFu, suffix >= want);   // lanes 0..L satisfy it
    if (ok != 0u) {
      wsel = 31u - (uint32_t)__clz(ok);
      above = __shfl_sync(0xFFFFFFFFu, suffix - mine, wsel);
    }
  }
  uint32_t result = 0xFFFFFFFFu;                   // no such bin: fewer than `want` samples in total
  if (searching && wsel != 0xFFFFFFFFu) {
    // inside the chosen 1024 bins: lane g sums group g (32 bins), a suffix scan over the lanes finds the
    // group, a second one over that group's bins finds the bin -- two rounds instead of a walk over groups
    const uint32_t* hb = s_hist + wsel * 1024;
    uint32_t gsum = 0;
#pragma unroll 8
    for (int i = 0; i < 32; ++i) gsum += hb[lane * 32 + ((i + lane) & 31)];      // staggered: no bank conflicts
    uint32_t suffix = gsum;                          // entries in this group and the higher ones
#pragma unroll
    for (int s = 1; s < 32; s <<= 1) {
      const uint32_t o = __shfl_down_sync(0xFFFFFFFFu, suffix, s);
      if (lane + s < 32) suffix += o;
    }
    const uint32_t okg = __ballot_sync(0xFFFFFFFFu, above + suffix >= want);      // groups 0..G satisfy it (not empty)
    const uint32_t g = 31u - (uint32_t)__clz(okg);
    above += __shfl_sync(0xFFFFFFFFu, suffix - gsum, g);                          // entries in the groups above g
    uint32_t bsuf = hb[g * 32 + lane];                                            // bins of group g, then their suffix sums
#pragma unroll
    for (int s = 1; s < 32; s <<= 1) {
      const uint32_t o = __shfl_down_sync(0xFFFFFFFFu, bsuf, s);
      if (lane + s < 32) bsuf += o;
    }
    const uint32_t okb = __ballot_sync(0xFFFFFFFFu, above + bsuf >= want);        // bins 0..B of the group satisfy it
    const uint32_t bsel = 31u - (uint32_t)__clz(okb);
    result = wsel * 1024 + g * 32 + bsel;
    // sampled entries in bins above the chosen one (for the refinement below)
    above += __shfl_sync(0xFFFFFFFFu, bsuf, bsel) - hb[g * 32 + bsel];
  }
  if (lane == 0 && warp == 0) {
    s_res[0] = result == 0xFFFFFFFFu ? 0u : result << 16;   // too few samples: keep everything
    s_fine[0] = result;
    s_fine[1] = above;
  }
  // bins run to 32767, so the bin above the highest one gives 0x80000000 = kNoPrevote by itself
  if (lane == 0 && warp == 1) s_res[1] = !searching ? kNoPrevote : (result == 0xFFFFFFFFu ? 0u : (result + 1u) << 16);
  __syncthreads();
  if (kEF && s_fine[0] != 0xFFFFFFFFu) {
    // With error memory the magnitudes of the entries that were not kept climb towards the threshold step
    // after step, so a bin of the first histogram (2^-7 relative width) just below the K-th magnitude can
    // hold many times K entries, and a threshold on a bin edge would let all of them through.  Place it
    // inside the bin: a second look at the sample counts the bin's entries by their next 8 bits, and tau_lo
    // becomes the lower edge of the sub-bin that holds rank j (2^-15 relative).
    const uint32_t bin = s_fine[0], above_bin = s_fine[1];
    for (uint32_t b = tid; b < 256u; b += 1024) s_hist[b] = 0u;          // (both searches are past the barrier)
    __syncthreads();
    visit_all([&](uint32_t b) {
      const uint32_t key = b & kAbsMask;
      if ((key >> 16) == bin) atomicAdd(&s_hist[(key >> 8) & 0xFFu], 1u);
    });
    __syncthreads();
    if (warp == 0) {
      uint32_t c[8], mine = 0;                                           // lane l owns sub-bins 8l .. 8l + 7
#pragma unroll
      for (int i = 0; i < 8; ++i) { c[i] = s_hist[lane * 8 + i]; mine += c[i]; }
      uint32_t suffix = mine;
#pragma unroll
      for (int s = 1; s < 32; s <<= 1) {
        const uint32_t o = __shfl_down_sync(0xFFFFFFFFu, suffix, s);
        if (lane + s < 32) suffix += o;
      }
      const uint32_t ok = __ballot_sync(0xFFFFFFFFu, above_bin + suffix >= j_rank);   // not empty: the bin holds rank j
      const uint32_t lsel = ok ? 31u - (uint32_t)__clz(ok) : 0u;
      if (lane == lsel) {
        uint32_t a = above_bin + suffix - mine, sub = 0;
        for (int i = 7; i >= 0; --i) {
          if (a + c[i] >= j_rank) { sub = (uint32_t)i; break; }
          a += c[i];
        }
        s_res[0] = (bin << 16) | ((lane * 8u + sub) << 8);
      }
    }
    __syncthreads();
  }
  if (tid == 0) {
    rows[row].tau_lo = s_res[0];
    rows[row].tau_hi = s_res[1] > s_res[0] ? s_res[1] : s_res[0];      // never below tau_lo: what votes early has passed the filter
  }
}

// Persistent CTAs over (row, tile); CTA c takes the items c, c + gridDim.x, ...  Survivors of a
// tile are appended to the row's candidate list in ascending index order; the list position
// of a tile is claimed with one atomic, and (position, count) is recorded per tile so that
// later passes can walk a row's candidates in index order without sorting.
//
// Fast path (whole tile inside the row, no warp with more than kWarpStage survivors): a warp
// tests its 1024 entries 128 at a time; only iterations in which some lane has a survivor (a
// warp vote) are ranked, by ballot, and their survivors go to the warp's staging list in
// shared memory.  One block barrier per tile publishes the eight warp counts.  The atomic
// that claims the list position is issued and left in flight; after the barrier of the NEXT
// tile -- a whole tile of loads and compares later -- its result is there and every warp
// copies its staged survivors out.
// Other tiles (the ragged last tile of a row, dense regions) are ranked in registers with a
// packed scan, claim at once and store directly, with more barriers.
constexpr int kWarpStage = 64;                 // survivors a warp can stage per tile (8 bytes each, two buffers)

// magnitude >= tau_lo, decided on the float value: |x| < tau is false for NaN, whose bit
// pattern is above every threshold, so !(|x| < tau) agrees with the unsigned compare of the
// sign-less bit patterns for every input (the library is compiled without flush-to-zero: denormals compare as they are).
__device__ __forceinline__ bool hit(uint32_t b, float tau) { return !(fabsf(__uint_as_float(b)) < tau); }

template <bool kEF>
__global__ void __launch_bounds__(kTileThreads, kEF ? 3 : 4) filter_kernel(const uint32_t* __restrict__ gbits, int M,
                                                                           uint64_t d, RowState* __restrict__ rows,
                                                                           uint2* __restrict__ cand, uint32_t cap,
                                                                           uint2* __restrict__ seg, uint32_t n_tiles,
                                                                           float* __restrict__ err, float eta) {
  __shared__ uint2 s_stage[2][kWarpsPerTile][kWarpStage];
  __shared__ __align__(16) uint32_t s_wtot[3][kWarpsPerTile];   // survivors per warp of tile k in slot k % 3
  __shared__ uint32_t s_base[2];
  __shared__ uint32_t s_slow_wtot[kWarpsPerTile + 1];
  __shared__ uint32_t s_slow_base;
  const uint32_t tid = threadIdx.x, warp = tid >> 5, lane = tid & 31, lt = lanemask_lt();
  const uint64_t n_work = (uint64_t)M * n_tiles;
  grid_dependency_wait();                          // (launched with launch_after)
  if (blockIdx.x >= n_work) return;
  // walk (row, tile) without dividing in the loop
  uint32_t row = (uint32_t)(blockIdx.x / n_tiles), t = (uint32_t)(blockIdx.x - (uint64_t)row * n_tiles);
  uint32_t cur_row = 0xFFFFFFFFu, head = 0;
  const uint32_t* rowp = gbits;
  float tau = 0.f;
  uint32_t pend_n = 0, pend_row = 0, pend_t = 0;   // staged survivors of the previous tile (uniform)
  uint32_t pend_base = 0;                          // thread 0: the claim made for them (may still be in flight)
  uint32_t k = 0;
  for (uint64_t w = blockIdx.x; w < n_work; w += gridDim.x, ++k) {
    if (row != cur_row) {
      cur_row = row;
      rowp = gbits + (uint64_t)row * d;
      head = row_head(rowp, d);
      tau = __uint_as_float(rows[row].tau_lo);
    }
    const int par = (int)(k & 1), slot = (int)(k % 3), prev_slot = (slot + 2) % 3;
    const bool whole = (uint64_t)head + (uint64_t)(t + 1) * kTileElems <= d;
    Tile T;
    load_tile(T, rowp, d, head, t);
    if (kEF) ef_materialise(T, err + (uint64_t)row * d, eta);
    uint32_t run = 0;                              // survivors of this warp so far (uniform in the warp)
    if (whole) {
      uint2* wl = s_stage[par][warp];
      if (T.head_valid || (t == 0 && head != 0u && warp == 0)) {      // warp 0 of a row's first tile
        const uint32_t hb = __ballot_sync(0xFFFFFFFFu, T.head_valid && hit(T.head_bits, tau));
        if (hb >> lane & 1u) wl[__popc(hb & lt)] = make_uint2(T.head_bits, lane);
        run = __popc(hb);
      }
      const uint32_t idx0 = (uint32_t)T.e0;
#pragma unroll
      for (int it = 0; it < kTileIters; ++it) {
        const bool h0 = hit(T.bits[it][0], tau), h1 = hit(T.bits[it][1], tau);
        const bool h2 = hit(T.bits[it][2], tau), h3 = hit(T.bits[it][3], tau);
        if (__any_sync(0xFFFFFFFFu, h0 | h1 | h2 | h3)) {
          const uint32_t b0 = __ballot_sync(0xFFFFFFFFu, h0), b1 = __ballot_sync(0xFFFFFFFFu, h1);
          const uint32_t b2 = __ballot_sync(0xFFFFFFFFu, h2), b3 = __ballot_sync(0xFFFFFFFFu, h3);
          uint32_t pos = run + __popc(b0 & lt) + __popc(b1 & lt) + __popc(b2 & lt) + __popc(b3 & lt);
          const uint32_t idx = idx0 + it * 128;
          if (h0) { if (pos < (uint32_t)kWarpStage) wl[pos] = make_uint2(T.bits[it][0], idx); ++pos; }
          if (h1) { if (pos < (uint32_t)kWarpStage) wl[pos] = make_uint2(T.bits[it][1], idx + 1); ++pos; }
          if (h2) { if (pos < (uint32_t)kWarpStage) wl[pos] = make_uint2(T.bits[it][2], idx + 2); ++pos; }
          if (h3) { if (pos < (uint32_t)kWarpStage) wl[pos] = make_uint2(T.bits[it][3], idx + 3); }
          run += __popc(b0) + __popc(b1) + __popc(b2) + __popc(b3);
        }
      }
    }
    if (lane == 0) s_wtot[slot][warp] = run;       // may exceed kWarpStage: the tile then takes the other path
    if (tid == 0 && pend_n) {                      // the claim of the previous tile has had a tile's time to return
      s_base[par ^ 1] = pend_base;
      seg[(uint64_t)pend_row * n_tiles + pend_t] = make_uint2(pend_base, pend_n);
    }
    __syncthreads();
    if (pend_n) {                                  // every warp copies out what it staged for the previous tile
      const uint4 a = *reinterpret_cast<const uint4*>(&s_wtot[prev_slot][0]);
      const uint4 b = *reinterpret_cast<const uint4*>(&s_wtot[prev_slot][4]);
      const uint32_t c[8] = {a.x, a.y, a.z, a.w, b.x, b.y, b.z, b.w};
      uint32_t off = s_base[par ^ 1], n = 0;
#pragma unroll
      for (int wv = 0; wv < kWarpsPerTile; ++wv) {
        off += (uint32_t)wv < warp ? c[wv] : 0u;
        n = (uint32_t)wv == warp ? c[wv] : n;
      }
      uint2* out = cand + (uint64_t)pend_row * cap;
      for (uint32_t i = lane; i < n; i += 32)
        if (off + i < cap) out[off + i] = s_stage[par ^ 1][warp][i];
    }
    uint32_t total, wmax;
    {
      const uint4 a = *reinterpret_cast<const uint4*>(&s_wtot[slot][0]);
      const uint4 b = *reinterpret_cast<const uint4*>(&s_wtot[slot][4]);
      total = a.x + a.y + a.z + a.w + b.x + b.y + b.z + b.w;
      wmax = max(max(max(a.x, a.y), max(a.z, a.w)), max(max(b.x, b.y), max(b.z, b.w)));
    }
    if (whole && wmax <= (uint32_t)kWarpStage) {
      if (total != 0u) {
        if (tid == 0) pend_base = atomicAdd(&rows[row].n_cand, total);
        pend_row = row; pend_t = t;
      } else if (tid == 0) {
        seg[(uint64_t)row * n_tiles + t] = make_uint2(0u, 0u);
      }
      pend_n = total;
    } else {
      // ragged or dense tile: flags and ranks in registers, claim now, store directly
      pend_n = 0;
      uint32_t flags[kTileIters];
#pragma unroll
      for (int it = 0; it < kTileIters; ++it)
        flags[it] = ((uint32_t)hit(T.bits[it][0], tau) | ((uint32_t)hit(T.bits[it][1], tau) << 1) |
                     ((uint32_t)hit(T.bits[it][2], tau) << 2) | ((uint32_t)hit(T.bits[it][3], tau) << 3)) & T.valid[it];
      const bool head_flag = T.head_valid && hit(T.head_bits, tau);
      TileRanks R;
      tile_ranks(R, flags, head_flag, s_slow_wtot);
      if (tid == 0) {
        const uint32_t bse = R.tile_total ? atomicAdd(&rows[row].n_cand, R.tile_total) : 0u;
        s_slow_base = bse;
        seg[(uint64_t)row * n_tiles + t] = make_uint2(bse, R.tile_total);
      }
      __syncthreads();
      const uint32_t base = s_slow_base;
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
    }
    // next item of this CTA
    uint64_t nt = (uint64_t)t + gridDim.x;
    while (nt >= n_tiles) { nt -= n_tiles; ++row; }
    t = (uint32_t)nt;
  }
  if (pend_n) {                                    // the last tile's survivors
    const int par = (int)((k - 1) & 1), slot = (int)((k - 1) % 3);
    if (tid == 0) {
      s_base[par] = pend_base;
      seg[(uint64_t)pend_row * n_tiles + pend_t] = make_uint2(pend_base, pend_n);
    }
    __syncthreads();
    uint32_t off = s_base[par], n = 0;
#pragma unroll
    for (int wv = 0; wv < kWarpsPerTile; ++wv) {
      off += (uint32_t)wv < warp ? s_wtot[slot][wv] : 0u;
      n = (uint32_t)wv == warp ? s_wtot[slot][wv] : n;
    }
    uint2* out = cand + (uint64_t)pend_row * cap;
    for (uint32_t i = lane; i < n; i += 32)
      if (off + i < cap) out[off + i] = s_stage[par][warp][i];
  }
}

// ---- the same pass for denser survivors (more than about one in 250 entries): nearly every
// 128-entry iteration then holds a survivor, so ranking all of them with one packed warp scan
// is cheaper than a vote and four ballots per iteration; survivors are staged per CTA.
constexpr int kStageCap = 512;                 // survivors staged per tile (8 bytes each, two buffers)

// (row, tile) of a persistent CTA's next work item, gridDim.x items further on
__device__ __forceinline__ void next_tile(uint32_t& row, uint32_t& t, uint32_t n_tiles) {
  uint64_t nt = (uint64_t)t + gridDim.x;
  while (nt >= n_tiles) { nt -= n_tiles; ++row; }
  t = (uint32_t)nt;
}

template <bool kEF>
__global__ void __launch_bounds__(kTileThreads, kEF ? 3 : 4) filter_scan_kernel(const uint32_t* __restrict__ gbits, int M, uint64_t d,
                                                              RowState* __restrict__ rows, uint2* __restrict__ cand,
                                                              uint32_t cap, uint2* __restrict__ seg,
                                                              uint32_t n_tiles, float* __restrict__ err, float eta) {
  __shared__ uint2 s_stage[2][kStageCap];
  __shared__ uint32_t s_wtot[2][kWarpsPerTile + 1];
  __shared__ uint32_t s_base[2];
  __shared__ uint32_t s_direct_base;
  const uint32_t tid = threadIdx.x, lane = tid & 31;
  const uint64_t n_work = (uint64_t)M * n_tiles;
  grid_dependency_wait();                          // (launched with launch_after)
  uint32_t pend_n = 0, pend_row = 0, pend_t = 0;   // staged survivors of the previous tile (uniform)
  uint32_t pend_base = 0;                          // thread 0: the claim made for them (may still be in flight)
  int par = 0;
  // walk (row, tile) without dividing in the loop (a 64-bit division per tile is a few percent of
  // the instructions of this issue-bound kernel)
  uint32_t row = (uint32_t)(blockIdx.x / n_tiles), t = (uint32_t)(blockIdx.x - (uint64_t)row * n_tiles);
  for (uint64_t w = blockIdx.x; w < n_work; w += gridDim.x, par ^= 1, next_tile(row, t, n_tiles)) {
    const uint32_t* rowp = gbits + (uint64_t)row * d;
    const uint32_t head = row_head(rowp, d);
    const float tau = __uint_as_float(rows[row].tau_lo);
    Tile T;
    load_tile(T, rowp, d, head, t);
    if (kEF) ef_materialise(T, err + (uint64_t)row * d, eta);
    uint32_t flags[kTileIters];
#pragma unroll
    for (int it = 0; it < kTileIters; ++it)
      flags[it] = ((uint32_t)hit(T.bits[it][0], tau) | ((uint32_t)hit(T.bits[it][1], tau) << 1) |
                   ((uint32_t)hit(T.bits[it][2], tau) << 2) | ((uint32_t)hit(T.bits[it][3], tau) << 3)) & T.valid[it];
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
      // a lane rarely holds more than one survivor among its four entries of an iteration: walk
      // the set bits instead of testing all four slots
#pragma unroll
      for (int it = 0; it < kTileIters; ++it) {
        uint32_t f = flags[it];
        if (f == 0u) continue;
        uint32_t pos = R.warp_off + R.it_off[it] + R.lane_excl[it];
        const uint32_t first = (uint32_t)T.first(it);
        do {
          const uint32_t q = (uint32_t)__ffs((int)f) - 1u;
          const uint32_t lo = (q & 1u) ? T.bits[it][1] : T.bits[it][0];
          const uint32_t hi = (q & 1u) ? T.bits[it][3] : T.bits[it][2];
          s_stage[par][pos++] = make_uint2((q & 2u) ? hi : lo, first + q);
          f &= f - 1u;
        } while (f);
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


// ---- the band form of the pass, for every fused step that wants only the votes (no message, no error memory).
// Two thresholds come from the sample: tau_lo as above and tau_hi, placed so that (with the same
// confidence) FEWER than K entries of the row lie at or above it.  Those entries are the largest
// of the row, hence part of its top K whenever there are at most K of them, so they vote at once
// and are only counted; what is listed is the band tau_lo <= magnitude < tau_hi, from which the
// remaining K - n_hi are selected afterwards -- a fraction of what the plain form lists.  Whether
// the guess held (n_hi <= K <= n_hi + band) is checked per row on the device after the pass; a row
// where it did not is redone over the whole row, and the emission of that route takes back the votes
// of entries that voted here without belonging to the top K.
// Votes need no order, and ties at the K-th magnitude are cut by index, which every listed entry
// carries; so the list is unordered and nothing is ranked.  The kernel is built to issue few
// instructions per entry, because with survivors in nearly every 128-entry step the ranked forms
// are bound by instruction issue, not by memory:
//   A  a lane takes the largest magnitude of its four entries of a step (three max operations that
//      keep NaN) and compares once; the warp branches together if any lane has a survivor, and only
//      then are the four entries tested one by one and the survivors pushed (bit pattern, index) onto
//      the CTA's queue with one shared-memory atomic each;
//   C  after the tile's one barrier all threads drain the queue side by side, one entry each: an
//      entry at or above tau_hi votes, a band entry moves to the CTA's band buffer;
//   D  one tile later the band buffer's count is final and thread 0 claims room in the row's list;
//   F  another tile later the claim has returned and the buffer is copied out, coalesced.
// Three buffers of each kind, so that a buffer is never refilled before its readers have passed
// the next barrier.  A tile that pushes more than the queue holds is redone entry by entry after the
// barrier; a band entry that finds the band buffer full claims its place in the row's list by itself (rare).

__device__ __forceinline__ float max_keep_nan(float a, float b) {   // maximum that is NaN if either operand is
  float r;
  asm("max.NaN.f32 %0, %1, %2;" : "=f"(r) : "f"(a), "f"(b));
  return r;
}

struct BandCtx {
  uint32_t tau_hi, packed, cap;
  int32_t* counter;
  uint32_t* n_cand;          // the row's list counter
  uint2* out;                // the row's list
};

// An entry that found no room in a shared-memory buffer: vote, or claim one place in the row's list.
// Returns 1 if it voted.
__device__ __noinline__ uint32_t band_direct(const BandCtx c, uint32_t bits, uint32_t idx) {
  if ((bits & kAbsMask) >= c.tau_hi) {
    add_vote(c.counter, c.packed, idx, bits >> 31);
    return 1u;
  }
  const uint32_t g = atomicAdd(c.n_cand, 1u);
  if (g < c.cap) c.out[g] = make_uint2(bits, idx);
  return 0u;
}

// Push onto the CTA's queue.  An entry that finds the queue full lands in the spare slot behind it;
// the count keeps running, and a tile that pushed more than the queue holds is redone entry by entry.
__device__ __forceinline__ void queue_push(uint2* q, uint32_t* q_cnt, uint32_t bits, uint32_t idx) {
  const uint32_t slot = atomicAdd(q_cnt, 1u);
  q[min(slot, 4u * blockDim.x)] = make_uint2(bits, idx);      // (the queue holds 4 entries per thread)
}

// The first tile of a row whose start is not on a 128-byte boundary, the ragged last tile, and
// (direct) any tile that pushed more than the queue holds: every entry is loaded and tested by
// itself and either pushed or, in the direct form, handled at once.  e0: row index of the thread's
// first entry of the tile (its others follow in steps of 128, four at a time); head: entries of the
// row before its first 128-byte boundary, which belong to tile 0.  Returns the number of entries that voted.
__device__ __noinline__ uint32_t band_tile_slow(const uint32_t* __restrict__ rowp, uint64_t d, uint32_t head, bool first,
                                                uint32_t e0, float tau, uint2* q, uint32_t* q_cnt, const BandCtx c,
                                                bool direct) {
  uint32_t voted = 0;
  auto take = [&](uint32_t e) {
    const uint32_t bits = ld_stream_u32(rowp + e);
    if (!hit(bits, tau)) return;
    if (direct) voted += band_direct(c, bits, e);
    else queue_push(q, q_cnt, bits, e);
  };
  if (first && threadIdx.x < head) take(threadIdx.x);
#pragma unroll 1
  for (int it = 0; it < kTileIters; ++it) {
#pragma unroll 1
    for (uint32_t k = 0; k < 4; ++k) {
      const uint64_t e = (uint64_t)e0 + (uint32_t)it * 128u + k;
      if (e < d) take((uint32_t)e);
    }
  }
  return voted;
}

// kThreads threads take tiles of 32 * kThreads entries (a warp owns 1024 contiguous ones, as in the
// other forms).  Measured on the resnet50 shape at K = 1 % (filter pass alone): 256 threads with 4 / 5 / 6
// CTAs per SM 0.578 / 0.551 / 0.675 ms (56 / 46 / 40 registers); 128 and 64 threads with 8 and 16 CTAs per SM
// 0.68 and 1.06 ms.  Five CTAs of 256 threads it is: 1280 threads per SM.
constexpr int kBandThreadsPerSm = 1280;
template <int kThreads>
__global__ void __launch_bounds__(kThreads, kBandThreadsPerSm / kThreads) filter_band_kernel(const uint32_t* __restrict__ gbits, int M,
                                                                                uint64_t d, RowState* __restrict__ rows,
                                                                                uint2* __restrict__ cand, uint32_t cap,
                                                                                int32_t* __restrict__ counter,
                                                                                uint32_t packed) {
  grid_dependency_wait();                                        // (launched with launch_after)
  constexpr uint32_t kElems = (uint32_t)kThreads * 32u;          // entries per tile
  constexpr int kQueueCap = 4 * kThreads;                        // survivors of a tile the queue holds
  constexpr int kBandStage = 2 * kThreads;                       // band entries of a tile the band buffer holds
  const uint32_t n_tiles = (uint32_t)((d + kElems - 1) / kElems);
  __shared__ uint2 s_q[3][kQueueCap + 1];            // + the spare slot that takes pushes beyond the capacity
  __shared__ uint2 s_b[3][kBandStage];
  __shared__ uint32_t s_qcnt[3], s_bcnt[3], s_hi[3], s_base[3];
  const uint32_t tid = threadIdx.x, lane = tid & 31, warp = tid >> 5;
  const uint64_t n_work = (uint64_t)M * n_tiles;
  if (tid < 3) { s_qcnt[tid] = 0u; s_bcnt[tid] = 0u; s_hi[tid] = 0u; }
  __syncthreads();
  // tiles of this CTA, and two more rounds to let the last two tiles through steps D and F
  const uint64_t n_mine = blockIdx.x < n_work ? (n_work - blockIdx.x + gridDim.x - 1) / gridDim.x : 0;
  uint32_t row = (uint32_t)(blockIdx.x / n_tiles), t = (uint32_t)(blockIdx.x - (uint64_t)row * n_tiles);
  uint32_t loaded_row = 0xFFFFFFFFu, tau_hi = kNoPrevote, e0 = 0;
  float tau = 0.f;
  bool fast = false;                               // the tile in flight is whole and starts on a 128-byte boundary
  uint4 v[kTileIters];
  auto issue_loads = [&]() {
    const uint32_t* rowp = gbits + (uint64_t)row * d;
    const uint32_t head = row_head(rowp, d);
    if (row != loaded_row) {
      loaded_row = row;
      tau = __uint_as_float(rows[row].tau_lo);
      tau_hi = rows[row].tau_hi;
    }
    fast = (uint64_t)head + (uint64_t)(t + 1) * kElems <= d && !(t == 0 && head != 0u);
    e0 = head + t * kElems + warp * 1024u + lane * 4u;
    if (fast) {
      const uint32_t* p = rowp + e0;
#pragma unroll
      for (int it = 0; it < kTileIters; ++it) v[it] = ld_stream_v4(p + it * 128);
    }
  };
  auto ctx_of = [&](uint32_t r, uint32_t th) {
    BandCtx c;
    c.tau_hi = th; c.packed = packed; c.cap = cap; c.counter = counter;
    c.n_cand = &rows[r].n_cand; c.out = cand + (uint64_t)r * cap;
    return c;
  };
  uint32_t row1 = 0;                               // tile k-1: its band buffer fills until this round's barrier
  bool have1 = false;
  uint32_t n2 = 0, row2 = 0, base2 = 0;            // tile k-2: claimed (thread 0 holds base2), copied out this round
  int cur = 0;                                     // k % 3
  for (uint64_t k = 0; k < n_mine + 2; ++k, cur = cur == 2 ? 0 : cur + 1) {
    const int p1 = cur == 0 ? 2 : cur - 1, p2 = cur == 2 ? 0 : cur + 1;      // (k-1) % 3, (k-2) % 3
    const bool live = k < n_mine;
    if (live) {
      if (k) next_tile(row, t, n_tiles);
      issue_loads();
    }
    // tile k's identity, for the steps after the barrier
    const uint32_t row_c = row, t_c = t, tau_hi_c = tau_hi, e0_c = e0;
    const float tau_c = tau;
    if (live) {
      // ---- A: survivors of this tile -> queue
      if (fast) {
#pragma unroll
        for (int it = 0; it < kTileIters; ++it) {
          const float a = max_keep_nan(fabsf(__uint_as_float(v[it].x)), fabsf(__uint_as_float(v[it].y)));
          const float b = max_keep_nan(fabsf(__uint_as_float(v[it].z)), fabsf(__uint_as_float(v[it].w)));
          // a branch the whole warp takes together (no divergence to manage)
          if (__any_sync(0xFFFFFFFFu, !(max_keep_nan(a, b) < tau))) {
            const uint32_t idx = e0 + it * 128;
            if (hit(v[it].x, tau)) queue_push(s_q[cur], &s_qcnt[cur], v[it].x, idx);
            if (hit(v[it].y, tau)) queue_push(s_q[cur], &s_qcnt[cur], v[it].y, idx + 1);
            if (hit(v[it].z, tau)) queue_push(s_q[cur], &s_qcnt[cur], v[it].z, idx + 2);
            if (hit(v[it].w, tau)) queue_push(s_q[cur], &s_qcnt[cur], v[it].w, idx + 3);
          }
        }
      } else {
        const uint32_t* rowp = gbits + (uint64_t)row * d;
        band_tile_slow(rowp, d, row_head(rowp, d), t == 0, e0, tau, s_q[cur], &s_qcnt[cur], ctx_of(row, tau_hi), false);
      }
    }
    // ---- E: the claim made for tile k-2 a round ago has had a tile's time to return
    if (tid == 0 && n2) s_base[p2] = base2;
    __syncthreads();
    // ---- F: copy out the band entries of tile k-2
    if (n2) {
      const uint32_t base = s_base[p2];
      uint2* out = cand + (uint64_t)row2 * cap;
      for (uint32_t i = tid; i < n2; i += kThreads)
        if (base + i < cap) out[base + i] = s_b[p2][i];
    }
    // ---- C: drain this tile's queue, one entry per thread and round
    if (live) {
      uint32_t my_hi = 0;
      const uint32_t pushed = s_qcnt[cur];
      uint32_t n = pushed;
      if (pushed > (uint32_t)kQueueCap) {          // (the same for every thread) more survivors than the queue holds:
        n = 0;                                     // drop it and handle the tile's entries one by one
        const uint32_t* rowp = gbits + (uint64_t)row_c * d;
        my_hi = band_tile_slow(rowp, d, row_head(rowp, d), t_c == 0, e0_c, tau_c, s_q[cur], &s_qcnt[cur],
                               ctx_of(row_c, tau_hi_c), true);
      }
      for (uint32_t i = tid; i < n; i += kThreads) {
        const uint2 e = s_q[cur][i];
        if ((e.x & kAbsMask) >= tau_hi_c) {
          add_vote(counter, packed, e.y, e.x >> 31);
          ++my_hi;
        } else {
          const uint32_t pos = atomicAdd(&s_bcnt[cur], 1u);
          if (pos < (uint32_t)kBandStage) s_b[cur][pos] = e;
          else band_direct(ctx_of(row_c, tau_hi_c), e.x, e.y);
        }
      }
      my_hi = __reduce_add_sync(0xFFFFFFFFu, my_hi);
      if (lane == 0 && my_hi) atomicAdd(&s_hi[cur], my_hi);
    }
    // ---- D: tile k-1's band buffer and vote count became final at this round's barrier
    uint32_t n1_final = 0;
    if (have1) {
      const uint32_t c = s_bcnt[p1];
      n1_final = c < (uint32_t)kBandStage ? c : (uint32_t)kBandStage;
    }
    uint32_t base1 = 0;
    if (tid == 0) {
      if (n1_final) base1 = atomicAdd(&rows[row1].n_cand, n1_final);
      if (have1 && s_hi[p1]) atomicAdd(&rows[row1].n_hi, s_hi[p1]);
      // buffers whose readers are all past this round's barrier: the queue of tile k-1 (drained a round
      // ago), the band buffer and vote count of tile k-2 (claimed a round ago, copied out by threads that
      // reach the next barrier before anyone refills it)
      s_qcnt[p1] = 0u;
      s_hi[p2] = 0u;
      s_bcnt[p2] = 0u;
    }
    n2 = n1_final; row2 = row1; base2 = base1;
    have1 = live; row1 = row_c;
  }
}

}  // namespace

cudaError_t launch_sample_and_filter(const uint32_t* gbits, const Layout& L, RowState* rows, uint2* cand, uint2* seg,
                                     uint32_t* hdr, uint32_t* hist, float* ef_err, float eta, int32_t* zero_counter,
                                     bool packed, bool band, cudaStream_t st) {
  // ef_err != NULL: gbits are the raw gradients g~, ef_err holds e and leaves holding g = g~ + eta * e
  // 128 KB of dynamic shared memory needs the opt-in on every device this runs on
  const size_t smem = (size_t)kSampleBins * sizeof(uint32_t);
  auto sample = ef_err ? sample_threshold_kernel<true> : sample_threshold_kernel<false>;
  static int opted[2][kMaxDevices];
  cudaError_t e = opt_in_dynamic_smem(reinterpret_cast<const void*>(sample), (int)smem, opted[ef_err ? 1 : 0]);
  if (e != cudaSuccess) return e;
  // clearing blocks: the SMs the M sampling blocks leave idle, and never fewer than 32
  unsigned n_clear = 0;
  if (zero_counter) {
    const unsigned used = (unsigned)L.M % (unsigned)sm_count();
    n_clear = (unsigned)sm_count() - used;
    if (n_clear < 32u) n_clear += (unsigned)sm_count();
  }
  e = launch_after(sample, dim3((unsigned)L.M + n_clear), dim3(1024), smem, st, gbits, L.d, rows, L.n_sample,
                   L.sample_stride, L.j_rank, band ? L.j_hi_rank : 0u, (uint32_t)L.K, hdr, hist, ef_err, eta, (uint32_t)L.M,
                   zero_counter, packed ? (L.d + 3) / 4 : L.d, packed ? kPackedZero : 0u);
  if (e != cudaSuccess) return e;
  prof_mark(kPhaseSampled, st);
  count_launch(2);
  const uint64_t n_work = (uint64_t)L.M * L.n_tiles;
  const uint64_t blocks = n_work < (uint64_t)sm_count() * 8 ? n_work : (uint64_t)sm_count() * 8;
  if (band) {                                    // (the caller asks for it only without error memory and with counters)
    constexpr int kBandThreads = 256;
    const uint64_t tiles = (uint64_t)L.M * ((L.d + kBandThreads * 32 - 1) / (kBandThreads * 32));
    const uint64_t resident = (uint64_t)sm_count() * (kBandThreadsPerSm / kBandThreads);
    return launch_after(filter_band_kernel<kBandThreads>, dim3((unsigned)(tiles < resident ? tiles : resident)),
                        dim3(kBandThreads), 0, st, gbits, L.M, L.d, rows, cand, L.cap, zero_counter, packed ? 1u : 0u);
  }
  const bool dense = L.dense;
  auto filter = dense ? (ef_err ? filter_scan_kernel<true> : filter_scan_kernel<false>)
                      : (ef_err ? filter_kernel<true> : filter_kernel<false>);
  return launch_after(filter, dim3((unsigned)blocks), dim3(kTileThreads), 0, st, gbits, L.M, L.d, rows, cand, L.cap, seg,
                      L.n_tiles, ef_err, eta);
}

}  // namespace s3gd

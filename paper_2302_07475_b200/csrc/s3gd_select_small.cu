// Selection of a row whose filtered candidates fit one SM's shared memory: one CTA per
// row does the three radix passes, the per-tile counts, their scan and the ordered
// emission without leaving the chip, so the chain of dependent global round trips that
// a sequence of small launches pays per pass is paid once.
//
// Same arithmetic as the general passes in s3gd_select.cu: MSB-first radix select on the
// 31 magnitude bits (11 + 10 + 10), then index-ordered emission tile by tile with the
// lowest-index rule for entries equal to the K-th magnitude (Eq. (3)-(4) plus the tie
// reading).  Rows it cannot take (no valid candidate list, or too many candidates) are
// left untouched for the general passes; rows it finishes are marked done.
#include "s3gd_common.cuh"

namespace s3gd {
namespace {

constexpr int kSmallThreads = 1024;
constexpr int kSmallWarps = kSmallThreads / 32;

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

__global__ void __launch_bounds__(kSmallThreads, 1)
select_small_kernel(RowState* __restrict__ rows, const uint2* __restrict__ cand, uint32_t cap,
                    const uint2* __restrict__ seg, uint32_t n_tiles, uint32_t* __restrict__ hdr, EmitOut o) {
  extern __shared__ __align__(16) unsigned char smem_raw[];
  __shared__ uint32_t s_hist[kHistBins];
  __shared__ uint32_t s_warp[kSmallWarps];
  __shared__ uint32_t s_sel[2];
  const uint32_t row = blockIdx.x, tid = threadIdx.x, lane = tid & 31, warp = tid >> 5, lt = lanemask_lt();
  const RowState rs = rows[row];
  if (!row_uses_candidates(rs, o.K, cap) || !fits_single_cta(rs.n_cand, n_tiles)) return;
  const uint32_t n = rs.n_cand;
  uint2* s_seg = reinterpret_cast<uint2*>(smem_raw);                 // [n_tiles] (position, count) of a tile's segment
  uint2* s_cnt = s_seg + n_tiles;                                    // [n_tiles] (#above, #equal) -> (output position, ties before)
  uint32_t* s_bits = reinterpret_cast<uint32_t*>(s_cnt + n_tiles);   // [n] bit patterns of the candidates
  const uint2* c = cand + (uint64_t)row * cap;
#pragma unroll 8
  for (uint32_t i = tid; i < n; i += kSmallThreads) s_bits[i] = c[i].x;
  for (uint32_t t = tid; t < n_tiles; t += kSmallThreads) s_seg[t] = seg[(uint64_t)row * n_tiles + t];

  // ---- radix select: tau = K-th largest magnitude, take = how many entries equal to tau are kept
  uint32_t prefix = 0, k_rem = o.K;
  const uint32_t n_round = (n + 31u) & ~31u;
  for (int pass = 0; pass < kNumPasses; ++pass) {
    const int nbins = 1 << pass_bits(pass);
    const uint32_t mask = (uint32_t)(nbins - 1);
    for (int b = tid; b < nbins; b += kSmallThreads) s_hist[b] = 0u;
    __syncthreads();                             // also: s_bits / s_seg are complete (first pass)
    for (uint32_t i = tid; i < n_round; i += kSmallThreads) {
      const uint32_t key = i < n ? (s_bits[i] & kAbsMask) : 0u;
      const bool on = i < n && (pass == 0 || (key >> pass_shift(pass - 1)) == prefix);
      const uint32_t digit = (key >> pass_shift(pass)) & mask;
      const uint32_t peers = __match_any_sync(0xFFFFFFFFu, on ? digit : 0xFFFFFFFFu);
      if (on && (peers & lt) == 0u) atomicAdd(&s_hist[digit], (uint32_t)__popc(peers));
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
    if (digit == 0xFFFFFFFFu) {                          // fewer than k_rem entries: cannot happen for a valid row
      if (tid == 0) atomicOr(hdr + kHdrStatus, (uint32_t)kFlagInternal);
      digit = 0u; a = 0u;
    }
    prefix = (prefix << pass_bits(pass)) | digit;
    k_rem -= a;
    __syncthreads();                             // s_sel and s_hist are reused by the next pass
  }
  const uint32_t tau = prefix, take = k_rem;

  // ---- per-tile counts (one warp per tile segment)
  for (uint32_t t = warp; t < n_tiles; t += kSmallWarps) {
    const uint2 sg = s_seg[t];
    uint32_t gt = 0, eq = 0;
    for (uint32_t i0 = 0; i0 < sg.y; i0 += 32) {
      const uint32_t i = i0 + lane;
      const uint32_t key = i < sg.y ? (s_bits[sg.x + i] & kAbsMask) : 0u;
      gt += __popc(__ballot_sync(0xFFFFFFFFu, i < sg.y && key > tau));
      eq += __popc(__ballot_sync(0xFFFFFFFFu, i < sg.y && key == tau));
    }
    if (lane == 0) s_cnt[t] = make_uint2(gt, eq);
  }
  __syncthreads();

  // ---- scan over the tiles in index order: (output position, ties before) per tile
  uint32_t carry_eq = 0, carry_out = 0;
  for (uint32_t base = 0; base < n_tiles; base += kSmallThreads) {
    const uint32_t t = base + tid;
    const uint2 v = t < n_tiles ? s_cnt[t] : make_uint2(0u, 0u);
    uint32_t tot_eq, tot_sel;
    const uint32_t run_eq = carry_eq + block_scan_excl_1024(v.y, s_warp, &tot_eq);
    const uint32_t room = run_eq < take ? take - run_eq : 0u;
    const uint32_t sel = v.x + (v.y < room ? v.y : room);
    const uint32_t out = carry_out + block_scan_excl_1024(sel, s_warp, &tot_sel);
    if (t < n_tiles) s_cnt[t] = make_uint2(out, run_eq);
    carry_eq += tot_eq;
    carry_out += tot_sel;
  }
  __syncthreads();
  if (tid == 0) {
    rows[row].tau = tau;
    rows[row].take_ties = take;
    rows[row].n_emitted = carry_out;
    rows[row].done = 1u;
    if (carry_out != o.K) {
      atomicAdd(hdr + kHdrBadCount, 1u);
      atomicOr(hdr + kHdrStatus, (uint32_t)kFlagInternal);
    }
    atomicMax(hdr + kHdrMaxCand, n);
  }

  // ---- ordered emission, in two sweeps so that no warp waits on a global load per tile.
  // Sweep 1 (one warp per tile segment, shared memory only): output position of every kept
  // entry, written over its bit pattern as (position << 1 | negative); sign-bit words by
  // ballot.  Entries that are not kept get the code kNotKept.
  constexpr uint32_t kNotKept = 0xFFFFFFFFu;
  for (uint32_t t = warp; t < n_tiles; t += kSmallWarps) {
    const uint2 sg = s_seg[t];
    if (sg.y == 0) continue;
    const uint2 sc = s_cnt[t];
    uint32_t run_out = sc.x, run_eq = sc.y;
    for (uint32_t i0 = 0; i0 < sg.y; i0 += 32) {
      const uint32_t i = i0 + lane;
      const bool in = i < sg.y;
      const uint32_t bits = in ? s_bits[sg.x + i] : 0u;
      const uint32_t key = bits & kAbsMask;
      const bool eq = in && key == tau;
      const uint32_t eqb = __ballot_sync(0xFFFFFFFFu, eq);
      const bool sel = in && (key > tau || (eq && run_eq + __popc(eqb & lt) < take));
      const uint32_t selb = __ballot_sync(0xFFFFFFFFu, sel);
      const uint32_t pos = run_out + __popc(selb & lt);
      const uint32_t neg = bits >> 31;
      const bool put = sel && pos < o.K;
      if (in) s_bits[sg.x + i] = put ? ((pos << 1) | neg) : kNotKept;
      if (o.signbits && selb) {
        const uint32_t w0 = run_out >> 5;
        const uint32_t bit = put ? (neg << (pos & 31)) : 0u;
        const uint32_t v0 = __reduce_or_sync(0xFFFFFFFFu, (pos >> 5) == w0 ? bit : 0u);
        const uint32_t v1 = __reduce_or_sync(0xFFFFFFFFu, (pos >> 5) == w0 + 1 ? bit : 0u);
        if (lane == 0) {
          if (v0) atomicOr(o.signbits + (uint64_t)row * o.words + w0, v0);
          if (v1) atomicOr(o.signbits + (uint64_t)row * o.words + w0 + 1, v1);
        }
      }
      run_out += __popc(selb);
      run_eq += __popc(eqb);
    }
  }
  __syncthreads();
  // Sweep 2 (flat over the candidate list): fetch the index of every kept entry and write it /
  // cast its vote.  The loads are independent, so many are in flight per thread.
  if (o.idx == nullptr && o.counter == nullptr) return;
#pragma unroll 4
  for (uint32_t i = tid; i < n; i += kSmallThreads) {
    const uint32_t code = s_bits[i];
    if (code != kNotKept) {
      const uint32_t idx = c[i].y;
      if (o.idx) o.idx[(uint64_t)row * o.K + (code >> 1)] = idx;
      if (o.counter) atomicAdd(o.counter + idx, (code & 1u) ? -1 : 1);
    }
  }
}

}  // namespace

cudaError_t launch_select_small(const Layout& L, RowState* rows, const uint2* cand, const uint2* seg, uint32_t* hdr,
                                const EmitOut& o, cudaStream_t st) {
  // enough dynamic shared memory for the largest row this kernel accepts
  uint64_t need = (uint64_t)L.cap * 4u + (uint64_t)L.n_tiles * 16u;
  if (need > kSmallSelectBytes) need = kSmallSelectBytes;
  if ((uint64_t)L.n_tiles * 16u > need) return cudaSuccess;      // not even the tile tables fit: nothing to do here
  cudaError_t e = cudaFuncSetAttribute(select_small_kernel, cudaFuncAttributeMaxDynamicSharedMemorySize,
                                       (int)kSmallSelectBytes);
  if (e != cudaSuccess) return e;
  select_small_kernel<<<L.M, kSmallThreads, (size_t)need, st>>>(rows, cand, L.cap, seg, L.n_tiles, hdr, o);
  e = cudaGetLastError();
  if (e == cudaSuccess) count_launch();
  return e;
}

}  // namespace s3gd

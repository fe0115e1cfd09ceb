// Second half of s3gd_select.cu: per-tile counts and their scan, the ordered emission,
// and the host-side sequencing of the whole selection.
namespace s3gd {
namespace {

// ------------------------------------------------------------ per-tile counts
// cnt[row][tile] = (#entries above tau, #entries equal to tau) in that tile.
// candidates: one warp per tile segment
__device__ __forceinline__ void count_cand(const uint2* __restrict__ cand, uint32_t cap, const uint2* __restrict__ seg,
                                           uint32_t n_tiles, const RowState& rs, uint32_t row, uint32_t bx,
                                           uint32_t gx, uint2* __restrict__ cnt) {
  const uint32_t lane = threadIdx.x & 31;
  const uint32_t warps = gx * (kSelThreads >> 5);
  const uint2* c = cand + (uint64_t)row * cap;
  const uint2* sgp = seg + (uint64_t)row * n_tiles;
  uint32_t t = bx * (kSelThreads >> 5) + (threadIdx.x >> 5);
  uint2 sg_next = t < n_tiles ? sgp[t] : make_uint2(0u, 0u);
  for (; t < n_tiles; t += warps) {
    const uint2 sg = sg_next;
    if (t + warps < n_tiles) sg_next = sgp[t + warps];        // next tile's segment is on its way meanwhile
    uint32_t gt = 0, eq = 0;
    for (uint32_t i0 = 0; i0 < sg.y; i0 += 128) {             // four 32-entry loads in flight
      uint32_t key[4];
#pragma unroll
      for (int u = 0; u < 4; ++u) {
        const uint32_t i = i0 + u * 32 + lane;
        key[u] = i < sg.y ? (c[sg.x + i].x & kAbsMask) : 0u;
      }
#pragma unroll
      for (int u = 0; u < 4; ++u) {
        const bool in = i0 + u * 32 + lane < sg.y;
        gt += __popc(__ballot_sync(0xFFFFFFFFu, in && key[u] > rs.tau));
        eq += __popc(__ballot_sync(0xFFFFFFFFu, in && key[u] == rs.tau));
      }
    }
    if (lane == 0) cnt[(uint64_t)row * n_tiles + t] = make_uint2(gt, eq);
  }
}

// whole row: one CTA per tile
__device__ __forceinline__ void count_row(const uint32_t* __restrict__ gbits, uint64_t d, uint32_t n_tiles,
                                          const RowState& rs, uint32_t row, uint32_t bx, uint32_t gx,
                                          uint2* __restrict__ cnt, uint32_t* s_gt, uint32_t* s_eq) {
  const uint32_t* rowp = gbits + (uint64_t)row * d;
  const uint32_t head = row_head(rowp, d);
  const uint32_t warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
  for (uint32_t t = bx; t < n_tiles; t += gx) {
    Tile T;
    load_tile(T, rowp, d, head, t);
    uint32_t gt = 0, eq = 0;
    if (T.head_valid) {
      const uint32_t key = T.head_bits & kAbsMask;
      gt += key > rs.tau; eq += key == rs.tau;
    }
#pragma unroll
    for (int it = 0; it < kTileIters; ++it) {
#pragma unroll
      for (int q = 0; q < 4; ++q) {
        const uint32_t key = T.bits[it][q] & kAbsMask;
        const uint32_t ok = T.valid[it] >> q & 1u;
        gt += ok & (uint32_t)(key > rs.tau);
        eq += ok & (uint32_t)(key == rs.tau);
      }
    }
#pragma unroll
    for (int s = 16; s > 0; s >>= 1) {
      gt += __shfl_xor_sync(0xFFFFFFFFu, gt, s);
      eq += __shfl_xor_sync(0xFFFFFFFFu, eq, s);
    }
    __syncthreads();
    if (lane == 0) { s_gt[warp] = gt; s_eq[warp] = eq; }
    __syncthreads();
    if (threadIdx.x == 0) {
      uint32_t a = 0, b = 0;
      for (int w = 0; w < kWarpsPerTile; ++w) { a += s_gt[w]; b += s_eq[w]; }
      cnt[(uint64_t)row * n_tiles + t] = make_uint2(a, b);
    }
  }
}

// ------------------------------------------------------------------- scan
// One block per row (the last one to finish counting).  In: cnt[tile] = (gt, eq).  Out, in
// place: (first output position of the tile, number of entries equal to tau in earlier
// tiles).  A tile keeps all its entries above tau, and of its entries equal to tau those
// whose running number (in index order over the whole row) is below take_ties.
__device__ __forceinline__ uint32_t block_exclusive_scan(uint32_t v, uint32_t* s_warp, uint32_t* total) {
  const uint32_t lane = threadIdx.x & 31, warp = threadIdx.x >> 5;
  uint32_t inc = v;
#pragma unroll
  for (int s = 1; s < 32; s <<= 1) {
    const uint32_t o = __shfl_up_sync(0xFFFFFFFFu, inc, s);
    if (lane >= (uint32_t)s) inc += o;
  }
  __syncthreads();
  if (lane == 31) s_warp[warp] = inc;
  __syncthreads();
  uint32_t off = 0, tot = 0;
#pragma unroll
  for (int w = 0; w < kSelThreads / 32; ++w) {
    const uint32_t c = s_warp[w];
    if ((uint32_t)w < warp) off += c;
    tot += c;
  }
  *total = tot;
  return off + inc - v;
}

__device__ __forceinline__ void scan_row(uint2* __restrict__ c, uint32_t n_tiles, RowState* __restrict__ rows,
                                         uint32_t row, uint32_t K, uint32_t cap, uint32_t* __restrict__ hdr,
                                         uint32_t* s_warp) {
  constexpr int kPer = 8;                            // consecutive tiles per thread and round
  const uint32_t tid = threadIdx.x;
  const uint32_t take = __ldcg(&rows[row].take_ties);
  uint32_t carry_eq = 0, carry_out = 0;
  for (uint32_t base = 0; base < n_tiles; base += kSelThreads * kPer) {
    const uint32_t t0 = base + tid * kPer;
    uint2 v[kPer];
#pragma unroll
    for (int q = 0; q < kPer; ++q) v[q] = t0 + q < n_tiles ? __ldcg(&c[t0 + q]) : make_uint2(0u, 0u);
    uint32_t eq_sum = 0;
#pragma unroll
    for (int q = 0; q < kPer; ++q) eq_sum += v[q].y;
    uint32_t tot_eq, tot_sel;
    uint32_t run_eq = carry_eq + block_exclusive_scan(eq_sum, s_warp, &tot_eq);
    const uint32_t eq0 = run_eq;
    uint32_t sel_sum = 0;
#pragma unroll
    for (int q = 0; q < kPer; ++q) {
      const uint32_t room = run_eq < take ? take - run_eq : 0u;
      sel_sum += v[q].x + (v[q].y < room ? v[q].y : room);
      run_eq += v[q].y;
    }
    uint32_t out = carry_out + block_exclusive_scan(sel_sum, s_warp, &tot_sel);
    run_eq = eq0;
#pragma unroll
    for (int q = 0; q < kPer; ++q) {
      const uint32_t room = run_eq < take ? take - run_eq : 0u;
      if (t0 + q < n_tiles) c[t0 + q] = make_uint2(out, run_eq);
      out += v[q].x + (v[q].y < room ? v[q].y : room);
      run_eq += v[q].y;
    }
    carry_eq += tot_eq;
    carry_out += tot_sel;
  }
  if (tid == 0) {
    const RowState rs = load_row_state<true>(rows + row);
    rows[row].n_emitted = carry_out;
    if (carry_out != K) {
      atomicAdd(hdr + kHdrBadCount, 1u);
      atomicOr(hdr + kHdrStatus, (uint32_t)kFlagInternal);
    }
    if (!row_uses_candidates(rs, K, cap)) atomicAdd(hdr + kHdrExactRows, 1u);
    atomicMax(hdr + kHdrMaxCand, rs.n_cand);
  }
}

// One (virtual) block of the counting pass; the last block of a row scans the row's counts.
template <bool kFromL2>
__device__ __forceinline__ void count_scan_block(const uint32_t* __restrict__ gbits, uint64_t d, uint32_t n_tiles,
                                                 const uint2* __restrict__ cand, uint32_t cap,
                                                 const uint2* __restrict__ seg, RowState* __restrict__ rows,
                                                 uint32_t K, uint2* __restrict__ cnt, uint32_t* __restrict__ hdr,
                                                 uint32_t gx_c, uint32_t bx, uint32_t row, uint32_t gx,
                                                 uint32_t want_done = 0u) {
  __shared__ uint32_t s_gt[kWarpsPerTile], s_eq[kWarpsPerTile], s_warp[kSelThreads / 32];
  __shared__ uint32_t s_flag;
  const RowState rs = load_row_state<kFromL2>(rows + row);
  if (rs.done != want_done) return;                  // 0: rows still open; kRowTwoPass: rows of the two-pass form
  const bool use_c = row_uses_candidates(rs, K, cap);
  const bool is_c = bx < gx_c;
  if (is_c && use_c) count_cand(cand, cap, seg, n_tiles, rs, row, bx, gx_c, cnt);
  else if (!is_c && !use_c) count_row(gbits, d, n_tiles, rs, row, bx - gx_c, gx - gx_c, cnt, s_gt, s_eq);
  if (last_block_of_row(&rows[row].ticket_count, gx, &s_flag))
    scan_row(cnt + (uint64_t)row * n_tiles, n_tiles, rows, row, K, cap, hdr, s_warp);
}

// ------------------------------------------------------------------- emit

// candidates: one warp per tile segment, 32 entries per step.  Sign bits of the (at most
// two) output words a step touches are gathered with a warp OR-reduction and merged
// into the zeroed output with one atomic per word.
__device__ __forceinline__ void emit_cand(const uint2* __restrict__ cand, uint32_t cap, const uint2* __restrict__ seg,
                                          const uint2* __restrict__ scan, uint32_t n_tiles, const RowState& rs,
                                          uint32_t row, uint32_t bx, uint32_t gx, const EmitOut& o) {
  const uint32_t lane = threadIdx.x & 31, lt = lanemask_lt();
  const uint32_t warps = gx * (kSelThreads >> 5);
  const uint2* c = cand + (uint64_t)row * cap;
  const uint2* sgp = seg + (uint64_t)row * n_tiles;
  const uint2* scp = scan + (uint64_t)row * n_tiles;
  uint32_t t = bx * (kSelThreads >> 5) + (threadIdx.x >> 5);
  uint2 sg_next = make_uint2(0u, 0u), sc_next = make_uint2(0u, 0u);
  if (t < n_tiles) { sg_next = sgp[t]; sc_next = scp[t]; }
  for (; t < n_tiles; t += warps) {
    const uint2 sg = sg_next, sc = sc_next;
    if (t + warps < n_tiles) { sg_next = sgp[t + warps]; sc_next = scp[t + warps]; }   // in flight meanwhile
    uint32_t run_out = sc.x, run_eq = sc.y;
    for (uint32_t i0 = 0; i0 < sg.y; i0 += 128) {             // four 32-entry loads in flight
      uint2 ent[4];
#pragma unroll
      for (int u = 0; u < 4; ++u) {
        const uint32_t i = i0 + u * 32 + lane;
        ent[u] = i < sg.y ? c[sg.x + i] : make_uint2(0u, 0u);
      }
#pragma unroll
      for (int u = 0; u < 4; ++u) {
        if (i0 + u * 32 >= sg.y) break;                        // warp-uniform
        const bool in = i0 + u * 32 + lane < sg.y;
        const uint2 e = ent[u];
        const uint32_t key = e.x & kAbsMask;
        const bool eq = in && key == rs.tau;
        const uint32_t eqb = __ballot_sync(0xFFFFFFFFu, eq);
        const bool sel = in && (key > rs.tau || (eq && run_eq + __popc(eqb & lt) < rs.take_ties));
        const uint32_t selb = __ballot_sync(0xFFFFFFFFu, sel);
        const uint32_t pos = run_out + __popc(selb & lt);
        const uint32_t neg = e.x >> 31;
        if (sel && pos < o.K) {
          if (o.idx) o.idx[(uint64_t)row * o.K + pos] = e.y;
          if (o.counter) add_vote(o.counter, o.packed, e.y, neg);
          if (o.err) o.err[(uint64_t)row * o.d + e.y] = 0.f;
        }
        if (o.signbits && selb) {
          const uint32_t w0 = run_out >> 5;
          const uint32_t bit = (sel && pos < o.K) ? (neg << (pos & 31)) : 0u;
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
  }
}

// whole row: one CTA per tile; two ordered rankings (ties, then kept entries)
__device__ __forceinline__ void emit_row(const uint32_t* __restrict__ gbits, uint64_t d, uint32_t n_tiles,
                                         const uint2* __restrict__ scan, const RowState& rs, uint32_t row,
                                         uint32_t bx, uint32_t gx, const EmitOut& o, uint32_t* s_wtot) {
  const uint32_t* rowp = gbits + (uint64_t)row * d;
  const uint32_t head = row_head(rowp, d);
  const uint32_t lane = threadIdx.x & 31;
  for (uint32_t t = bx; t < n_tiles; t += gx) {
    const uint2 sc = scan[(uint64_t)row * n_tiles + t];
    Tile T;
    load_tile(T, rowp, d, head, t);
    uint32_t eqf[kTileIters], gtf[kTileIters];
#pragma unroll
    for (int it = 0; it < kTileIters; ++it) {
      uint32_t e = 0, g = 0;
#pragma unroll
      for (int q = 0; q < 4; ++q) {
        uint32_t key = T.bits[it][q] & kAbsMask;
        e |= (uint32_t)(key == rs.tau) << q;
        g |= (uint32_t)(key > rs.tau) << q;
      }
      eqf[it] = e & T.valid[it];
      gtf[it] = g & T.valid[it];
    }
    const uint32_t hkey = T.head_bits & kAbsMask;
    const bool head_eq = T.head_valid && hkey == rs.tau;
    TileRanks Re;
    tile_ranks(Re, eqf, head_eq, s_wtot);
    // kept = above tau, or equal to tau with a running tie number below take_ties
    uint32_t self[kTileIters];
#pragma unroll
    for (int it = 0; it < kTileIters; ++it) {
      uint32_t s = gtf[it];
#pragma unroll
      for (int q = 0; q < 4; ++q)
        if ((eqf[it] >> q & 1u) && sc.y + rank_of(Re, eqf, it, q) < rs.take_ties) s |= 1u << q;
      self[it] = s;
    }
    const bool head_sel = T.head_valid && (hkey > rs.tau || (head_eq && sc.y + Re.head_rank < rs.take_ties));
    // Band form of the filter pass: every entry at or above tau_hi has voted there already.  This route
    // is the one that redoes such a row, so the kept ones among them do not vote again and the others
    // take their vote back (an opposite vote; the counters are sums).
    const bool prevoted = o.counter != nullptr && rs.tau_hi != kNoPrevote;     // the same for the whole row
    if (prevoted) {
      if (T.head_valid && hkey >= rs.tau_hi && !head_sel) add_vote(o.counter, o.packed, lane, (T.head_bits >> 31) ^ 1u);
#pragma unroll
      for (int it = 0; it < kTileIters; ++it) {
#pragma unroll
        for (int q = 0; q < 4; ++q) {
          const uint32_t b = T.bits[it][q];
          if ((T.valid[it] >> q & 1u) && (b & kAbsMask) >= rs.tau_hi && !(self[it] >> q & 1u))
            add_vote(o.counter, o.packed, (uint32_t)(T.first(it) + q), (b >> 31) ^ 1u);
        }
      }
    }
    TileRanks Rs;
    tile_ranks(Rs, self, head_sel, s_wtot);
    if (Rs.tile_total == 0) continue;
    if (head_sel) {
      const uint32_t pos = sc.x + Rs.head_rank;
      const uint32_t neg = T.head_bits >> 31;
      if (pos < o.K) {
        if (o.idx) o.idx[(uint64_t)row * o.K + pos] = lane;
        if (o.counter && !(prevoted && hkey >= rs.tau_hi)) add_vote(o.counter, o.packed, lane, neg);
        if (o.err) o.err[(uint64_t)row * o.d + lane] = 0.f;
        if (o.signbits && neg) atomicOr(o.signbits + (uint64_t)row * o.words + (pos >> 5), 1u << (pos & 31));
      }
    }
#pragma unroll
    for (int it = 0; it < kTileIters; ++it) {
      const uint32_t cnt_it = __reduce_add_sync(0xFFFFFFFFu, (uint32_t)__popc(self[it]));
      if (cnt_it == 0) continue;                  // warp-uniform
      const uint32_t p0 = sc.x + Rs.warp_off + Rs.it_off[it];   // first output position of this warp-iteration
      uint32_t mybits[5] = {0u, 0u, 0u, 0u, 0u};   // sign bits of my entries, by output word relative to p0 >> 5
#pragma unroll
      for (int q = 0; q < 4; ++q) {
        if (self[it] >> q & 1u) {
          const uint32_t pos = sc.x + rank_of(Rs, self, it, q);
          if (pos < o.K) {
            const uint32_t n = (uint32_t)(T.first(it) + q);
            const uint32_t neg = T.bits[it][q] >> 31;
            if (o.idx) o.idx[(uint64_t)row * o.K + pos] = n;
            if (o.counter && !(prevoted && (T.bits[it][q] & kAbsMask) >= rs.tau_hi)) add_vote(o.counter, o.packed, n, neg);
            if (o.err) o.err[(uint64_t)row * o.d + n] = 0.f;
            const uint32_t rel = (pos >> 5) - (p0 >> 5);      // 0..4: at most 128 entries per warp-iteration
#pragma unroll
            for (int w = 0; w < 5; ++w)
              if (rel == (uint32_t)w) mybits[w] |= neg << (pos & 31);
          }
        }
      }
      if (o.signbits) {
        const uint32_t n_words = ((p0 + cnt_it - 1) >> 5) - (p0 >> 5) + 1;
#pragma unroll
        for (int w = 0; w < 5; ++w) {
          if ((uint32_t)w < n_words) {
            const uint32_t v = __reduce_or_sync(0xFFFFFFFFu, mybits[w]);
            if (lane == 0 && v) atomicOr(o.signbits + (uint64_t)row * o.words + (p0 >> 5) + w, v);
          }
        }
      }
    }
  }
}

// One (virtual) block of the emission.
template <bool kFromL2>
__device__ __forceinline__ void emit_block(const uint32_t* __restrict__ gbits, uint64_t d, uint32_t n_tiles,
                                           const uint2* __restrict__ cand, uint32_t cap, const uint2* __restrict__ seg,
                                           const uint2* __restrict__ scan, const RowState* __restrict__ rows,
                                           const EmitOut& o, uint32_t gx_c, uint32_t bx, uint32_t row, uint32_t gx,
                                           uint32_t want_done = 0u) {
  __shared__ uint32_t s_wtot[kWarpsPerTile + 1];
  const RowState rs = load_row_state<kFromL2>(rows + row);
  if (rs.done != want_done) return;
  const bool use_c = row_uses_candidates(rs, o.K, cap);
  const bool is_c = bx < gx_c;
  if (is_c && use_c) emit_cand(cand, cap, seg, scan, n_tiles, rs, row, bx, gx_c, o);
  else if (!is_c && !use_c) emit_row(gbits, d, n_tiles, scan, rs, row, bx - gx_c, gx - gx_c, o, s_wtot);
}

// The passes as launches of their own, grid (gx, M): used when the general passes carry the
// selection of every row, where more resident blocks and per-pass register budgets pay.
__global__ void __launch_bounds__(kSelThreads, 6) hist_pick_kernel(const uint32_t* __restrict__ gbits, uint64_t d,
                                                                   uint32_t n_tiles, const uint2* __restrict__ cand,
                                                                   uint32_t cap, RowState* __restrict__ rows, uint32_t K,
                                                                   uint32_t* __restrict__ hist,
                                                                   uint32_t* __restrict__ hdr, int pass, uint32_t gx_c) {
  hist_pick_block<false>(gbits, d, n_tiles, cand, cap, rows, K, hist, hdr, pass, gx_c, blockIdx.x, blockIdx.y, gridDim.x);
}

__global__ void __launch_bounds__(kSelThreads, 6) count_scan_kernel(const uint32_t* __restrict__ gbits, uint64_t d,
                                                                    uint32_t n_tiles, const uint2* __restrict__ cand,
                                                                    uint32_t cap, const uint2* __restrict__ seg,
                                                                    RowState* __restrict__ rows, uint32_t K,
                                                                    uint2* __restrict__ cnt, uint32_t* __restrict__ hdr,
                                                                    uint32_t gx_c, uint32_t want_done) {
  count_scan_block<false>(gbits, d, n_tiles, cand, cap, seg, rows, K, cnt, hdr, gx_c, blockIdx.x, blockIdx.y, gridDim.x,
                          want_done);
}

__global__ void __launch_bounds__(kSelThreads, 6) hist_two_pass_kernel(const uint2* __restrict__ cand, uint32_t cap,
                                                                       RowState* __restrict__ rows, uint32_t K,
                                                                       uint32_t* __restrict__ hist,
                                                                       uint32_t* __restrict__ hdr, int pass,
                                                                       uint2* __restrict__ bin, uint32_t bin_cap,
                                                                       EmitOut o, bool band) {
  grid_dependency_wait();                          // (launched with launch_after)
  hist_two_pass_block(cand, cap, rows, K, hist, hdr, pass, blockIdx.x, blockIdx.y, gridDim.x, bin, bin_cap, o, band);
}

__global__ void __launch_bounds__(kSelThreads, 5) emit_kernel(const uint32_t* __restrict__ gbits, uint64_t d,
                                                              uint32_t n_tiles, const uint2* __restrict__ cand,
                                                              uint32_t cap, const uint2* __restrict__ seg,
                                                              const uint2* __restrict__ scan,
                                                              const RowState* __restrict__ rows, EmitOut o,
                                                              uint32_t gx_c, uint32_t want_done) {
  emit_block<false>(gbits, d, n_tiles, cand, cap, seg, scan, rows, o, gx_c, blockIdx.x, blockIdx.y, gridDim.x,
                    want_done);
}

// The same passes as ONE cooperative launch -- three histogram passes, the counting pass and the
// emission, separated by grid-wide barriers -- for the case in which the single-CTA selection is
// expected to finish every row.  The kernel then finds nothing to do and returns at once: a step
// in which every row stays on the fast route pays for one empty launch, not five.  If rows are
// left over, the resident blocks take the virtual blocks of each pass in turn; this is slower
// per row than the separate launches (fewer blocks, one register budget for all passes) and is
// only meant for the odd row.
struct GeneralArgs {
  const uint32_t* gbits;
  uint64_t d;
  uint32_t n_tiles;
  const uint2* cand;
  uint32_t cap;
  const uint2* seg;
  uint2* cnt;
  RowState* rows;
  uint32_t K;
  uint32_t* hist;
  uint32_t* hdr;
  EmitOut o;
  uint32_t M, gx_hist_c, gx_tile_c, gx_r;
};

__global__ void __launch_bounds__(kSelThreads, 4) general_passes_kernel(const GeneralArgs a) {
  cooperative_groups::grid_group grid = cooperative_groups::this_grid();
  // written by the previous launch, read-only here: every block takes the same branch
  if (__ldcg(a.hdr + kHdrRowsDone) == a.M) return;
  {
    const uint32_t gx = a.gx_hist_c + a.gx_r, nvb = gx * a.M;
    for (int pass = 0; pass < kNumPasses; ++pass) {
      for (uint32_t vb = blockIdx.x; vb < nvb; vb += gridDim.x) {
        hist_pick_block<true>(a.gbits, a.d, a.n_tiles, a.cand, a.cap, a.rows, a.K, a.hist, a.hdr, pass, a.gx_hist_c,
                        vb % gx, vb / gx, gx);
        __syncthreads();
      }
      grid.sync();
    }
  }
  const uint32_t gx = a.gx_tile_c + a.gx_r, nvb = gx * a.M;
  for (uint32_t vb = blockIdx.x; vb < nvb; vb += gridDim.x) {
    count_scan_block<true>(a.gbits, a.d, a.n_tiles, a.cand, a.cap, a.seg, a.rows, a.K, a.cnt, a.hdr, a.gx_tile_c, vb % gx,
                     vb / gx, gx);
    __syncthreads();
  }
  grid.sync();
  for (uint32_t vb = blockIdx.x; vb < nvb; vb += gridDim.x) {
    emit_block<true>(a.gbits, a.d, a.n_tiles, a.cand, a.cap, a.seg, a.cnt, a.rows, a.o, a.gx_tile_c, vb % gx, vb / gx, gx);
    __syncthreads();
  }
}

inline unsigned clampu(uint64_t v, uint64_t lo, uint64_t hi) { return (unsigned)(v < lo ? lo : (v > hi ? hi : v)); }

}  // namespace

bool select_clears_counter(const Layout& L) { return L.cap > 0; }   // the sampling launch does it

cudaError_t launch_select(const float* grads, const Layout& L, void* ws, uint32_t* out_idx, uint32_t* out_signbits,
                          int32_t* counter, bool packed, float* err_to_clear, const float* ef_raw, float eta,
                          cudaStream_t st) {
  char* base = static_cast<char*>(ws);
  uint32_t* hdr = reinterpret_cast<uint32_t*>(base + L.off_hdr);
  RowState* rows = reinterpret_cast<RowState*>(base + L.off_rows);
  uint32_t* hist = reinterpret_cast<uint32_t*>(base + L.off_hist);
  uint2* seg = reinterpret_cast<uint2*>(base + L.off_seg);
  uint2* cnt = reinterpret_cast<uint2*>(base + L.off_segscan);
  uint2* cand = reinterpret_cast<uint2*>(base + L.off_cand);
  const uint32_t* gbits = reinterpret_cast<const uint32_t*>(grads);
  const uint32_t K = (uint32_t)L.K;
  const bool use_filter = L.cap > 0;
  const int M = L.M;
#define S3GD_CHECK_LAUNCH()                         \
  do {                                              \
    cudaError_t e_ = cudaGetLastError();            \
    if (e_ != cudaSuccess) return e_;               \
    count_launch();                                 \
  } while (0)

  EmitOut o;
  o.idx = out_idx; o.signbits = out_signbits; o.counter = counter; o.packed = packed ? 1u : 0u;
  o.err = err_to_clear; o.d = L.d; o.unordered = 0u;
  o.K = K; o.words = (uint32_t)((L.K + 31) / 32);
  // Rows whose candidates fit one SM are finished by one CTA each; if only the votes are wanted and a
  // typical row needs the shared memory of up to four SMs, by a cluster of CTAs each.
  const bool votes_only = counter != nullptr && out_idx == nullptr && out_signbits == nullptr;
  // (With error compensation the residuals pile up just below the threshold; the sampler places tau_lo
  // inside its histogram bin there, which keeps the rows at the sampling estimate.)
  uint32_t cluster = 0u;
  if (use_filter && votes_only && !fits_single_cta(L.typical_cand)) cluster = cluster_size_for(L.typical_cand);
  // If a row's candidates are expected to fit an on-chip selection, the general passes only serve the
  // odd row that did not fit or fell back to the whole-row route.
  const bool only_fallback = use_filter && (fits_single_cta(L.typical_cand) || cluster != 0u);
  // With error compensation rows do run past the estimate (measured: the single launch then took
  // 1.07 ms where the five launches take 0.17 ms), so that mode keeps the five launches.
  // Where the general passes carry the selection of candidate rows, those rows take the two-pass form
  // first (two histogram launches instead of three, candidate blocks only); the single launch after it
  // does whatever is left -- rows on the whole-row route, rows whose K-th magnitude lies more than a
  // quarter octave above tau_lo -- and otherwise returns at once.
  const bool two_pass = use_filter && !only_fallback && err_to_clear == nullptr;
  // Only the votes wanted: the band form of the filter pass (s3gd_filter.cu), whose lists are unordered.
  // Every selection that follows either needs no order (the on-chip ones, the bin route of the two-pass
  // form) or sends the row to the whole-row route.
  const bool band = use_filter && votes_only && err_to_clear == nullptr;
  // (a row too long for the on-chip selection still has the two-pass form to go to, if that follows)
  o.unordered = band && only_fallback ? 1u : 0u;

  if (use_filter) {
    cudaError_t e = ef_raw ? launch_sample_and_filter(reinterpret_cast<const uint32_t*>(ef_raw), L, rows, cand, seg,
                                                      hdr, hist, err_to_clear, eta, counter, packed, false, st)
                           : launch_sample_and_filter(gbits, L, rows, cand, seg, hdr, hist, nullptr, 0.f, counter, packed,
                                                      band, st);
    if (e != cudaSuccess) return e;
  } else {
    init_kernel<<<clampu(((uint64_t)M * kHistBins + 255) / 256, 1, sm_count() * 4), 256, 0, st>>>(hdr, rows, hist, M, K, 1u);
    S3GD_CHECK_LAUNCH();
    prof_mark(kPhaseSampled, st);
  }
  prof_mark(kPhaseFiltered, st);
  if (use_filter && (cluster != 0u || fits_single_cta(K))) {    // a candidate row has at least K candidates
    cudaError_t e = cluster ? launch_select_cluster(L, rows, cand, hdr, o, cluster, st)
                            : launch_select_small(L, rows, cand, seg, hdr, o, st);
    if (e != cudaSuccess) return e;
  }
  // Blocks per row (each block strides over its row's candidates or tiles).  Launches that only
  // serve the odd row normally exit at once: keep them small.  Otherwise they carry the selection
  // of all rows: about eight CTAs per SM.
  const uint32_t per_row = (uint32_t)(((uint64_t)sm_count() * (only_fallback ? 4 : 8) + M - 1) / M);
  const uint32_t gx_hist_c = use_filter ? clampu(((uint64_t)L.cap + 4095) / 4096, 1, only_fallback ? per_row : 64) : 0u;
  // the sweeps of the two-pass form: all rows' blocks resident at once (six per SM), each with a longer
  // run of candidates -- their per-block costs (row state, barriers, the ticket) weigh more than tail
  // effects (resnet50 shape at K = 1 %: 64 blocks per row 0.826 ms, 27 per row 0.812 ms)
  const uint32_t gx_two = clampu(((uint64_t)L.cap + 4095) / 4096, 1, clampu((uint64_t)sm_count() * 6 / M, 8, 64));
  const uint32_t gx_tile_c = use_filter ? clampu(((uint64_t)L.n_tiles + 7) / 8, 1, per_row) : 0u;
  const uint32_t gx_r = clampu(L.n_tiles, 1, per_row);
  if (two_pass) {
    // bin lists only where the votes alone are wanted (the message needs positions)
    uint2* bin = reinterpret_cast<uint2*>(base + L.off_bin);
    const uint32_t bin_cap = band ? L.bin_cap : 0u;
    for (int pass = 0; pass <= 2; pass += 2) {
      cudaError_t e = launch_after(hist_two_pass_kernel, dim3(gx_two, M), dim3(kSelThreads), 0, st, cand, L.cap, rows, K, hist,
                                   hdr, pass, bin, bin_cap, o, band);
      if (e != cudaSuccess) return e;
      count_launch();
    }
    prof_mark(kPhaseThreshold, st);
    if (bin_cap) {
      cudaError_t e = launch_select_bin(L, rows, bin, bin_cap, hdr, o, st);
      if (e != cudaSuccess) return e;
    }
    if (!band) {                  // (the band form's lists are unordered: every row's bin goes to the bin selection)
      count_scan_kernel<<<dim3(gx_tile_c, M), kSelThreads, 0, st>>>(gbits, L.d, L.n_tiles, cand, L.cap, seg, rows, K, cnt,
                                                                    hdr, gx_tile_c, kRowTwoPass);
      S3GD_CHECK_LAUNCH();
      emit_kernel<<<dim3(gx_tile_c, M), kSelThreads, 0, st>>>(gbits, L.d, L.n_tiles, cand, L.cap, seg, cnt, rows, o,
                                                              gx_tile_c, kRowTwoPass);
      S3GD_CHECK_LAUNCH();
    }
  }
  if ((only_fallback || two_pass) && err_to_clear == nullptr) {
    // as many blocks as can be resident together, and no more than the largest pass has virtual blocks
    // (the occupancy of a kernel is a property of the device: asked once per device, and two threads
    //  that ask at the same time store the same number)
    static int occupancy[kMaxDevices];
    int dev = 0;
    if (cudaGetDevice(&dev) != cudaSuccess || dev < 0 || dev >= kMaxDevices) return cudaErrorInvalidDevice;
    int blocks_per_sm = __atomic_load_n(&occupancy[dev], __ATOMIC_RELAXED);
    if (blocks_per_sm == 0) {
      cudaError_t e = cudaOccupancyMaxActiveBlocksPerMultiprocessor(&blocks_per_sm, general_passes_kernel, kSelThreads, 0);
      if (e != cudaSuccess) return e;
      if (blocks_per_sm < 1) return cudaErrorLaunchOutOfResources;
      __atomic_store_n(&occupancy[dev], blocks_per_sm, __ATOMIC_RELAXED);
    }
    const int n_sm = sm_count();
    GeneralArgs ga;
    ga.gbits = gbits; ga.d = L.d; ga.n_tiles = L.n_tiles; ga.cand = cand; ga.cap = L.cap; ga.seg = seg; ga.cnt = cnt;
    ga.rows = rows; ga.K = K; ga.hist = hist; ga.hdr = hdr; ga.o = o; ga.M = (uint32_t)M;
    ga.gx_hist_c = gx_hist_c; ga.gx_tile_c = gx_tile_c; ga.gx_r = gx_r;
    const uint64_t most = (uint64_t)(gx_hist_c > gx_tile_c ? gx_hist_c : gx_tile_c) + gx_r;
    const unsigned grid = clampu(most * (uint64_t)M, 1, (uint64_t)blocks_per_sm * (uint64_t)n_sm);
    void* kargs[] = {&ga};
    cudaError_t ce = cudaLaunchCooperativeKernel(reinterpret_cast<void*>(general_passes_kernel), dim3(grid),
                                                 dim3(kSelThreads), kargs, 0, st);
    if (ce != cudaSuccess) return ce;
    count_launch();
    if (!two_pass) prof_mark(kPhaseThreshold, st);
  } else {
    for (int pass = 0; pass < kNumPasses; ++pass) {
      hist_pick_kernel<<<dim3(gx_hist_c + gx_r, M), kSelThreads, 0, st>>>(gbits, L.d, L.n_tiles, cand, L.cap, rows, K,
                                                                          hist, hdr, pass, gx_hist_c);
      S3GD_CHECK_LAUNCH();
    }
    prof_mark(kPhaseThreshold, st);
    count_scan_kernel<<<dim3(gx_tile_c + gx_r, M), kSelThreads, 0, st>>>(gbits, L.d, L.n_tiles, cand, L.cap, seg, rows,
                                                                         K, cnt, hdr, gx_tile_c, 0u);
    S3GD_CHECK_LAUNCH();
    emit_kernel<<<dim3(gx_tile_c + gx_r, M), kSelThreads, 0, st>>>(gbits, L.d, L.n_tiles, cand, L.cap, seg, cnt, rows, o,
                                                                   gx_tile_c, 0u);
    S3GD_CHECK_LAUNCH();
  }
#undef S3GD_CHECK_LAUNCH
  prof_mark(kPhaseEmitted, st);
  return cudaSuccess;
}

}  // namespace s3gd

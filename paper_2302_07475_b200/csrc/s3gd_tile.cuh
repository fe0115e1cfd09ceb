// One tile of one gradient row held in registers, and the ordered-rank machinery
// that every streaming kernel of the selection uses.
//
// A row of d fp32 values starts at an address that is only 4-byte aligned in
// general (d need not be a multiple of 4).  `head` = number of leading entries
// before the first 128-byte boundary (0..31).  Tile t covers the entries
// [head + t*kTileElems, head + (t+1)*kTileElems) with 16-byte loads, so every tile
// starts on a cache line; tile 0 also owns the `head` leading entries, which the
// low lanes of warp 0 load as scalars.
//
// Inside a tile warp w owns the contiguous 1024 entries starting at w*1024, and in
// iteration `it` lane l holds entries w*1024 + it*128 + l*4 + {0,1,2,3}.  So the
// ascending-index order of a tile is (head entries, then warp, iteration, lane, slot),
// and the rank of a flagged entry among all flagged entries of the tile follows from
// one packed warp scan plus the eight warp totals.
#pragma once

#include "s3gd_common.cuh"

namespace s3gd {

struct Tile {
  uint32_t bits[kTileIters][4];   // raw fp32 bit patterns
  uint32_t valid[kTileIters];     // low 4 bits: which of the 4 slots lie inside the row
  uint32_t head_bits;             // warp 0, lane < head of tile 0 only
  bool head_valid;
  uint64_t e0;                    // row index of this lane's slot 0 in iteration 0 (+128 per iteration)
  __device__ __forceinline__ uint64_t first(int it) const { return e0 + (uint64_t)it * 128; }
};

__device__ __forceinline__ uint32_t row_head(const uint32_t* rowp, uint64_t d) {
  uint32_t h = (uint32_t)(((128u - (uint32_t)(reinterpret_cast<uintptr_t>(rowp) & 127u)) & 127u) >> 2);
  return (uint64_t)h < d ? h : (uint32_t)d;
}

__device__ __forceinline__ void load_tile(Tile& T, const uint32_t* __restrict__ rowp, uint64_t d, uint32_t head,
                                          uint32_t t) {
  const uint32_t warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
  const uint64_t e0 = (uint64_t)head + (uint64_t)t * kTileElems + (uint64_t)warp * (kTileElems / kWarpsPerTile) +
                      (uint64_t)lane * 4;
  T.e0 = e0;
  if ((uint64_t)head + (uint64_t)(t + 1) * kTileElems <= d) {
#pragma unroll
    for (int it = 0; it < kTileIters; ++it) {
      uint4 v = ld_stream_v4(rowp + e0 + (uint64_t)it * 128);
      T.bits[it][0] = v.x; T.bits[it][1] = v.y; T.bits[it][2] = v.z; T.bits[it][3] = v.w;
      T.valid[it] = 0xFu;
    }
  } else {
#pragma unroll
    for (int it = 0; it < kTileIters; ++it) {
      const uint64_t e = e0 + (uint64_t)it * 128;
      if (e + 4 <= d) {
        uint4 v = ld_stream_v4(rowp + e);
        T.bits[it][0] = v.x; T.bits[it][1] = v.y; T.bits[it][2] = v.z; T.bits[it][3] = v.w;
        T.valid[it] = 0xFu;
      } else {
        T.valid[it] = 0u;
#pragma unroll
        for (int q = 0; q < 4; ++q) {
          T.bits[it][q] = 0u;
          if (e + q < d) {
            T.bits[it][q] = ld_stream_u32(rowp + e + q);
            T.valid[it] |= 1u << q;
          }
        }
      }
    }
  }
  T.head_valid = (t == 0 && warp == 0 && lane < head);
  T.head_bits = T.head_valid ? ld_stream_u32(rowp + lane) : 0u;
}

// Error compensation fused into the streaming pass (Eq. (5)): the tile holds g~; it becomes
// g = g~ + eta * e (product rounded, then sum rounded) and g is written to the error memory,
// where the later passes and Eq. (6) find it.  errp is the row of the error memory; it must
// be congruent to the gradient row modulo 16 bytes (the host checks) so that the same
// 16-byte accesses apply.  Done in halves of four iterations to bound the registers.
__device__ __forceinline__ uint32_t ef_value(uint32_t g_tilde_bits, float e, float eta) {
  return __float_as_uint(__fadd_rn(__uint_as_float(g_tilde_bits), __fmul_rn(eta, e)));
}

__device__ __forceinline__ void ef_materialise(Tile& T, float* __restrict__ errp, float eta) {
#pragma unroll
  for (int half = 0; half < kTileIters; half += 4) {
    float4 e[4];
#pragma unroll
    for (int i = 0; i < 4; ++i) {
      const int it = half + i;
      if (T.valid[it] == 0xFu) {
        e[i] = *reinterpret_cast<const float4*>(errp + T.first(it));
      } else {
        e[i] = make_float4(0.f, 0.f, 0.f, 0.f);
        if (T.valid[it] & 1u) e[i].x = errp[T.first(it)];
        if (T.valid[it] & 2u) e[i].y = errp[T.first(it) + 1];
        if (T.valid[it] & 4u) e[i].z = errp[T.first(it) + 2];
        if (T.valid[it] & 8u) e[i].w = errp[T.first(it) + 3];
      }
    }
#pragma unroll
    for (int i = 0; i < 4; ++i) {
      const int it = half + i;
      T.bits[it][0] = ef_value(T.bits[it][0], e[i].x, eta);
      T.bits[it][1] = ef_value(T.bits[it][1], e[i].y, eta);
      T.bits[it][2] = ef_value(T.bits[it][2], e[i].z, eta);
      T.bits[it][3] = ef_value(T.bits[it][3], e[i].w, eta);
      if (T.valid[it] == 0xFu) {
        *reinterpret_cast<uint4*>(errp + T.first(it)) =
            make_uint4(T.bits[it][0], T.bits[it][1], T.bits[it][2], T.bits[it][3]);
      } else {
#pragma unroll
        for (int q = 0; q < 4; ++q)
          if (T.valid[it] >> q & 1u) errp[T.first(it) + q] = __uint_as_float(T.bits[it][q]);
      }
    }
  }
  if (T.head_valid) {
    const uint32_t lane = threadIdx.x & 31;
    T.head_bits = ef_value(T.head_bits, errp[lane], eta);
    errp[lane] = __uint_as_float(T.head_bits);
  }
}

// Ranks of flagged entries in ascending-index order.
// flags[it] (low 4 bits) and head_flag mark entries; after the call
//   rank of (it, slot) = lane_excl(it) + popc(flags[it] & ((1u << slot) - 1))  + block offset of (warp, it)
// which rank_of() evaluates.  Uses s_wtot[kWarpsPerTile + 1] shared words; tile_ranks() is the
// two-barrier form, tile_ranks_publish()/tile_ranks_collect() let the caller own the barrier.
struct TileRanks {
  uint32_t lane_excl[kTileIters];  // flagged entries of this warp-iteration in lower lanes
  uint32_t it_off[kTileIters];     // flagged entries of this warp in earlier iterations
  uint32_t warp_off;               // flagged entries of earlier warps (and of the head)
  uint32_t head_rank;              // rank of this lane's head entry
  uint32_t tile_total;             // all flagged entries of the tile
};

// First half: per-warp packed scan; publishes this warp's total (and the head count) in
// s_wtot[0..kWarpsPerTile].  The caller places one block barrier between the halves.
__device__ __forceinline__ void tile_ranks_publish(TileRanks& R, const uint32_t (&flags)[kTileIters], bool head_flag,
                                                   uint32_t* s_wtot) {
  const uint32_t warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
  // counts are <= 4 per lane and <= 128 per warp-iteration, so the counts of four
  // iterations travel through the scan as the 8-bit fields of one word
  uint32_t lo = 0, hi = 0;
#pragma unroll
  for (int it = 0; it < 4; ++it) {
    lo |= (uint32_t)__popc(flags[it] & 0xFu) << (8 * it);
    hi |= (uint32_t)__popc(flags[it + 4] & 0xFu) << (8 * it);
  }
  uint32_t run = 0;
  if (__any_sync(0xFFFFFFFFu, (lo | hi) != 0u)) {
    uint32_t ilo = lo, ihi = hi;      // inclusive scans over lanes
#pragma unroll
    for (int s = 1; s < 32; s <<= 1) {
      uint32_t a = __shfl_up_sync(0xFFFFFFFFu, ilo, s);
      uint32_t b = __shfl_up_sync(0xFFFFFFFFu, ihi, s);
      if (lane >= (uint32_t)s) { ilo += a; ihi += b; }
    }
    // a full warp-iteration holds 128 flagged entries: 128 fits the 8-bit field (max 255)
    const uint32_t tlo = __shfl_sync(0xFFFFFFFFu, ilo, 31), thi = __shfl_sync(0xFFFFFFFFu, ihi, 31);
    const uint32_t elo = ilo - lo, ehi = ihi - hi;
#pragma unroll
    for (int it = 0; it < 4; ++it) {
      R.lane_excl[it] = (elo >> (8 * it)) & 0xFFu;
      R.it_off[it] = run;
      run += (tlo >> (8 * it)) & 0xFFu;
    }
#pragma unroll
    for (int it = 0; it < 4; ++it) {
      R.lane_excl[it + 4] = (ehi >> (8 * it)) & 0xFFu;
      R.it_off[it + 4] = run;
      run += (thi >> (8 * it)) & 0xFFu;
    }
  } else {                                         // nothing flagged in this warp: no scan needed
#pragma unroll
    for (int it = 0; it < kTileIters; ++it) { R.lane_excl[it] = 0u; R.it_off[it] = 0u; }
  }
  const uint32_t hb = __ballot_sync(0xFFFFFFFFu, head_flag);   // only warp 0 can have head entries
  R.head_rank = __popc(hb & lanemask_lt());
  if (lane == 0) {
    s_wtot[warp] = run;
    if (warp == 0) s_wtot[kWarpsPerTile] = __popc(hb);
  }
}

// Second half (after the barrier): offsets of this warp and the tile total.
__device__ __forceinline__ void tile_ranks_collect(TileRanks& R, const uint32_t* s_wtot) {
  const uint32_t warp = threadIdx.x >> 5;
  uint32_t off = s_wtot[kWarpsPerTile], tot = off;
#pragma unroll
  for (int w = 0; w < kWarpsPerTile; ++w) {
    const uint32_t c = s_wtot[w];
    if ((uint32_t)w < warp) off += c;
    tot += c;
  }
  R.warp_off = off;
  R.tile_total = tot;
}

__device__ __forceinline__ void tile_ranks(TileRanks& R, const uint32_t (&flags)[kTileIters], bool head_flag,
                                           uint32_t* s_wtot) {
  __syncthreads();                       // previous users of s_wtot are done
  tile_ranks_publish(R, flags, head_flag, s_wtot);
  __syncthreads();
  tile_ranks_collect(R, s_wtot);
}

__device__ __forceinline__ uint32_t rank_of(const TileRanks& R, const uint32_t (&flags)[kTileIters], int it, int slot) {
  return R.warp_off + R.it_off[it] + R.lane_excl[it] + __popc(flags[it] & ((1u << slot) - 1u));
}

}  // namespace s3gd

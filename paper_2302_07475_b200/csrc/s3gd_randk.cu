// RandKSign (Section 3.4; Algorithm 2 = Algorithm 1 with TopKSign replaced): worker m keeps
// K coordinates drawn uniformly without repetition and sends their signs.
//
// The paper names no generator.  Here the K coordinates of worker m at iteration t are
// pi(0), pi(1), ..., pi(K-1) for a keyed pseudo-random permutation pi of [0, d), listed in
// that order: a 4-round balanced Feistel network on 2h bits (2^(2h) >= d) whose round
// function is the 32-bit integer mixer "lowbias32" (C. Wellons, 2018), with cycle walking
// into [0, d) (Black & Rogaway, 2002).  Every entry of the message is independent of every
// other, so one thread computes one entry: permutation, one 4-byte gather from the
// gradient row, a warp ballot for the packed sign word, and (in the fused step) one
// integer atomic add into the vote counters.  The traffic is M*K scattered 32-byte
// sectors, far below one pass over the gradients.
#include "s3gd_common.cuh"

namespace s3gd {

namespace {

__host__ __device__ __forceinline__ uint32_t mix32(uint32_t v) {
  v ^= v >> 16; v *= 0x7FEB352Du;
  v ^= v >> 15; v *= 0x846CA68Bu;
  v ^= v >> 16;
  return v;
}

// Cycle walking ends because pi is a bijection of [0, 2^(2h)) and the start value is below d;
// each application leaves [0, d) with probability < 3/4, so kWalkLimit is never reached in
// practice.  If it were, the row is flagged instead of looping on.
constexpr int kWalkLimit = 4096;

__device__ __forceinline__ uint32_t permute(uint32_t j, uint32_t d, uint32_t h, const uint32_t (&key)[4],
                                            bool* gave_up) {
  const uint32_t mask = (1u << h) - 1u;
  uint32_t v = j;
  for (int walk = 0; walk < kWalkLimit; ++walk) {
    uint32_t left = v >> h, right = v & mask;
#pragma unroll
    for (int r = 0; r < 4; ++r) {
      const uint32_t f = mix32(right ^ key[r]) & mask;
      const uint32_t nl = right;
      right = left ^ f;
      left = nl;
    }
    v = (left << h) | right;
    if (v < d) return v;
  }
  *gave_up = true;
  return j;
}

// One warp per 32 consecutive message entries of one worker.
__global__ void __launch_bounds__(256) randk_kernel(const uint32_t* __restrict__ gbits, int M, uint32_t d, uint32_t K,
                                                    uint32_t h, uint32_t seed, uint32_t step,
                                                    uint32_t* __restrict__ out_idx, uint32_t* __restrict__ out_signbits,
                                                    int32_t* __restrict__ counter, uint32_t packed,
                                                    uint32_t* __restrict__ hdr) {
  const uint32_t words = (uint32_t)(((uint64_t)K + 31u) / 32u);      // (K + 31 would wrap for K near 2^32)
  const uint64_t total = (uint64_t)words * (uint64_t)M;
  const uint64_t warps = ((uint64_t)gridDim.x * blockDim.x) >> 5;
  const uint32_t lane = lane_id();
  bool gave_up = false;
  for (uint64_t w = ((uint64_t)blockIdx.x * blockDim.x + threadIdx.x) >> 5; w < total; w += warps) {
    const uint32_t m = (uint32_t)(w / words), ww = (uint32_t)(w - (uint64_t)m * words);
    const uint32_t base = seed ^ (m * 0x9E3779B9u) ^ (step * 0x85EBCA6Bu);
    uint32_t key[4];
#pragma unroll
    for (int r = 0; r < 4; ++r) key[r] = mix32(base + (uint32_t)(r + 1) * 0x9E3779B9u);
    const uint64_t j = (uint64_t)ww * 32u + lane;
    bool neg = false;
    if (j < K) {
      const uint32_t n = permute((uint32_t)j, d, h, key, &gave_up);
      neg = (__ldg(gbits + (uint64_t)m * d + n) >> 31) != 0u;
      if (out_idx) out_idx[(uint64_t)m * K + j] = n;
      if (counter) add_vote(counter, packed, n, neg ? 1u : 0u);
    }
    const uint32_t word = __ballot_sync(0xFFFFFFFFu, neg);
    if (out_signbits && lane == 0) out_signbits[w] = word;
  }
  if (gave_up) atomicOr(hdr + kHdrStatus, (uint32_t)kFlagInternal);
}

}  // namespace

cudaError_t launch_randk(const float* grads, int M, uint64_t d, uint64_t K, uint32_t seed, uint32_t step,
                         uint32_t* out_idx, uint32_t* out_signbits, int32_t* counter, bool packed, uint32_t* hdr,
                         cudaStream_t st) {
  if (K == 0) return cudaSuccess;
  uint32_t h = 1;
  while ((1ull << (2 * h)) < d) ++h;
  const uint64_t warps = (uint64_t)M * ((K + 31) / 32);
  uint64_t blocks = (warps + 7) / 8;
  const uint64_t cap = (uint64_t)sm_count() * 8;
  if (blocks > cap) blocks = cap;
  randk_kernel<<<(unsigned)blocks, 256, 0, st>>>(reinterpret_cast<const uint32_t*>(grads), M, (uint32_t)d, (uint32_t)K,
                                                 h, seed, step, out_idx, out_signbits, counter, packed ? 1u : 0u, hdr);
  count_launch();
  return cudaGetLastError();
}

}  // namespace s3gd

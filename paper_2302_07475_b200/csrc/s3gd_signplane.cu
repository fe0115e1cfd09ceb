// K = d: no sparsification, the step is signSGD with majority vote
// (Section 3.3, gamma = 1).  One streaming pass over the M sign planes: every
// thread owns a few adjacent coordinates, walks down the M rows adding
// 1 - 2 * signbit, and updates x from the sign of the total.
#include "s3gd_common.cuh"

namespace s3gd {

namespace {

template <int V> struct VecLoad;
template <> struct VecLoad<4> {
  static __device__ __forceinline__ void load(const float* p, uint32_t (&b)[4]) {
    uint4 v = ld_stream_v4(p);
    b[0] = v.x; b[1] = v.y; b[2] = v.z; b[3] = v.w;
  }
};
template <> struct VecLoad<2> {
  static __device__ __forceinline__ void load(const float* p, uint32_t (&b)[2]) {
    uint2 v = ld_stream_v2(p);
    b[0] = v.x; b[1] = v.y;
  }
};
// four adjacent coordinates from an address that is only 8-byte aligned (rows whose length is even but
// not a multiple of four start alternately on and off a 16-byte boundary): two 8-byte loads
struct VecLoad4Halves {
  static __device__ __forceinline__ void load(const float* p, uint32_t (&b)[4]) {
    uint2 lo = ld_stream_v2(p), hi = ld_stream_v2(p + 2);
    b[0] = lo.x; b[1] = lo.y; b[2] = hi.x; b[3] = hi.y;
  }
};
template <> struct VecLoad<1> {
  static __device__ __forceinline__ void load(const float* p, uint32_t (&b)[1]) { b[0] = ld_stream_u32(p); }
};

constexpr int kRowUnroll = 8;

// V adjacent coordinates per thread; requires every row start + column to be V*4-byte aligned.
template <int V, typename Load = VecLoad<V>>
__global__ void __launch_bounds__(256) signplane_step_kernel(float* __restrict__ x, const float* __restrict__ grads,
                                                             int M, uint64_t d, float lr,
                                                             int8_t* __restrict__ opt_vote) {
  const uint64_t nvec = d / V;   // (the host launches signplane_tail_kernel for the d % V columns left over)
  const uint64_t stride = (uint64_t)gridDim.x * blockDim.x;
  for (uint64_t v = (uint64_t)blockIdx.x * blockDim.x + threadIdx.x; v < nvec; v += stride) {
    const float* col = grads + v * V;
    int negs[V];
#pragma unroll
    for (int q = 0; q < V; ++q) negs[q] = 0;
    int m = 0;
    for (; m + kRowUnroll <= M; m += kRowUnroll) {
      uint32_t b[kRowUnroll][V];
#pragma unroll
      for (int u = 0; u < kRowUnroll; ++u) Load::load(col + (uint64_t)(m + u) * d, b[u]);
#pragma unroll
      for (int u = 0; u < kRowUnroll; ++u)
#pragma unroll
        for (int q = 0; q < V; ++q) negs[q] += (int)(b[u][q] >> 31);
    }
    for (; m < M; ++m) {
      uint32_t b[V];
      Load::load(col + (uint64_t)m * d, b);
#pragma unroll
      for (int q = 0; q < V; ++q) negs[q] += (int)(b[q] >> 31);
    }
#pragma unroll
    for (int q = 0; q < V; ++q) {
      int total = M - 2 * negs[q];            // sum over workers of (+1 | -1)
      uint64_t n = v * V + q;
      if (opt_vote) opt_vote[n] = (int8_t)((total > 0) - (total < 0));
      if (total > 0) x[n] = __fsub_rn(x[n], lr);
      else if (total < 0) x[n] = __fadd_rn(x[n], lr);
    }
  }
}

// coordinates [first, d): one thread each (the columns a vector form leaves over)
__global__ void signplane_tail_kernel(float* __restrict__ x, const float* __restrict__ grads, int M, uint64_t d,
                                      uint64_t first, float lr, int8_t* __restrict__ opt_vote) {
  const uint64_t n = first + threadIdx.x;
  if (n >= d) return;
  int negs = 0;
  for (int m = 0; m < M; ++m) negs += (int)(ld_stream_u32(reinterpret_cast<const uint32_t*>(grads) + (uint64_t)m * d + n) >> 31);
  const int total = M - 2 * negs;
  if (opt_vote) opt_vote[n] = (int8_t)((total > 0) - (total < 0));
  if (total > 0) x[n] = __fsub_rn(x[n], lr);
  else if (total < 0) x[n] = __fadd_rn(x[n], lr);
}

// The transmitted form of "keep everything": idx = 0..d-1, sign bits by warp ballot.
__global__ void __launch_bounds__(256) signplane_message_kernel(const float* __restrict__ grads, int M, uint64_t d,
                                                                uint32_t* __restrict__ out_idx,
                                                                uint32_t* __restrict__ out_signbits) {
  const uint64_t words = (d + 31) / 32;
  const uint64_t total_words = words * (uint64_t)M;
  const uint64_t warps = ((uint64_t)gridDim.x * blockDim.x) >> 5;
  const uint32_t lane = lane_id();
  for (uint64_t w = ((uint64_t)blockIdx.x * blockDim.x + threadIdx.x) >> 5; w < total_words; w += warps) {
    uint64_t m = w / words, ww = w - m * words;
    uint64_t n = ww * 32 + lane;
    bool neg = false;
    if (n < d) {
      neg = (__float_as_uint(grads[m * d + n]) >> 31) != 0u;
      out_idx[m * d + n] = (uint32_t)n;
    }
    uint32_t word = __ballot_sync(0xFFFFFFFFu, neg);
    if (lane == 0) out_signbits[w] = word;
  }
}

// Sign counts only: counter[n] = sum over workers of (+1 | -1).
__global__ void __launch_bounds__(256) signplane_counts_kernel(const float* __restrict__ grads, int M, uint64_t d,
                                                               int32_t* __restrict__ counter) {
  const uint64_t stride = (uint64_t)gridDim.x * blockDim.x;
  for (uint64_t n = (uint64_t)blockIdx.x * blockDim.x + threadIdx.x; n < d; n += stride) {
    int negs = 0;
    for (int m = 0; m < M; ++m) negs += (int)(ld_stream_u32(grads + (uint64_t)m * d + n) >> 31);
    counter[n] = M - 2 * negs;
  }
}

inline unsigned blocks_for(uint64_t threads) {
  uint64_t b = (threads + 255) / 256;
  uint64_t cap = (uint64_t)sm_count() * 8;
  if (b < 1) b = 1;
  return (unsigned)(b < cap ? b : cap);
}

// The walks down the M rows get one thread per column group, however many blocks that takes: blocks that
// come and go keep the memory system evenly loaded to the end, where a resident grid striding over the
// columns left the last round thin (resnet18 shape, K = d: 0.730 ms with 8 blocks per SM, 0.682 with 64,
// 0.676 ms unbounded; resnet50 shape 0.609 / 0.534 / 0.523 ms).
inline unsigned blocks_for_walk(uint64_t threads) {
  uint64_t b = (threads + 255) / 256;
  if (b < 1) b = 1;
  return (unsigned)(b < 0x7FFFFFFFull ? b : 0x7FFFFFFFull);
}

}  // namespace

cudaError_t launch_signplane_step(float* x, const float* grads, int M, uint64_t d, float lr, int8_t* opt_vote,
                                  cudaStream_t st) {
  uintptr_t a = reinterpret_cast<uintptr_t>(grads);
  if (d % 4 == 0 && a % 16 == 0) {
    signplane_step_kernel<4><<<blocks_for_walk(d / 4), 256, 0, st>>>(x, grads, M, d, lr, opt_vote);
    count_launch();
  } else if (d % 4 == 2 && a % 8 == 0 && d >= 4) {
    // columns in fours, the last two coordinates of every row by a second small launch
    signplane_step_kernel<4, VecLoad4Halves><<<blocks_for_walk(d / 4), 256, 0, st>>>(x, grads, M, d, lr, opt_vote);
    count_launch();
    signplane_tail_kernel<<<1, 32, 0, st>>>(x, grads, M, d, d - 2, lr, opt_vote);
    count_launch();
  } else if (d % 2 == 0 && a % 8 == 0) {
    signplane_step_kernel<2><<<blocks_for_walk(d / 2), 256, 0, st>>>(x, grads, M, d, lr, opt_vote);
    count_launch();
  } else {
    signplane_step_kernel<1><<<blocks_for_walk(d), 256, 0, st>>>(x, grads, M, d, lr, opt_vote);
    count_launch();
  }
  return cudaGetLastError();
}

cudaError_t launch_signplane_message(const float* grads, int M, uint64_t d, uint32_t* out_idx,
                                     uint32_t* out_signbits, cudaStream_t st) {
  uint64_t warps = (uint64_t)M * ((d + 31) / 32);
  signplane_message_kernel<<<blocks_for(warps * 32), 256, 0, st>>>(grads, M, d, out_idx, out_signbits);
  count_launch();
  return cudaGetLastError();
}

cudaError_t launch_signplane_counts(const float* grads, int M, uint64_t d, int32_t* counter, cudaStream_t st) {
  signplane_counts_kernel<<<blocks_for_walk(d), 256, 0, st>>>(grads, M, d, counter);
  count_launch();
  return cudaGetLastError();
}

}  // namespace s3gd

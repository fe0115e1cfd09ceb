// Server side of the step: integer vote accumulation, sign, and the update of x
// (Section 2.2 "Majority vote" and Eq. (7)).  Everything is integer work plus one
// fp32 add per changed coordinate, so results do not depend on execution order.
#include "s3gd_common.cuh"

namespace s3gd {

namespace {

__device__ __forceinline__ float moved(float x, int s, float lr) {
  // one IEEE round-to-nearest operation; __fadd_rn / __fsub_rn are never fused or reassociated
  return s > 0 ? __fsub_rn(x, lr) : __fadd_rn(x, lr);
}

// x[n] -= lr * sgn(vote[n])
__global__ void __launch_bounds__(256) apply_kernel(float* __restrict__ x, const int8_t* __restrict__ vote,
                                                    uint64_t d, float lr) {
  uint64_t stride = (uint64_t)gridDim.x * blockDim.x;
  for (uint64_t n = (uint64_t)blockIdx.x * blockDim.x + threadIdx.x; n < d; n += stride) {
    int s = vote[n];
    if (s != 0) x[n] = moved(x[n], s, lr);
  }
}

// 16 coordinates per thread step: one 16-byte load of votes, four of x.
__global__ void __launch_bounds__(256) apply_kernel_v16(float* __restrict__ x, const int8_t* __restrict__ vote,
                                                        uint64_t n16, float lr) {
  uint64_t stride = (uint64_t)gridDim.x * blockDim.x;
  for (uint64_t i = (uint64_t)blockIdx.x * blockDim.x + threadIdx.x; i < n16; i += stride) {
    uint4 v = *reinterpret_cast<const uint4*>(vote + i * 16);
    uint32_t w[4] = {v.x, v.y, v.z, v.w};
#pragma unroll
    for (int q = 0; q < 4; ++q) {
      if (w[q] == 0u) continue;
      float4* px = reinterpret_cast<float4*>(x + i * 16 + q * 4);
      float4 xv = *px;
      int s0 = (int8_t)(w[q] & 0xFF), s1 = (int8_t)((w[q] >> 8) & 0xFF);
      int s2 = (int8_t)((w[q] >> 16) & 0xFF), s3 = (int8_t)(w[q] >> 24);
      if (s0) xv.x = moved(xv.x, s0, lr);
      if (s1) xv.y = moved(xv.y, s1, lr);
      if (s2) xv.z = moved(xv.z, s2, lr);
      if (s3) xv.w = moved(xv.w, s3, lr);
      *px = xv;
    }
  }
}

// counter[idx] += 1 - 2 * signbit for every transmitted entry
__global__ void __launch_bounds__(256) vote_scatter_kernel(const uint32_t* __restrict__ idx,
                                                           const uint32_t* __restrict__ signbits, int M, uint64_t K,
                                                           uint64_t d, int32_t* __restrict__ counter,
                                                           uint32_t* __restrict__ hdr) {
  const uint64_t words = (K + 31) / 32;
  const uint64_t total = (uint64_t)M * K;
  uint64_t stride = (uint64_t)gridDim.x * blockDim.x;
  uint32_t bad = 0;
  for (uint64_t e = (uint64_t)blockIdx.x * blockDim.x + threadIdx.x; e < total; e += stride) {
    uint64_t m = e / K, j = e - m * K;
    uint32_t n = idx[e];
    uint32_t neg = (signbits[m * words + (j >> 5)] >> (j & 31)) & 1u;
    if (n < d) atomicAdd(counter + n, neg ? -1 : 1);
    else ++bad;
  }
  if (bad) {
    atomicAdd(hdr + kHdrBadIndex, bad);
    atomicOr(hdr + kHdrStatus, (uint32_t)kFlagIndexRange);
  }
}

__global__ void __launch_bounds__(256) counter_sign_v4_kernel(const int4* __restrict__ counter4, uint64_t n4,
                                                              uint32_t* __restrict__ vote4) {
  const uint64_t stride = (uint64_t)gridDim.x * blockDim.x;
  for (uint64_t i = (uint64_t)blockIdx.x * blockDim.x + threadIdx.x; i < n4; i += stride) {
    const int4 c = counter4[i];
    const int s[4] = {(c.x > 0) - (c.x < 0), (c.y > 0) - (c.y < 0), (c.z > 0) - (c.z < 0), (c.w > 0) - (c.w < 0)};
    uint32_t pk = 0;
#pragma unroll
    for (int q = 0; q < 4; ++q) pk |= (uint32_t)(uint8_t)(int8_t)s[q] << (8 * q);
    vote4[i] = pk;
  }
}

__global__ void __launch_bounds__(256) counter_sign_kernel(const int32_t* __restrict__ counter, uint64_t d,
                                                           int8_t* __restrict__ vote) {
  uint64_t stride = (uint64_t)gridDim.x * blockDim.x;
  for (uint64_t n = (uint64_t)blockIdx.x * blockDim.x + threadIdx.x; n < d; n += stride) {
    int c = counter[n];
    vote[n] = (int8_t)((c > 0) - (c < 0));
  }
}

// sign of the counters fused with the update: 4 coordinates per thread step
template <bool kVec>
__global__ void __launch_bounds__(256) counter_apply_kernel(const int32_t* __restrict__ counter,
                                                            float* __restrict__ x, uint64_t d, float lr,
                                                            int8_t* __restrict__ opt_vote) {
  uint64_t stride = (uint64_t)gridDim.x * blockDim.x;
  if (kVec) {
    const uint64_t n4 = d / 4;
    for (uint64_t i = (uint64_t)blockIdx.x * blockDim.x + threadIdx.x; i < n4; i += stride) {
      int4 c = *reinterpret_cast<const int4*>(counter + i * 4);
      if (opt_vote) {
        uint32_t pk = (uint32_t)(uint8_t)(int8_t)((c.x > 0) - (c.x < 0)) |
                      ((uint32_t)(uint8_t)(int8_t)((c.y > 0) - (c.y < 0)) << 8) |
                      ((uint32_t)(uint8_t)(int8_t)((c.z > 0) - (c.z < 0)) << 16) |
                      ((uint32_t)(uint8_t)(int8_t)((c.w > 0) - (c.w < 0)) << 24);
        *reinterpret_cast<uint32_t*>(opt_vote + i * 4) = pk;
      }
      if ((c.x | c.y | c.z | c.w) == 0) continue;
      float4* px = reinterpret_cast<float4*>(x + i * 4);
      float4 xv = *px;
      if (c.x) xv.x = moved(xv.x, c.x, lr);
      if (c.y) xv.y = moved(xv.y, c.y, lr);
      if (c.z) xv.z = moved(xv.z, c.z, lr);
      if (c.w) xv.w = moved(xv.w, c.w, lr);
      *px = xv;
    }
    // ragged tail (d % 4 entries)
    uint64_t n = n4 * 4 + (uint64_t)blockIdx.x * blockDim.x + threadIdx.x;
    if (n < d) {
      int c = counter[n];
      if (opt_vote) opt_vote[n] = (int8_t)((c > 0) - (c < 0));
      if (c) x[n] = moved(x[n], c, lr);
    }
  } else {
    for (uint64_t n = (uint64_t)blockIdx.x * blockDim.x + threadIdx.x; n < d; n += stride) {
      int c = counter[n];
      if (opt_vote) opt_vote[n] = (int8_t)((c > 0) - (c < 0));
      if (c) x[n] = moved(x[n], c, lr);
    }
  }
}

// The same for packed counters (one byte per coordinate holding 128 + count): a thread takes one
// 32-bit word = four coordinates.  kVec: x is 16-byte aligned and opt_vote (if given) 4-byte aligned.
template <bool kVec>
__global__ void __launch_bounds__(256) counter_apply_packed_kernel(const uint32_t* __restrict__ cw,
                                                                   float* __restrict__ x, uint64_t d, float lr,
                                                                   int8_t* __restrict__ opt_vote) {
  grid_dependency_wait();                            // (launched with launch_after)
  const uint64_t n_words = (d + 3) / 4;
  const uint64_t stride = (uint64_t)gridDim.x * blockDim.x;
  for (uint64_t i = (uint64_t)blockIdx.x * blockDim.x + threadIdx.x; i < n_words; i += stride) {
    const uint32_t w = cw[i];
    if (w == kPackedZero && opt_vote == nullptr) continue;
    int c[4];
#pragma unroll
    for (int q = 0; q < 4; ++q) c[q] = (int)((w >> (8 * q)) & 0xFFu) - 128;
    const bool full = i * 4 + 4 <= d;
    if (kVec && full) {
      if (opt_vote) {
        uint32_t pk = 0;
#pragma unroll
        for (int q = 0; q < 4; ++q) pk |= (uint32_t)(uint8_t)(int8_t)((c[q] > 0) - (c[q] < 0)) << (8 * q);
        *reinterpret_cast<uint32_t*>(opt_vote + i * 4) = pk;
      }
      if (w == kPackedZero) continue;
      float4* px = reinterpret_cast<float4*>(x + i * 4);
      float4 xv = *px;
      if (c[0]) xv.x = moved(xv.x, c[0], lr);
      if (c[1]) xv.y = moved(xv.y, c[1], lr);
      if (c[2]) xv.z = moved(xv.z, c[2], lr);
      if (c[3]) xv.w = moved(xv.w, c[3], lr);
      *px = xv;
    } else {
#pragma unroll
      for (int q = 0; q < 4; ++q) {
        const uint64_t n = i * 4 + q;
        if (n >= d) break;
        if (opt_vote) opt_vote[n] = (int8_t)((c[q] > 0) - (c[q] < 0));
        if (c[q]) x[n] = moved(x[n], c[q], lr);
      }
    }
  }
}

// Packed counters where few coordinates were voted on (at most one in 64): nearly every word is the
// zero pattern, so the pass is a scan of d bytes whose speed is set by the bytes each thread keeps in
// flight.  A thread loads two 16-byte groups (32 coordinates) at a time and only looks inside a group
// that differs from the zero pattern.  x 16-byte aligned, no vote output.
__global__ void __launch_bounds__(256) counter_apply_packed_sparse_kernel(const uint32_t* __restrict__ cw,
                                                                          float* __restrict__ x, uint64_t d, float lr) {
  grid_dependency_wait();                            // (launched with launch_after)
  const uint64_t n_words = (d + 3) / 4, n_groups = n_words / 4;
  const uint64_t stride = (uint64_t)gridDim.x * blockDim.x;
  const uint64_t first = (uint64_t)blockIdx.x * blockDim.x + threadIdx.x;
  const uint4* cg = reinterpret_cast<const uint4*>(cw);
  auto word = [&](uint64_t i, uint32_t w) {       // word i = coordinates 4i .. 4i+3
    if (w == kPackedZero) return;
    int c[4];
#pragma unroll
    for (int q = 0; q < 4; ++q) c[q] = (int)((w >> (8 * q)) & 0xFFu) - 128;
    if (i * 4 + 4 <= d) {
      float4* px = reinterpret_cast<float4*>(x + i * 4);
      float4 xv = *px;
      if (c[0]) xv.x = moved(xv.x, c[0], lr);
      if (c[1]) xv.y = moved(xv.y, c[1], lr);
      if (c[2]) xv.z = moved(xv.z, c[2], lr);
      if (c[3]) xv.w = moved(xv.w, c[3], lr);
      *px = xv;
    } else {
#pragma unroll
      for (int q = 0; q < 4; ++q) {
        const uint64_t n = i * 4 + q;
        if (n < d && c[q]) x[n] = moved(x[n], c[q], lr);
      }
    }
  };
  auto group = [&](uint64_t g, const uint4& v) {
    if (v.x == kPackedZero && v.y == kPackedZero && v.z == kPackedZero && v.w == kPackedZero) return;
    word(g * 4, v.x); word(g * 4 + 1, v.y); word(g * 4 + 2, v.z); word(g * 4 + 3, v.w);
  };
  uint64_t g = first;
  for (; g + stride < n_groups; g += 2 * stride) {
    const uint4 a = __ldcs(cg + g), b = __ldcs(cg + g + stride);
    group(g, a);
    group(g + stride, b);
  }
  if (g < n_groups) group(g, __ldcs(cg + g));
  // the words after the last whole group
  const uint64_t i = n_groups * 4 + first;
  if (i < n_words) word(i, cw[i]);
}

// err <- grads + eta * err: one rounding for the product, one for the sum (Eq. (5))
__global__ void __launch_bounds__(256) ef_accumulate_kernel(float* __restrict__ err, const float* __restrict__ grads,
                                                            float eta, uint64_t n) {
  const uint64_t stride = (uint64_t)gridDim.x * blockDim.x;
  for (uint64_t i = (uint64_t)blockIdx.x * blockDim.x + threadIdx.x; i < n; i += stride)
    err[i] = __fadd_rn(grads[i], __fmul_rn(eta, err[i]));
}

__global__ void __launch_bounds__(256) ef_accumulate_kernel_v4(float4* __restrict__ err, const float4* __restrict__ grads,
                                                               float eta, uint64_t n4) {
  const uint64_t stride = (uint64_t)gridDim.x * blockDim.x;
  for (uint64_t i = (uint64_t)blockIdx.x * blockDim.x + threadIdx.x; i < n4; i += stride) {
    const float4 g = grads[i];
    float4 e = err[i];
    e.x = __fadd_rn(g.x, __fmul_rn(eta, e.x));
    e.y = __fadd_rn(g.y, __fmul_rn(eta, e.y));
    e.z = __fadd_rn(g.z, __fmul_rn(eta, e.z));
    e.w = __fadd_rn(g.w, __fmul_rn(eta, e.w));
    err[i] = e;
  }
}

// Momentum form of the update: v <- mu * v + s ; x <- x - lr * v, every operation rounded once.
__device__ __forceinline__ void momentum_update(float& x, float& v, int s, float mu, float lr) {
  v = __fadd_rn(__fmul_rn(mu, v), (float)((s > 0) - (s < 0)));
  x = __fsub_rn(x, __fmul_rn(lr, v));
}

template <bool kPacked>
__global__ void __launch_bounds__(256) counter_apply_momentum_kernel(const int32_t* __restrict__ counter,
                                                                     float* __restrict__ x, float* __restrict__ v,
                                                                     uint64_t d, float mu, float lr,
                                                                     int8_t* __restrict__ opt_vote) {
  const uint64_t stride = (uint64_t)gridDim.x * blockDim.x;
  for (uint64_t n = (uint64_t)blockIdx.x * blockDim.x + threadIdx.x; n < d; n += stride) {
    const int c = kPacked ? (int)reinterpret_cast<const uint8_t*>(counter)[n] - 128 : counter[n];
    if (opt_vote) opt_vote[n] = (int8_t)((c > 0) - (c < 0));
    float xv = x[n], vv = v[n];
    momentum_update(xv, vv, c, mu, lr);
    x[n] = xv;
    v[n] = vv;
  }
}

__global__ void __launch_bounds__(256) apply_momentum_kernel(float* __restrict__ x, float* __restrict__ v,
                                                             const int8_t* __restrict__ vote, uint64_t d, float mu,
                                                             float lr) {
  const uint64_t stride = (uint64_t)gridDim.x * blockDim.x;
  for (uint64_t n = (uint64_t)blockIdx.x * blockDim.x + threadIdx.x; n < d; n += stride) {
    float xv = x[n], vv = v[n];
    momentum_update(xv, vv, vote[n], mu, lr);
    x[n] = xv;
    v[n] = vv;
  }
}

// Four coordinates per thread: one word of byte counters (or four int32 counters, or four int8 votes:
// kSource 0 / 1 / 2), x and v as float4.  x and v 16-byte aligned, counters 16-byte aligned, votes 4-byte aligned.
template <int kSource>
__global__ void __launch_bounds__(256) momentum_v4_kernel(const void* __restrict__ src, float4* __restrict__ x4,
                                                          float4* __restrict__ v4, uint64_t n4, float mu, float lr,
                                                          uint32_t* __restrict__ opt_vote4) {
  const uint64_t stride = (uint64_t)gridDim.x * blockDim.x;
  for (uint64_t i = (uint64_t)blockIdx.x * blockDim.x + threadIdx.x; i < n4; i += stride) {
    int c[4];
    if (kSource == 0) {
      const uint32_t w = static_cast<const uint32_t*>(src)[i];
#pragma unroll
      for (int q = 0; q < 4; ++q) c[q] = (int)((w >> (8 * q)) & 0xFFu) - 128;
    } else if (kSource == 1) {
      const int4 cc = static_cast<const int4*>(src)[i];
      c[0] = cc.x; c[1] = cc.y; c[2] = cc.z; c[3] = cc.w;
    } else {
      const uint32_t w = static_cast<const uint32_t*>(src)[i];
#pragma unroll
      for (int q = 0; q < 4; ++q) c[q] = (int)(int8_t)((w >> (8 * q)) & 0xFFu);
    }
    float4 xv = x4[i], vv = v4[i];
    momentum_update(xv.x, vv.x, c[0], mu, lr);
    momentum_update(xv.y, vv.y, c[1], mu, lr);
    momentum_update(xv.z, vv.z, c[2], mu, lr);
    momentum_update(xv.w, vv.w, c[3], mu, lr);
    x4[i] = xv;
    v4[i] = vv;
    if (kSource != 2 && opt_vote4) {
      uint32_t pk = 0;
#pragma unroll
      for (int q = 0; q < 4; ++q) pk |= (uint32_t)(uint8_t)(int8_t)((c[q] > 0) - (c[q] < 0)) << (8 * q);
      opt_vote4[i] = pk;
    }
  }
}

inline unsigned grid_for(uint64_t items, int per_block, int max_blocks) {
  uint64_t b = (items + per_block - 1) / per_block;
  if (b < 1) b = 1;
  if (b > (uint64_t)max_blocks) b = max_blocks;
  return (unsigned)b;
}

inline bool aligned(const void* p, size_t a) { return (reinterpret_cast<uintptr_t>(p) % a) == 0; }

}  // namespace

cudaError_t launch_apply(float* x, const int8_t* vote, uint64_t d, float lr, cudaStream_t st) {
  if (aligned(x, 16) && aligned(vote, 16) && d >= 16) {
    uint64_t n16 = d / 16;
    apply_kernel_v16<<<grid_for(n16, 256, 0x7FFFFFFF), 256, 0, st>>>(x, vote, n16, lr);
    count_launch();
    uint64_t done = n16 * 16;
    if (done < d) apply_kernel<<<1, 256, 0, st>>>(x + done, vote + done, d - done, lr);
    if (done < d) count_launch();
  } else {
    apply_kernel<<<grid_for(d, 256, sm_count() * 8), 256, 0, st>>>(x, vote, d, lr);
    count_launch();
  }
  return cudaGetLastError();
}

cudaError_t launch_vote_scatter(const uint32_t* idx, const uint32_t* signbits, int M, uint64_t K, uint64_t d,
                                int32_t* counter, uint32_t* hdr, cudaStream_t st) {
  uint64_t total = (uint64_t)M * K;
  if (total == 0) return cudaSuccess;
  vote_scatter_kernel<<<grid_for(total, 256, sm_count() * 16), 256, 0, st>>>(idx, signbits, M, K, d, counter, hdr);
  count_launch();
  return cudaGetLastError();
}

cudaError_t launch_counter_sign(const int32_t* counter, uint64_t d, int8_t* vote, cudaStream_t st) {
  uint64_t done = 0;
  if (d >= 4 && aligned(counter, 16) && aligned(vote, 4)) {      // four counters in, one word of votes out
    const uint64_t n4 = d / 4;
    counter_sign_v4_kernel<<<grid_for(n4, 256, 0x7FFFFFFF), 256, 0, st>>>(reinterpret_cast<const int4*>(counter), n4,
                                                                         reinterpret_cast<uint32_t*>(vote));
    count_launch();
    done = n4 * 4;
    if (done == d) return cudaGetLastError();
  }
  counter_sign_kernel<<<grid_for(d - done, 256, sm_count() * 16), 256, 0, st>>>(counter + done, d - done, vote + done);
  count_launch();
  return cudaGetLastError();
}

cudaError_t launch_counter_apply(const int32_t* counter, bool packed, float* x, uint64_t d, float lr, int8_t* opt_vote,
                                 uint64_t max_votes, cudaStream_t st) {
  if (packed) {
    const uint32_t* cw = reinterpret_cast<const uint32_t*>(counter);
    if (max_votes != 0 && max_votes <= d / kSparseVotesRatio && opt_vote == nullptr && aligned(x, 16) &&
        aligned(counter, 16)) {
      count_launch();
      return launch_after(counter_apply_packed_sparse_kernel, dim3(grid_for((d + 15) / 16, 256, sm_count() * 8)), dim3(256), 0,
                          st, cw, x, d, lr);
    }
    const bool vecp = aligned(x, 16) && (opt_vote == nullptr || aligned(opt_vote, 4));
    const dim3 grid(grid_for((d + 3) / 4, 256, sm_count() * 8));
    count_launch();
    return vecp ? launch_after(counter_apply_packed_kernel<true>, grid, dim3(256), 0, st, cw, x, d, lr, opt_vote)
                : launch_after(counter_apply_packed_kernel<false>, grid, dim3(256), 0, st, cw, x, d, lr, opt_vote);
  }
  bool vec = aligned(x, 16) && aligned(counter, 16) && (opt_vote == nullptr || aligned(opt_vote, 4)) && d >= 4;
  if (vec) {
    counter_apply_kernel<true><<<grid_for(d / 4, 256, sm_count() * 8), 256, 0, st>>>(counter, x, d, lr, opt_vote);
    count_launch();
  } else {
    counter_apply_kernel<false><<<grid_for(d, 256, sm_count() * 8), 256, 0, st>>>(counter, x, d, lr, opt_vote);
    count_launch();
  }
  return cudaGetLastError();
}

cudaError_t launch_ef_accumulate(float* err, const float* grads, float eta, uint64_t n, cudaStream_t st) {
  if (aligned(err, 16) && aligned(grads, 16) && n >= 4) {
    const uint64_t n4 = n / 4;
    ef_accumulate_kernel_v4<<<grid_for(n4, 256, sm_count() * 16), 256, 0, st>>>(reinterpret_cast<float4*>(err),
                                                                         reinterpret_cast<const float4*>(grads), eta, n4);
    count_launch();
    if (n4 * 4 < n) {
      ef_accumulate_kernel<<<1, 256, 0, st>>>(err + n4 * 4, grads + n4 * 4, eta, n - n4 * 4);
      count_launch();
    }
  } else {
    ef_accumulate_kernel<<<grid_for(n, 256, sm_count() * 16), 256, 0, st>>>(err, grads, eta, n);
    count_launch();
  }
  return cudaGetLastError();
}

cudaError_t launch_counter_apply_momentum(const int32_t* counter, bool packed, float* x, float* v, uint64_t d, float mu,
                                          float lr, int8_t* opt_vote, cudaStream_t st) {
  // dense over d (v decays everywhere): four coordinates per thread and one thread per group where the
  // alignment allows, the scalar form for what is left over
  uint64_t done = 0;
  if (d >= 4 && aligned(x, 16) && aligned(v, 16) && aligned(counter, 16) && (opt_vote == nullptr || aligned(opt_vote, 4))) {
    const uint64_t n4 = d / 4;
    const unsigned grid = grid_for(n4, 256, 0x7FFFFFFF);
    if (packed)
      momentum_v4_kernel<0><<<grid, 256, 0, st>>>(counter, reinterpret_cast<float4*>(x), reinterpret_cast<float4*>(v), n4,
                                                  mu, lr, reinterpret_cast<uint32_t*>(opt_vote));
    else
      momentum_v4_kernel<1><<<grid, 256, 0, st>>>(counter, reinterpret_cast<float4*>(x), reinterpret_cast<float4*>(v), n4,
                                                  mu, lr, reinterpret_cast<uint32_t*>(opt_vote));
    count_launch();
    done = n4 * 4;
    if (done == d) return cudaGetLastError();
  }
  const uint64_t rest = d - done;
  int8_t* ov = opt_vote ? opt_vote + done : nullptr;
  if (packed)
    counter_apply_momentum_kernel<true><<<grid_for(rest, 256, sm_count() * 16), 256, 0, st>>>(
        reinterpret_cast<const int32_t*>(reinterpret_cast<const uint8_t*>(counter) + done), x + done, v + done, rest, mu, lr, ov);
  else
    counter_apply_momentum_kernel<false><<<grid_for(rest, 256, sm_count() * 16), 256, 0, st>>>(counter + done, x + done,
                                                                                             v + done, rest, mu, lr, ov);
  count_launch();
  return cudaGetLastError();
}

cudaError_t launch_apply_momentum(float* x, float* v, const int8_t* vote, uint64_t d, float mu, float lr,
                                  cudaStream_t st) {
  uint64_t done = 0;
  if (d >= 4 && aligned(x, 16) && aligned(v, 16) && aligned(vote, 4)) {
    const uint64_t n4 = d / 4;
    momentum_v4_kernel<2><<<grid_for(n4, 256, 0x7FFFFFFF), 256, 0, st>>>(vote, reinterpret_cast<float4*>(x),
                                                                        reinterpret_cast<float4*>(v), n4, mu, lr, nullptr);
    count_launch();
    done = n4 * 4;
    if (done == d) return cudaGetLastError();
  }
  apply_momentum_kernel<<<grid_for(d - done, 256, sm_count() * 16), 256, 0, st>>>(x + done, v + done, vote + done, d - done,
                                                                                mu, lr);
  count_launch();
  return cudaGetLastError();
}

}  // namespace s3gd

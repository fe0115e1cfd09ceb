// The pieces of the step that sit on either side of an exchange between GPUs when the workers
// of Algorithm 1 are spread over several of them: the vote over a message gathered from several
// senders fused with the update, vote sums that can be added up across GPUs, and the voted
// vector in a dense two-bit form for the way back (Section 2.2, "Majority vote": the server's
// message is the ternary vector sgn(sum of votes)).  Nothing here communicates; the exchange
// itself is the caller's collective between these calls.
#include "s3gd_common.cuh"

namespace s3gd {
namespace {

inline bool aligned(const void* p, size_t a) { return (reinterpret_cast<uintptr_t>(p) % a) == 0; }

inline unsigned grid_for(uint64_t items, int per_block, int max_blocks) {
  uint64_t b = (items + per_block - 1) / per_block;
  if (b < 1) b = 1;
  if (b > (uint64_t)max_blocks) b = max_blocks;
  return (unsigned)b;
}

// Votes of a message that lies in n_groups pieces (one per sender), group_stride words apart:
// piece g has the indices of its M_group workers, [M_group x K], at idx + g * group_stride and
// their sign words, [M_group x ceil(K/32)], at sgn + g * group_stride.  An index >= d is skipped
// and counted.
__global__ void __launch_bounds__(256) vote_groups_kernel(const uint32_t* __restrict__ idx,
                                                          const uint32_t* __restrict__ sgn, uint32_t n_groups,
                                                          uint64_t group_stride, uint32_t M_group, uint64_t K,
                                                          uint64_t d, int32_t* __restrict__ counter, uint32_t packed,
                                                          uint32_t* __restrict__ bad_count, uint32_t* __restrict__ status) {
  const uint64_t words = (K + 31) / 32;
  const uint64_t per_group = (uint64_t)M_group * K;
  const uint64_t total = per_group * n_groups;
  const uint64_t stride = (uint64_t)gridDim.x * blockDim.x;
  uint32_t bad = 0;
  for (uint64_t e = (uint64_t)blockIdx.x * blockDim.x + threadIdx.x; e < total; e += stride) {
    const uint64_t g = e / per_group, r = e - g * per_group;
    const uint64_t m = r / K, j = r - m * K;
    const uint32_t n = idx[g * group_stride + r];
    const uint32_t neg = (sgn[g * group_stride + m * words + (j >> 5)] >> (j & 31)) & 1u;
    if (n < d) add_vote(counter, packed, n, neg);
    else ++bad;
  }
  if (bad) {
    if (bad_count) atomicAdd(bad_count, bad);
    if (status) atomicOr(status, (uint32_t)kFlagIndexRange);
  }
}

// words of `value` repeated (the zero of the counters: 0, or 0x80808080 for biased bytes)
__global__ void __launch_bounds__(256) fill_words_kernel(uint32_t* __restrict__ p, uint64_t n_words, uint32_t value) {
  const uint64_t stride = (uint64_t)gridDim.x * blockDim.x;
  for (uint64_t i = (uint64_t)blockIdx.x * blockDim.x + threadIdx.x; i < n_words; i += stride) p[i] = value;
}

__device__ __forceinline__ uint32_t code_of(int c) { return c > 0 ? 1u : (c < 0 ? 3u : 0u); }   // 00, 01 (+1), 11 (-1)

// Sixteen consecutive sums starting at coordinate i (a multiple of 16), as signed totals.  Whole groups
// from a 16-byte aligned source are fetched with 16-byte loads; the ragged end and other alignments one by one.
template <int kKind>   // 0: int32 sums, 1: biased bytes, 2: int8 votes
__device__ __forceinline__ void load_sixteen(const void* __restrict__ src, uint32_t bias, uint64_t n, uint64_t i,
                                             bool src_aligned, int (&c)[16]) {
  if (src_aligned && i + 16 <= n) {
    if (kKind == 0) {
      const int4* p = reinterpret_cast<const int4*>(static_cast<const int32_t*>(src) + i);
#pragma unroll
      for (int g = 0; g < 4; ++g) {
        const int4 v = p[g];
        c[4 * g] = v.x; c[4 * g + 1] = v.y; c[4 * g + 2] = v.z; c[4 * g + 3] = v.w;
      }
    } else {
      const uint4 v = *reinterpret_cast<const uint4*>(static_cast<const uint8_t*>(src) + i);
      const uint32_t w[4] = {v.x, v.y, v.z, v.w};
#pragma unroll
      for (int q = 0; q < 16; ++q) {
        const uint32_t b = (w[q >> 2] >> (8 * (q & 3))) & 0xFFu;
        c[q] = kKind == 1 ? (int)(int8_t)(uint8_t)(b - bias) : (int)(int8_t)(uint8_t)b;
      }
    }
    return;
  }
#pragma unroll
  for (int q = 0; q < 16; ++q) {
    c[q] = 0;
    if (i + q < n) {
      if (kKind == 0) c[q] = static_cast<const int32_t*>(src)[i + q];
      else if (kKind == 1) c[q] = (int)(int8_t)(uint8_t)(static_cast<const uint8_t*>(src)[i + q] - bias);
      else c[q] = static_cast<const int8_t*>(src)[i + q];
    }
  }
}

// sixteen coordinates -> one word of two-bit codes.  kBytes: one byte per coordinate holding the
// sum of `n_summed` biased bytes (each 128 + a partial sum), reduced modulo 256; the total then is
// (byte - 128 * n_summed) as a signed byte.  Otherwise int32 sums (or int8 votes, kVotes).
template <int kKind>   // 0: int32 sums, 1: biased bytes, 2: int8 votes
__global__ void __launch_bounds__(256) encode2_kernel(const void* __restrict__ src, uint32_t bias, uint64_t n,
                                                      uint32_t* __restrict__ out) {
  const uint64_t n_words = (n + 15) / 16;
  const uint64_t stride = (uint64_t)gridDim.x * blockDim.x;
  const bool src_aligned = (reinterpret_cast<uintptr_t>(src) & 15u) == 0u;
  for (uint64_t w = (uint64_t)blockIdx.x * blockDim.x + threadIdx.x; w < n_words; w += stride) {
    int c[16];
    load_sixteen<kKind>(src, bias, n, w * 16, src_aligned, c);
    uint32_t word = 0;
#pragma unroll
    for (int q = 0; q < 16; ++q) word |= code_of(c[q]) << (2 * q);      // (beyond n: 0, the code of "no vote")
    out[w] = word;
  }
}

__device__ __forceinline__ float moved2(float x, uint32_t code, float lr) {
  return code == 1u ? __fsub_rn(x, lr) : __fadd_rn(x, lr);      // one rounding, as s3gd_apply
}

// x <- x - lr * vote from the two-bit form: a thread takes one word = sixteen coordinates
__global__ void __launch_bounds__(256) apply2_kernel(float* __restrict__ x, const uint32_t* __restrict__ words,
                                                     uint64_t d, float lr, int8_t* __restrict__ opt_vote) {
  const uint64_t n_words = (d + 15) / 16;
  const uint64_t stride = (uint64_t)gridDim.x * blockDim.x;
  for (uint64_t w = (uint64_t)blockIdx.x * blockDim.x + threadIdx.x; w < n_words; w += stride) {
    const uint32_t word = words[w];
    if (word == 0u && opt_vote == nullptr) continue;
#pragma unroll
    for (int q = 0; q < 16; ++q) {
      const uint64_t i = w * 16 + q;
      if (i >= d) break;
      const uint32_t code = (word >> (2 * q)) & 3u;
      const bool moves = (code & 1u) != 0u;                     // the pair 10 is never sent; it leaves x alone
      if (opt_vote) opt_vote[i] = moves ? (code == 1u ? 1 : -1) : 0;
      if (moves) x[i] = moved2(x[i], code, lr);
    }
  }
}


// ---- the sparse form of the server's message: the coordinates with a non-zero vote, ascending, and
// their sign bits, in the layout of a worker's message.  Three launches: non-zero votes per block of
// kSparseBlock coordinates; exclusive scan of the block counts (one CTA); ordered emission.
constexpr int kSparseThreads = 256;
constexpr int kSparsePer = 16;                                     // consecutive coordinates per thread
constexpr int kSparseBlock = kSparseThreads * kSparsePer;          // coordinates per block

// bit q of the results: coordinate first + q has a non-zero vote / a negative one
template <int kKind>
__device__ __forceinline__ void thread_votes(const void* __restrict__ src, uint32_t bias, uint64_t n, uint64_t first,
                                             uint32_t* moved, uint32_t* negative) {
  static_assert(kSparsePer == 16, "a thread's coordinates are one group of load_sixteen");
  int c[16];
  load_sixteen<kKind>(src, bias, n, first, (reinterpret_cast<uintptr_t>(src) & 15u) == 0u, c);
  uint32_t mv = 0, ng = 0;
#pragma unroll
  for (int q = 0; q < kSparsePer; ++q) {
    mv |= (uint32_t)(c[q] != 0) << q;                 // (beyond n: 0)
    ng |= (uint32_t)(c[q] < 0) << q;
  }
  *moved = mv; *negative = ng;
}

__device__ __forceinline__ uint32_t block_exclusive_scan_256(uint32_t v, uint32_t* s_warp, uint32_t* total) {
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
  for (int w = 0; w < kSparseThreads / 32; ++w) {
    const uint32_t c = s_warp[w];
    if ((uint32_t)w < warp) off += c;
    tot += c;
  }
  *total = tot;
  return off + inc - v;
}

template <int kKind>
__global__ void __launch_bounds__(kSparseThreads) sparse_count_kernel(const void* __restrict__ src, uint32_t bias,
                                                                      uint64_t n, uint32_t* __restrict__ blk) {
  __shared__ uint32_t s_warp[kSparseThreads / 32];
  uint32_t mv, ng;
  thread_votes<kKind>(src, bias, n, (uint64_t)blockIdx.x * kSparseBlock + (uint64_t)threadIdx.x * kSparsePer, &mv, &ng);
  uint32_t total;
  block_exclusive_scan_256((uint32_t)__popc(mv), s_warp, &total);
  if (threadIdx.x == 0) blk[blockIdx.x] = total;
}

// blk[b] <- number of non-zero votes in the blocks before b; *out_count <- their total.  One CTA.
__global__ void __launch_bounds__(kSparseThreads) sparse_scan_kernel(uint32_t* __restrict__ blk, uint32_t n_blocks,
                                                                     uint32_t* __restrict__ out_count) {
  __shared__ uint32_t s_warp[kSparseThreads / 32];
  uint32_t carry = 0;
  for (uint32_t base = 0; base < n_blocks; base += kSparseThreads) {
    const uint32_t b = base + threadIdx.x;
    const uint32_t v = b < n_blocks ? blk[b] : 0u;
    uint32_t total;
    const uint32_t ex = block_exclusive_scan_256(v, s_warp, &total);
    if (b < n_blocks) blk[b] = carry + ex;
    carry += total;
  }
  if (threadIdx.x == 0) *out_count = carry;
}

template <int kKind>
__global__ void __launch_bounds__(kSparseThreads) sparse_emit_kernel(const void* __restrict__ src, uint32_t bias,
                                                                     uint64_t n, uint32_t index_base,
                                                                     const uint32_t* __restrict__ blk, uint32_t cap,
                                                                     uint32_t* __restrict__ out_idx,
                                                                     uint32_t* __restrict__ out_signbits) {
  __shared__ uint32_t s_warp[kSparseThreads / 32];
  const uint64_t first = (uint64_t)blockIdx.x * kSparseBlock + (uint64_t)threadIdx.x * kSparsePer;
  uint32_t mv, ng;
  thread_votes<kKind>(src, bias, n, first, &mv, &ng);
  uint32_t total;
  uint32_t pos = blk[blockIdx.x] + block_exclusive_scan_256((uint32_t)__popc(mv), s_warp, &total);
  // a thread's entries are consecutive in the output: at most two sign words are touched
  uint32_t w0 = pos >> 5, bits0 = 0, bits1 = 0;
  while (mv) {
    const uint32_t q = (uint32_t)__ffs((int)mv) - 1u;
    if (pos < cap) {
      out_idx[pos] = index_base + (uint32_t)(first + q);
      const uint32_t bit = (ng >> q & 1u) << (pos & 31u);
      if ((pos >> 5) == w0) bits0 |= bit; else bits1 |= bit;
    }
    ++pos;
    mv &= mv - 1u;
  }
  if (bits0) atomicOr(out_signbits + w0, bits0);
  if (bits1) atomicOr(out_signbits + w0 + 1, bits1);
}

// x <- x - lr * vote from n_pieces sparse messages, piece_stride words apart: a piece is its count, then
// cap indices, then ceil(cap / 32) sign words.  One thread per (piece, entry).
__global__ void __launch_bounds__(256) sparse_apply_kernel(float* __restrict__ x, const uint32_t* __restrict__ msg,
                                                           uint32_t n_pieces, uint64_t piece_stride, uint32_t cap,
                                                           uint64_t d, float lr, uint32_t* __restrict__ bad_count) {
  const uint64_t total = (uint64_t)n_pieces * cap;
  const uint64_t stride = (uint64_t)gridDim.x * blockDim.x;
  uint32_t bad = 0;
  for (uint64_t e = (uint64_t)blockIdx.x * blockDim.x + threadIdx.x; e < total; e += stride) {
    const uint64_t p = e / cap, j = e - p * cap;
    const uint32_t* piece = msg + p * piece_stride;
    const uint32_t count = piece[0] < cap ? piece[0] : cap;
    if (j >= count) continue;
    const uint32_t n = piece[1 + j];
    const uint32_t neg = (piece[1 + cap + (j >> 5)] >> (j & 31)) & 1u;
    if (n < d) x[n] = neg ? __fadd_rn(x[n], lr) : __fsub_rn(x[n], lr);
    else ++bad;
  }
  if (bad && bad_count) atomicAdd(bad_count, bad);
}

}  // namespace
}  // namespace s3gd

using namespace s3gd;

extern "C" {

s3gd_status s3gd_vote_apply(float* x, const uint32_t* msg, int n_groups, uint64_t group_stride, int M_group,
                            uint64_t K, uint64_t d, float lr, int8_t* opt_vote, void* ws, size_t ws_bytes,
                            void* stream) {
  if (n_groups <= 0 || M_group <= 0 || (uint64_t)n_groups * (uint64_t)M_group > 65535u) return S3GD_ERR_INVALID_ARG;
  const int M = n_groups * M_group;
  Layout L;
  if (!make_layout(M, d, K, &L) || x == nullptr || !aligned(x, 4)) return S3GD_ERR_INVALID_ARG;
  const uint64_t piece = (uint64_t)M_group * (K + (K + 31) / 32);
  if (K > 0 && (msg == nullptr || !aligned(msg, 4) || group_stride < piece)) return S3GD_ERR_INVALID_ARG;
  if (ws == nullptr || ws_bytes < L.total || !aligned(ws, 256)) return S3GD_ERR_WORKSPACE;
  cudaStream_t st = static_cast<cudaStream_t>(stream);
  char* base = static_cast<char*>(ws);
  uint32_t* hdr = reinterpret_cast<uint32_t*>(base + L.off_hdr);
  int32_t* counter = reinterpret_cast<int32_t*>(base + L.off_counter);
  // every worker votes at most once per coordinate (the message's contract), so up to 127 workers fit bytes
  const bool packed = M <= kPackedMaxWorkers;
  if (cudaMemsetAsync(hdr, 0, kHdrWords * sizeof(uint32_t), st) != cudaSuccess) return S3GD_ERR_CUDA;
  const cudaError_t ez = packed ? cudaMemsetAsync(counter, 0x80, (size_t)((d + 3) / 4) * 4, st)
                                : cudaMemsetAsync(counter, 0, (size_t)d * sizeof(int32_t), st);
  if (ez != cudaSuccess) return S3GD_ERR_CUDA;
  const uint64_t total = (uint64_t)M * K;
  if (total) {
    vote_groups_kernel<<<grid_for(total, 256, sm_count() * 16), 256, 0, st>>>(
        msg, msg + (uint64_t)M_group * K, (uint32_t)n_groups, group_stride, (uint32_t)M_group, K, d, counter,
        packed ? 1u : 0u, hdr + kHdrBadIndex, hdr + kHdrStatus);
    if (cudaGetLastError() != cudaSuccess) return S3GD_ERR_CUDA;
    count_launch();
  }
  return launch_counter_apply(counter, packed, x, d, lr, opt_vote, total, st) == cudaSuccess ? S3GD_OK : S3GD_ERR_CUDA;
}

s3gd_status s3gd_vote_counts(const uint32_t* idx, const uint32_t* signbits, int M, uint64_t K, uint64_t d,
                             uint64_t d_padded, void* out_counts, int bytes_per_count, uint32_t* opt_bad_count,
                             void* stream) {
  if (M <= 0 || M > 65535 || d == 0 || d >= (1ull << 32) || K > d || d_padded < d || d_padded % 4 != 0 ||
      out_counts == nullptr || !aligned(out_counts, 4) || (bytes_per_count != 1 && bytes_per_count != 4))
    return S3GD_ERR_INVALID_ARG;
  if (bytes_per_count == 1 && M > kPackedMaxWorkers) return S3GD_ERR_INVALID_ARG;
  if (K > 0 && (idx == nullptr || signbits == nullptr || !aligned(idx, 4) || !aligned(signbits, 4)))
    return S3GD_ERR_INVALID_ARG;
  if (opt_bad_count != nullptr && !aligned(opt_bad_count, 4)) return S3GD_ERR_INVALID_ARG;
  cudaStream_t st = static_cast<cudaStream_t>(stream);
  const bool packed = bytes_per_count == 1;
  const uint64_t n_words = packed ? d_padded / 4 : d_padded;
  fill_words_kernel<<<grid_for(n_words, 256, sm_count() * 8), 256, 0, st>>>(static_cast<uint32_t*>(out_counts), n_words,
                                                                           packed ? kPackedZero : 0u);
  if (cudaGetLastError() != cudaSuccess) return S3GD_ERR_CUDA;
  count_launch();
  if (opt_bad_count && cudaMemsetAsync(opt_bad_count, 0, sizeof(uint32_t), st) != cudaSuccess) return S3GD_ERR_CUDA;
  const uint64_t total = (uint64_t)M * K;
  if (total) {
    vote_groups_kernel<<<grid_for(total, 256, sm_count() * 16), 256, 0, st>>>(
        idx, signbits, 1u, 0u, (uint32_t)M, K, d, static_cast<int32_t*>(out_counts), packed ? 1u : 0u, opt_bad_count,
        nullptr);
    if (cudaGetLastError() != cudaSuccess) return S3GD_ERR_CUDA;
    count_launch();
  }
  return S3GD_OK;
}

s3gd_status s3gd_encode_vote2(const void* src, int src_kind, uint32_t n_summed, uint64_t n, uint32_t* out_words,
                              void* stream) {
  if (src == nullptr || out_words == nullptr || n == 0 || !aligned(out_words, 4) || src_kind < 0 || src_kind > 2)
    return S3GD_ERR_INVALID_ARG;
  if (src_kind == 0 && !aligned(src, 4)) return S3GD_ERR_INVALID_ARG;
  cudaStream_t st = static_cast<cudaStream_t>(stream);
  const unsigned grid = grid_for((n + 15) / 16, 256, 0x7FFFFFFF);     // one thread per word: blocks that come and go
  const uint32_t bias = (128u * n_summed) & 0xFFu;
  if (src_kind == 0) encode2_kernel<0><<<grid, 256, 0, st>>>(src, 0u, n, out_words);
  else if (src_kind == 1) encode2_kernel<1><<<grid, 256, 0, st>>>(src, bias, n, out_words);
  else encode2_kernel<2><<<grid, 256, 0, st>>>(src, 0u, n, out_words);
  if (cudaGetLastError() != cudaSuccess) return S3GD_ERR_CUDA;
  count_launch();
  return S3GD_OK;
}

s3gd_status s3gd_apply_vote2(float* x, const uint32_t* words, uint64_t d, float lr, int8_t* opt_vote, void* stream) {
  if (x == nullptr || words == nullptr || d == 0 || d >= (1ull << 32) || !aligned(x, 4) || !aligned(words, 4))
    return S3GD_ERR_INVALID_ARG;
  cudaStream_t st = static_cast<cudaStream_t>(stream);
  apply2_kernel<<<grid_for((d + 15) / 16, 256, 0x7FFFFFFF), 256, 0, st>>>(x, words, d, lr, opt_vote);
  if (cudaGetLastError() != cudaSuccess) return S3GD_ERR_CUDA;
  count_launch();
  return S3GD_OK;
}

size_t s3gd_sparse_workspace_bytes(uint64_t n) {
  if (n == 0 || n >= (1ull << 32)) return 0;
  return (size_t)((n + kSparseBlock - 1) / kSparseBlock) * sizeof(uint32_t);
}

s3gd_status s3gd_encode_vote_sparse(const void* src, int src_kind, uint32_t n_summed, uint64_t n, uint32_t index_base,
                                    uint32_t cap, uint32_t* out_piece, void* ws, size_t ws_bytes, void* stream) {
  if (src == nullptr || out_piece == nullptr || n == 0 || n >= (1ull << 32) || cap == 0 || !aligned(out_piece, 4) ||
      src_kind < 0 || src_kind > 2 || (uint64_t)index_base + n > (1ull << 32))
    return S3GD_ERR_INVALID_ARG;
  if (src_kind == 0 && !aligned(src, 4)) return S3GD_ERR_INVALID_ARG;
  const size_t need = s3gd_sparse_workspace_bytes(n);
  if (ws == nullptr || ws_bytes < need || !aligned(ws, 4)) return S3GD_ERR_WORKSPACE;
  cudaStream_t st = static_cast<cudaStream_t>(stream);
  uint32_t* blk = static_cast<uint32_t*>(ws);
  const uint32_t n_blocks = (uint32_t)((n + kSparseBlock - 1) / kSparseBlock);
  const uint32_t bias = (128u * n_summed) & 0xFFu;
  uint32_t* out_idx = out_piece + 1;
  uint32_t* out_sgn = out_piece + 1 + cap;
  if (cudaMemsetAsync(out_sgn, 0, (size_t)((cap + 31) / 32) * sizeof(uint32_t), st) != cudaSuccess) return S3GD_ERR_CUDA;
  if (src_kind == 0) sparse_count_kernel<0><<<n_blocks, kSparseThreads, 0, st>>>(src, 0u, n, blk);
  else if (src_kind == 1) sparse_count_kernel<1><<<n_blocks, kSparseThreads, 0, st>>>(src, bias, n, blk);
  else sparse_count_kernel<2><<<n_blocks, kSparseThreads, 0, st>>>(src, 0u, n, blk);
  sparse_scan_kernel<<<1, kSparseThreads, 0, st>>>(blk, n_blocks, out_piece);
  if (src_kind == 0) sparse_emit_kernel<0><<<n_blocks, kSparseThreads, 0, st>>>(src, 0u, n, index_base, blk, cap, out_idx, out_sgn);
  else if (src_kind == 1) sparse_emit_kernel<1><<<n_blocks, kSparseThreads, 0, st>>>(src, bias, n, index_base, blk, cap, out_idx, out_sgn);
  else sparse_emit_kernel<2><<<n_blocks, kSparseThreads, 0, st>>>(src, 0u, n, index_base, blk, cap, out_idx, out_sgn);
  if (cudaGetLastError() != cudaSuccess) return S3GD_ERR_CUDA;
  count_launch(3);
  return S3GD_OK;
}

s3gd_status s3gd_apply_vote_sparse(float* x, const uint32_t* pieces, int n_pieces, uint64_t piece_stride, uint32_t cap,
                                   uint64_t d, float lr, uint32_t* opt_bad_count, void* stream) {
  if (x == nullptr || pieces == nullptr || n_pieces <= 0 || cap == 0 || d == 0 || d >= (1ull << 32) || !aligned(x, 4) ||
      !aligned(pieces, 4) || piece_stride < 1ull + cap + (cap + 31) / 32)
    return S3GD_ERR_INVALID_ARG;
  if (opt_bad_count != nullptr && !aligned(opt_bad_count, 4)) return S3GD_ERR_INVALID_ARG;
  cudaStream_t st = static_cast<cudaStream_t>(stream);
  if (opt_bad_count && cudaMemsetAsync(opt_bad_count, 0, sizeof(uint32_t), st) != cudaSuccess) return S3GD_ERR_CUDA;
  sparse_apply_kernel<<<grid_for((uint64_t)n_pieces * cap, 256, sm_count() * 16), 256, 0, st>>>(
      x, pieces, (uint32_t)n_pieces, piece_stride, cap, d, lr, opt_bad_count);
  if (cudaGetLastError() != cudaSuccess) return S3GD_ERR_CUDA;
  count_launch();
  return S3GD_OK;
}

}  // extern "C"

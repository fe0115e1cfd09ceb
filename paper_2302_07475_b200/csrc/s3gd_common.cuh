// Shared declarations of the S3GD-MV CUDA library (sm_100a): workspace layout,
// per-row selection state, small device helpers.  Internal; the public
// interface is include/s3gd.h.
#pragma once

#include <cuda_runtime.h>
#include <stddef.h>
#include <stdint.h>

#include "s3gd.h"

namespace s3gd {

// ------------------------------------------------------------------ geometry
constexpr int kTileThreads = 256;                  // threads of a streaming CTA
constexpr int kTileIters = 8;                      // 16-byte loads per thread per tile
constexpr int kTileElems = kTileThreads * kTileIters * 4;   // 8192 gradient entries per tile
constexpr int kWarpsPerTile = kTileThreads / 32;

constexpr int kHistBins = 2048;                    // 11-bit digit of the first radix pass
constexpr int kNumPasses = 3;                      // 11 + 10 + 10 bits = the 31 magnitude bits
__host__ __device__ constexpr int pass_shift(int p) { return p == 0 ? 20 : (p == 1 ? 10 : 0); }
__host__ __device__ constexpr int pass_bits(int p) { return p == 0 ? 11 : 10; }

constexpr int kSampleBins = 32768;                 // magnitude >> 16: sign-less bf16 pattern
constexpr uint32_t kAbsMask = 0x7FFFFFFFu;

constexpr int kDefaultSMs = 148;                   // B200; used only if the device query fails
constexpr int kMaxDevices = 64;                    // per-device host caches are this long

// SMs of the current device (asked once per device).  Grids are sized in multiples of it.
int sm_count();
// cudaFuncSetAttribute(func, MaxDynamicSharedMemorySize, bytes), issued once per device and
// kernel: `done` is a zero-initialised array of kMaxDevices flags owned by the call site.
cudaError_t opt_in_dynamic_smem(const void* func, int bytes, int* done);

// --------------------------------------------------------------- device state
// Header at the start of the workspace (64 x uint32).
enum HeaderWord : int {
  kHdrStatus = 0,        // bit mask of DeviceFlag
  kHdrExactRows = 1,     // rows that took the exact multi-pass route
  kHdrBadIndex = 2,      // out-of-range indices skipped by the vote scatter
  kHdrBadCount = 3,      // rows whose selection size != K
  kHdrMaxCand = 4,       // largest candidate count of a row
  kHdrRowsDone = 8,      // rows finished by the single-CTA selection (words 5..7 are reported as 0)
  kHdrWords = 64
};
enum DeviceFlag : uint32_t { kFlagIndexRange = 1u, kFlagInternal = 2u };

// Selection state of one worker (row).  64 bytes.
struct RowState {
  uint32_t tau_lo;     // conservative magnitude threshold from the sample
  uint32_t n_cand;     // entries with magnitude >= tau_lo found by the filter pass
  uint32_t prefix;     // magnitude bits fixed so far by the radix passes
  uint32_t k_rem;      // entries still to take among those matching prefix
  uint32_t tau;        // K-th largest magnitude (valid after the last pass)
  uint32_t take_ties;  // how many entries equal to tau are kept (lowest indices)
  uint32_t n_emitted;  // entries written by the emit pass (checked against K)
  uint32_t exact;      // 1: this row uses the exact multi-pass route over the whole row
  uint32_t ticket_hist;   // blocks of the current histogram pass that have finished this row
  uint32_t ticket_count;  // blocks of the count pass that have finished this row
  uint32_t done;          // 0: open; 1: finished by an on-chip selection; 2, 3: taken by the two-pass form (s3gd_select.cu)
  uint32_t n_bin;         // entries collected so far in the row's bin list (two-pass form, votes only)
  uint32_t tau_hi;        // band form of the filter pass: entries with magnitude >= tau_hi voted during that pass
                          // (kNoPrevote: no entry did); the candidates are then the band [tau_lo, tau_hi)
  uint32_t n_hi;          // how many entries voted during the filter pass
  uint32_t pad[2];
};
static_assert(sizeof(RowState) == 64, "one row state per 64 bytes");
constexpr uint32_t kNoPrevote = 0x80000000u;       // above every magnitude key

// Byte offsets of the workspace regions; computed identically for sizing and use.
struct Layout {
  uint64_t d, K;
  int M;
  uint32_t n_tiles;      // tiles per row
  uint32_t cap;          // candidate capacity per row
  uint32_t typical_cand; // survivors a row is expected to have (mean of the sampling plan plus grid slack)
  uint32_t n_sample;     // sampled entries per row
  uint32_t j_rank;       // sample rank that fixes tau_lo
  uint32_t j_hi_rank;    // sample rank that fixes tau_hi in the band form (0: nothing votes during the filter pass)
  uint32_t sample_stride;  // distance between sampled groups of 8 (0: whole row sampled)
  uint32_t bin_cap;      // entries per row of the bin list (0: none)
  bool dense;            // survivors are expected in nearly every 128-entry step of the filter pass
  size_t off_hdr, off_rows, off_hist, off_seg, off_segscan, off_cand, off_bin, off_counter, total;
};

bool make_layout(int M, uint64_t d, uint64_t K, Layout* L);

inline size_t align_up(size_t v, size_t a) { return (v + a - 1) / a * a; }

// ------------------------------------------------------------ device helpers
#ifdef __CUDACC__
__device__ __forceinline__ uint32_t lane_id() { return threadIdx.x & 31; }
__device__ __forceinline__ uint32_t lanemask_lt() {
  uint32_t m;
  asm("mov.u32 %0, %%lanemask_lt;" : "=r"(m));
  return m;
}

// Streaming loads: the gradients are read once, so keep them out of L1.
__device__ __forceinline__ uint4 ld_stream_v4(const void* p) {
  uint4 v;
  asm volatile("ld.global.nc.L1::no_allocate.v4.u32 {%0,%1,%2,%3}, [%4];"
               : "=r"(v.x), "=r"(v.y), "=r"(v.z), "=r"(v.w) : "l"(p));
  return v;
}
__device__ __forceinline__ uint2 ld_stream_v2(const void* p) {
  uint2 v;
  asm volatile("ld.global.nc.L1::no_allocate.v2.u32 {%0,%1}, [%2];" : "=r"(v.x), "=r"(v.y) : "l"(p));
  return v;
}
__device__ __forceinline__ uint32_t ld_stream_u32(const void* p) {
  uint32_t v;
  asm volatile("ld.global.nc.L1::no_allocate.u32 %0, [%1];" : "=r"(v) : "l"(p));
  return v;
}

// RowState::done beyond 0 (open) and 1 (finished on chip): rows the two-pass form of the general
// selection has taken (s3gd_select.cu).  kRowTwoPass: last histogram pass, count and emission follow;
// kRowBin (votes only): the entries of the K-th magnitude's bin are collected and one CTA finishes them.
constexpr uint32_t kRowTwoPass = 2u, kRowBin = 3u;

// Does this row take its top-K from the filtered candidates (true) or from the whole row?
// Band form: the n_hi entries at or above tau_hi have voted already.  They are the n_hi largest of
// the row, so they belong to the top K exactly if n_hi <= K, and the other K - n_hi are then the
// largest of the band, provided it holds that many.  (n_hi is 0 in the plain form.)  A row whose early
// votes are exactly K has nothing left to select; the selections all look for at least one entry, so
// that rare row is redone as well.
__device__ __forceinline__ bool row_uses_candidates(const RowState& rs, uint32_t K, uint32_t cap) {
  return rs.exact == 0u && rs.n_hi < K && rs.n_cand >= K - rs.n_hi && rs.n_cand <= cap;
}
// Shared memory the single-CTA selection needs for a row: bit pattern and index of every
// candidate.  Rows that fit are finished by that kernel; the others by the general passes.
constexpr uint32_t kSmallSelectBytes = 212 * 1024;
__host__ __device__ __forceinline__ bool fits_single_cta(uint32_t n_cand) {
  return (uint64_t)n_cand * 8u <= kSmallSelectBytes;
}
#endif

// Vote counters.  Plain form: one int32 per coordinate.  Packed form (fused steps with at most
// kPackedMaxWorkers workers, each of which votes at most once per coordinate): one byte per
// coordinate holding 128 + (sum of votes), four coordinates per 32-bit word.  A vote adds or
// subtracts 1 << (8 * slot) in the word; because every byte stays within [1, 255] no carry or
// borrow ever crosses into a neighbour, so one 32-bit atomic serves.  A quarter of the bytes
// means the counters of a 25M-coordinate model stay in L2 while the votes arrive at random.
constexpr int kPackedMaxWorkers = 127;
constexpr uint32_t kPackedZero = 0x80808080u;
#ifdef __CUDACC__
__device__ __forceinline__ void add_vote(int32_t* counter, uint32_t packed, uint32_t idx, uint32_t neg) {
  if (packed) {
    const uint32_t inc = 1u << ((idx & 3u) * 8u);
    atomicAdd(reinterpret_cast<uint32_t*>(counter) + (idx >> 2), neg ? 0u - inc : inc);
  } else {
    atomicAdd(counter + idx, neg ? -1 : 1);
  }
}
#endif

// ------------------------------------------------------------------ launches that overlap their predecessor's tail
// launch_after(): the kernel's blocks may be scheduled while the previous kernel on the stream is still
// draining (programmatic stream serialization); the kernel must call grid_dependency_wait() before it
// touches anything, which returns once every earlier kernel has completed and its writes are visible.
// In a kernel launched the ordinary way the wait returns at once.
#ifdef __CUDACC__
__device__ __forceinline__ void grid_dependency_wait() { asm volatile("griddepcontrol.wait;" ::: "memory"); }
template <typename... KArgs, typename... Args>
inline cudaError_t launch_after(void (*kernel)(KArgs...), dim3 grid, dim3 block, size_t smem, cudaStream_t st,
                                Args&&... args) {
  cudaLaunchConfig_t cfg = {};
  cfg.gridDim = grid; cfg.blockDim = block; cfg.dynamicSmemBytes = smem; cfg.stream = st;
  cudaLaunchAttribute attr[1];
  attr[0].id = cudaLaunchAttributeProgrammaticStreamSerialization;
  attr[0].val.programmaticStreamSerializationAllowed = 1;
  cfg.attrs = attr; cfg.numAttrs = 1;
  return cudaLaunchKernelEx(&cfg, kernel, static_cast<KArgs>(args)...);
}
#endif

// ------------------------------------------------------------------ profiling
// Optional event marks at the phase boundaries of s3gd_step (see s3gd_profile_begin).
enum Phase : int { kPhaseStart = 0, kPhaseSampled, kPhaseFiltered, kPhaseThreshold, kPhaseEmitted, kPhaseApplied,
                   kPhaseMarks };
void prof_mark(int phase, cudaStream_t st);   // no-op unless profiling is on
void count_launch(int n = 1);                 // bookkeeping of kernels enqueued by this library

// ------------------------------------------------------------ kernel launchers
// (each returns the cudaError_t of its launches; all work goes to `st`)
cudaError_t launch_apply(float* x, const int8_t* vote, uint64_t d, float lr, cudaStream_t st);
cudaError_t launch_vote_scatter(const uint32_t* idx, const uint32_t* signbits, int M, uint64_t K, uint64_t d,
                                int32_t* counter, uint32_t* hdr, cudaStream_t st);
cudaError_t launch_counter_sign(const int32_t* counter, uint64_t d, int8_t* vote, cudaStream_t st);
// max_votes: an upper bound on the votes the counters hold (0 = unknown); when they are at most one per
// kSparseVotesRatio coordinates the packed form is read in a way that suits mostly untouched counters
constexpr uint64_t kSparseVotesRatio = 64;
cudaError_t launch_counter_apply(const int32_t* counter, bool packed, float* x, uint64_t d, float lr, int8_t* opt_vote,
                                 uint64_t max_votes, cudaStream_t st);
cudaError_t launch_signplane_step(float* x, const float* grads, int M, uint64_t d, float lr, int8_t* opt_vote,
                                  cudaStream_t st);
cudaError_t launch_signplane_message(const float* grads, int M, uint64_t d, uint32_t* out_idx,
                                     uint32_t* out_signbits, cudaStream_t st);
cudaError_t launch_sample_and_filter(const uint32_t* gbits, const Layout& L, RowState* rows, uint2* cand, uint2* seg,
                                     uint32_t* hdr, uint32_t* hist, float* ef_err, float eta, int32_t* zero_counter,
                                     bool packed, bool band, cudaStream_t st);
// (zero_counter != NULL: the d vote counters there, 16-byte aligned, are cleared by the sampling launch;
//  band: the band form of the filter pass -- entries at or above a second sampled threshold vote into
//  zero_counter at once and only the band between the two thresholds is listed, in no particular order)
struct EmitOut {
  uint32_t* idx;        // [M x K] or NULL
  uint32_t* signbits;   // [M x words] or NULL (zeroed before the launch)
  int32_t* counter;     // [d] or NULL
  uint32_t packed;      // 1: the counters are bytes (see add_vote)
  uint32_t unordered;   // 1: the candidate lists are in no particular order (band form of the filter pass)
  float* err;           // [M x d] or NULL: error memory whose kept entries are set to zero (Eq. (6))
  uint64_t d;
  uint32_t K, words;
};
cudaError_t launch_select_small(const Layout& L, RowState* rows, const uint2* cand, const uint2* seg, uint32_t* hdr,
                                const EmitOut& o, cudaStream_t st);
// Votes only, two-pass form: one CTA per row finishes the rows marked kRowBin from their bin lists
// (bin_cap: entries per row of the list; lists longer than one CTA's shared memory are selected from where they lie)
cudaError_t launch_select_bin(const Layout& L, RowState* rows, const uint2* bin, uint32_t bin_cap, uint32_t* hdr,
                              const EmitOut& o, cudaStream_t st);
// Votes only, rows too large for one SM: a cluster of 2 or 4 CTAs per row (cluster_size_for; 0 = none fits)
uint32_t cluster_size_for(uint32_t n_cand);
cudaError_t launch_select_cluster(const Layout& L, RowState* rows, const uint2* cand, uint32_t* hdr, const EmitOut& o,
                                  uint32_t cluster, cudaStream_t st);
// Top-K selection of every row; writes the message if out_idx != NULL and adds the
// votes into counter if counter != NULL.
cudaError_t launch_select(const float* grads, const Layout& L, void* ws, uint32_t* out_idx, uint32_t* out_signbits,
                          int32_t* counter, bool packed, float* err_to_clear, const float* ef_raw, float eta,
                          cudaStream_t st);
// Does launch_select clear the counters it adds into (true), or must the caller do so first?
bool select_clears_counter(const Layout& L);
// (ef_raw != NULL: error compensation fused into the filter pass -- ef_raw are the raw gradients g~,
//  `grads` is the error memory, which holds e on entry and g = g~ + eta * e after the filter pass)
// err <- grads + eta * err, element-wise over n entries (Eq. (5))
cudaError_t launch_ef_accumulate(float* err, const float* grads, float eta, uint64_t n, cudaStream_t st);
// v <- mu * v + sgn(counter); x <- x - lr * v (momentum form of the update)
cudaError_t launch_counter_apply_momentum(const int32_t* counter, bool packed, float* x, float* v, uint64_t d, float mu,
                                          float lr, int8_t* opt_vote, cudaStream_t st);
cudaError_t launch_apply_momentum(float* x, float* v, const int8_t* vote, uint64_t d, float mu, float lr,
                                  cudaStream_t st);
// counter[n] <- sum over workers of (+1 | -1) by sign bit (K = d, when the sign counts are needed as such)
cudaError_t launch_signplane_counts(const float* grads, int M, uint64_t d, int32_t* counter, cudaStream_t st);
// RandKSign of every row under (seed, step): message if out_idx != NULL, votes added into counter if != NULL
cudaError_t launch_randk(const float* grads, int M, uint64_t d, uint64_t K, uint32_t seed, uint32_t step,
                         uint32_t* out_idx, uint32_t* out_signbits, int32_t* counter, bool packed, uint32_t* hdr,
                         cudaStream_t st);

}  // namespace s3gd

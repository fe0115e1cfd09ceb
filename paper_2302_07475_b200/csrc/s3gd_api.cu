// C ABI of the library: argument checks, workspace layout, and the order in which
// the kernels of each call are enqueued.  See include/s3gd.h for the contract.
#include <math.h>

#include <atomic>

#include "s3gd_common.cuh"

namespace s3gd {

// Workspace regions for (M, d, K).  The same function sizes the workspace and
// locates the regions at run time, so the two can never disagree.
//
// Sampling plan (only for K <= d/4, otherwise rows are selected with full passes):
//   n_sample = 65536 entries per row are inspected (all of them for short rows); if p = K/d, the number of sampled entries
//   that belong to the true top-K is ~ Binomial(n_sample, p) with mean s = n_sample * p.
//   tau_lo is put at sample rank j = s + 6 sqrt(s) + 4, so the chance that fewer than K
//   entries pass the filter is below about 1e-8; the expected number that pass is
//   j * d / n_sample, and `cap` leaves room for 6 standard deviations, for the coarse
//   threshold grid (2^-7 relative) and for ties.  Exceeding either bound only makes the
//   row take the full-pass route.
bool make_layout(int M, uint64_t d, uint64_t K, Layout* L) {
  if (M <= 0 || M > 65535 || d == 0 || d >= (1ull << 32) || K > d) return false;
  L->M = M; L->d = d; L->K = K;
  L->n_tiles = (uint32_t)((d + kTileElems - 1) / kTileElems);
  L->cap = 0; L->typical_cand = 0; L->n_sample = 0; L->j_rank = 0; L->sample_stride = 0;
  L->j_hi_rank = 0; L->dense = false;
  const bool use_filter = K > 0 && K < d && K * 4 <= d;
  if (use_filter) {
    const double p = (double)K / (double)d;
    const uint64_t s_target = 65536;       // 2048 chunks of 32 neighbouring entries
    double j;
    if (d <= 2 * s_target) {
      L->n_sample = (uint32_t)d;
      L->sample_stride = 0;
      j = (double)K;                       // the whole row is inspected: rank K is exact
    } else {
      const uint64_t chunks = s_target / 32;
      L->sample_stride = (uint32_t)(d / chunks);
      L->n_sample = (uint32_t)(chunks * 32);
      const double s = (double)L->n_sample * p;
      j = ceil(s + 6.0 * sqrt(s) + 4.0);
      // the mirror image for the band form: with at most j_hi sampled entries at or above tau_hi, the
      // chance that more than K entries of the row are is as small as the one above
      const double jh = floor(s - 6.0 * sqrt(s) - 4.0);
      L->j_hi_rank = jh >= 1.0 ? (uint32_t)jh : 0u;
    }
    if (j > (double)L->n_sample) j = (double)L->n_sample;
    if (j < 1.0) j = 1.0;
    L->j_rank = (uint32_t)j;
    const double r = (double)d / (double)L->n_sample;
    double cap = ceil(r * (j + 6.0 * sqrt(j) + 8.0) * 1.25) + 1024.0;
    if (cap < (double)K) cap = (double)K;
    if (cap > (double)d) cap = (double)d;
    L->cap = (uint32_t)cap;
    double typical = ceil(r * j * 1.25);
    if (typical > cap) typical = cap;
    L->typical_cand = (uint32_t)typical;
    L->dense = (uint64_t)L->typical_cand * 250u > d;
  }
  size_t off = 0;
  L->off_hdr = off;      off = align_up(off + kHdrWords * sizeof(uint32_t), 256);
  L->off_rows = off;     off = align_up(off + (size_t)M * sizeof(RowState), 256);
  L->off_hist = off;     off = align_up(off + (size_t)M * kHistBins * sizeof(uint32_t), 256);
  L->off_seg = off;      off = align_up(off + (size_t)M * L->n_tiles * sizeof(uint2), 256);
  L->off_segscan = off;  off = align_up(off + (size_t)M * L->n_tiles * sizeof(uint2), 256);
  L->off_cand = off;     off = align_up(off + (size_t)M * L->cap * sizeof(uint2), 256);
  // bin list of the two-pass selection: room for a whole row's candidates, because the band form of the
  // filter pass leaves its list unordered and has no other route for a row whose bin is long
  L->bin_cap = L->cap;
  L->off_bin = off;      off = align_up(off + (size_t)M * L->bin_cap * sizeof(uint2), 256);
  L->off_counter = off;  off = align_up(off + (size_t)d * sizeof(int32_t), 256);
  L->total = off;
  return true;
}

// ------------------------------------------------------- per-device host caches
// Filled on first use and never changed afterwards; two threads that race on the first use
// store the same value, so relaxed atomics are enough.
namespace {
std::atomic<int> g_sm_count[kMaxDevices];
}  // namespace

int sm_count() {
  int dev = 0;
  if (cudaGetDevice(&dev) != cudaSuccess || dev < 0 || dev >= kMaxDevices) return kDefaultSMs;
  int n = g_sm_count[dev].load(std::memory_order_relaxed);
  if (n == 0) {
    if (cudaDeviceGetAttribute(&n, cudaDevAttrMultiProcessorCount, dev) != cudaSuccess || n <= 0) n = kDefaultSMs;
    g_sm_count[dev].store(n, std::memory_order_relaxed);
  }
  return n;
}

cudaError_t opt_in_dynamic_smem(const void* func, int bytes, int* done) {
  int dev = 0;
  cudaError_t e = cudaGetDevice(&dev);
  if (e != cudaSuccess) return e;
  const bool cached = dev >= 0 && dev < kMaxDevices;
  if (cached && __atomic_load_n(&done[dev], __ATOMIC_RELAXED) >= bytes) return cudaSuccess;
  e = cudaFuncSetAttribute(func, cudaFuncAttributeMaxDynamicSharedMemorySize, bytes);
  if (e == cudaSuccess && cached) __atomic_store_n(&done[dev], bytes, __ATOMIC_RELAXED);
  return e;
}

// ---------------------------------------------------------------- profiling
namespace {
struct Profiler {
  bool on = false;
  bool filter_only = false;           // record only the two marks around the filter pass
  int max_steps = 0, n_steps = 0;     // steps to record at most / recorded so far
  int every = 1, n_calls = 0;         // every `every`-th step is recorded / steps seen so far
  cudaEvent_t* ev = nullptr;          // kPhaseMarks events per recorded step
} g_prof;
std::atomic<unsigned long long> g_launches{0};   // kernels enqueued while a profiling session is open
}  // namespace

void prof_mark(int phase, cudaStream_t st) {
  if (!g_prof.on) return;
  const bool recorded = g_prof.n_steps < g_prof.max_steps && g_prof.n_calls % g_prof.every == 0;
  if (recorded && (!g_prof.filter_only || phase == kPhaseSampled || phase == kPhaseFiltered))
    cudaEventRecord(g_prof.ev[(size_t)g_prof.n_steps * kPhaseMarks + phase], st);
  if (phase == kPhaseApplied) {                  // the last mark of a step
    if (recorded) ++g_prof.n_steps;
    ++g_prof.n_calls;
  }
}

void count_launch(int n) {
  if (g_prof.on) g_launches.fetch_add((unsigned long long)n, std::memory_order_relaxed);
}

namespace {

inline bool aligned(const void* p, size_t a) { return (reinterpret_cast<uintptr_t>(p) % a) == 0; }

s3gd_status check_ws(const Layout& L, const void* ws, size_t ws_bytes) {
  if (ws == nullptr || ws_bytes < L.total || !aligned(ws, 256)) return S3GD_ERR_WORKSPACE;
  return S3GD_OK;
}

inline s3gd_status from_cuda(cudaError_t e) { return e == cudaSuccess ? S3GD_OK : S3GD_ERR_CUDA; }

#define S3GD_TRY(expr)                                  \
  do {                                                  \
    cudaError_t e_ = (expr);                            \
    if (e_ != cudaSuccess) return S3GD_ERR_CUDA;        \
  } while (0)

}  // namespace
}  // namespace s3gd

using namespace s3gd;

extern "C" {

const char* s3gd_status_string(s3gd_status st) {
  switch (st) {
    case S3GD_OK: return "S3GD_OK";
    case S3GD_ERR_INVALID_ARG: return "S3GD_ERR_INVALID_ARG";
    case S3GD_ERR_WORKSPACE: return "S3GD_ERR_WORKSPACE";
    case S3GD_ERR_CUDA: return "S3GD_ERR_CUDA";
    case S3GD_ERR_INDEX_RANGE: return "S3GD_ERR_INDEX_RANGE";
    case S3GD_ERR_INTERNAL: return "S3GD_ERR_INTERNAL";
    case S3GD_ERR_TOO_LARGE: return "S3GD_ERR_TOO_LARGE";
  }
  return "S3GD_ERR_UNKNOWN";
}

size_t s3gd_workspace_bytes(int M, uint64_t d, uint64_t K) {
  Layout L;
  return make_layout(M, d, K, &L) ? L.total : 0;
}

namespace {
// sample_rank != 0 replaces the sampling plan's rank (the debug entry points); the workspace
// layout, and with it the candidate capacity, stays that of the plan.
void override_sample_rank(Layout* L, uint32_t sample_rank, uint32_t prevote_rank) {
  if (L->cap == 0u) return;
  if (sample_rank != 0u) L->j_rank = sample_rank < L->n_sample ? sample_rank : L->n_sample;
  if (prevote_rank != 0u) L->j_hi_rank = prevote_rank < L->n_sample ? prevote_rank : L->n_sample;
}

s3gd_status topk_sign_impl(const float* grads, int M, uint64_t d, uint64_t K, uint32_t* out_idx,
                           uint32_t* out_signbits, void* ws, size_t ws_bytes, void* stream, uint32_t sample_rank) {
  Layout L;
  if (!make_layout(M, d, K, &L) || grads == nullptr || !aligned(grads, 4)) return S3GD_ERR_INVALID_ARG;
  override_sample_rank(&L, sample_rank, 0u);
  if (K > 0 && (out_idx == nullptr || out_signbits == nullptr || !aligned(out_idx, 4) || !aligned(out_signbits, 4)))
    return S3GD_ERR_INVALID_ARG;
  s3gd_status s = check_ws(L, ws, ws_bytes);
  if (s != S3GD_OK) return s;
  cudaStream_t st = static_cast<cudaStream_t>(stream);
  char* base = static_cast<char*>(ws);
  if (K == 0 || K == d) {
    S3GD_TRY(cudaMemsetAsync(base + L.off_hdr, 0, kHdrWords * sizeof(uint32_t), st));
    if (K == d) S3GD_TRY(launch_signplane_message(grads, M, d, out_idx, out_signbits, st));
    return S3GD_OK;
  }
  S3GD_TRY(cudaMemsetAsync(out_signbits, 0, (size_t)M * ((K + 31) / 32) * sizeof(uint32_t), st));
  return from_cuda(launch_select(grads, L, ws, out_idx, out_signbits, nullptr, false, nullptr, nullptr, 0.f, st));
}
}  // namespace

s3gd_status s3gd_topk_sign(const float* grads, int M, uint64_t d, uint64_t K, uint32_t* out_idx,
                           uint32_t* out_signbits, void* ws, size_t ws_bytes, void* stream) {
  return topk_sign_impl(grads, M, d, K, out_idx, out_signbits, ws, ws_bytes, stream, 0u);
}

s3gd_status s3gd_debug_topk_sign(const float* grads, int M, uint64_t d, uint64_t K, uint32_t* out_idx,
                                 uint32_t* out_signbits, void* ws, size_t ws_bytes, void* stream,
                                 uint32_t sample_rank) {
  return topk_sign_impl(grads, M, d, K, out_idx, out_signbits, ws, ws_bytes, stream, sample_rank);
}

s3gd_status s3gd_majority_vote(const uint32_t* idx, const uint32_t* signbits, int M, uint64_t K, uint64_t d,
                               int8_t* out_vote, void* ws, size_t ws_bytes, void* stream) {
  Layout L;
  if (!make_layout(M, d, K, &L) || out_vote == nullptr) return S3GD_ERR_INVALID_ARG;
  if (K > 0 && (idx == nullptr || signbits == nullptr || !aligned(idx, 4) || !aligned(signbits, 4)))
    return S3GD_ERR_INVALID_ARG;
  s3gd_status s = check_ws(L, ws, ws_bytes);
  if (s != S3GD_OK) return s;
  cudaStream_t st = static_cast<cudaStream_t>(stream);
  char* base = static_cast<char*>(ws);
  uint32_t* hdr = reinterpret_cast<uint32_t*>(base + L.off_hdr);
  int32_t* counter = reinterpret_cast<int32_t*>(base + L.off_counter);
  S3GD_TRY(cudaMemsetAsync(hdr, 0, kHdrWords * sizeof(uint32_t), st));
  S3GD_TRY(cudaMemsetAsync(counter, 0, (size_t)d * sizeof(int32_t), st));
  S3GD_TRY(launch_vote_scatter(idx, signbits, M, K, d, counter, hdr, st));
  S3GD_TRY(launch_counter_sign(counter, d, out_vote, st));
  return S3GD_OK;
}

s3gd_status s3gd_apply(float* x, const int8_t* vote, uint64_t d, float lr, void* stream) {
  if (x == nullptr || vote == nullptr || d == 0 || d >= (1ull << 32) || !aligned(x, 4)) return S3GD_ERR_INVALID_ARG;
  return from_cuda(launch_apply(x, vote, d, lr, static_cast<cudaStream_t>(stream)));
}

namespace {

// The step on `sel` (the gradients the selection looks at).  err_to_clear: error memory whose kept
// entries are zeroed (it is `sel` itself when error compensation is on).  v: momentum buffer or NULL.
s3gd_status step_impl(float* x, const float* sel, float* err_to_clear, float* v, float mu, int M, uint64_t d,
                      uint64_t K, float lr, uint32_t* opt_idx, uint32_t* opt_signbits, int8_t* opt_vote,
                      const Layout& L, void* ws, cudaStream_t st, bool mark_start = true,
                      const float* ef_raw = nullptr, float eta = 0.f) {
  char* base = static_cast<char*>(ws);
  int32_t* counter = reinterpret_cast<int32_t*>(base + L.off_counter);
  if (K == 0 || K == d) {
    S3GD_TRY(cudaMemsetAsync(base + L.off_hdr, 0, kHdrWords * sizeof(uint32_t), st));
    for (int ph = mark_start ? kPhaseStart : kPhaseSampled; ph < kPhaseApplied; ++ph) prof_mark(ph, st);
    if (K == 0) {
      if (opt_vote) S3GD_TRY(cudaMemsetAsync(opt_vote, 0, (size_t)d, st));
      if (v) {                                 // no votes, but the momentum still decays and moves x
        S3GD_TRY(cudaMemsetAsync(counter, 0, (size_t)d * sizeof(int32_t), st));
        S3GD_TRY(launch_counter_apply_momentum(counter, false, x, v, d, mu, lr, nullptr, st));
      }
      prof_mark(kPhaseApplied, st);
      return S3GD_OK;
    }
    if (opt_idx) S3GD_TRY(launch_signplane_message(sel, M, d, opt_idx, opt_signbits, st));
    if (v) {
      S3GD_TRY(launch_signplane_counts(sel, M, d, counter, st));
      S3GD_TRY(launch_counter_apply_momentum(counter, false, x, v, d, mu, lr, opt_vote, st));
    } else {
      S3GD_TRY(launch_signplane_step(x, sel, M, d, lr, opt_vote, st));
    }
    if (err_to_clear) S3GD_TRY(cudaMemsetAsync(err_to_clear, 0, (size_t)M * d * sizeof(float), st));   // everything was kept
    prof_mark(kPhaseApplied, st);
    return S3GD_OK;
  }
  if (mark_start) prof_mark(kPhaseStart, st);
  // every worker votes at most once per coordinate here, so up to 127 workers fit byte counters
  const bool packed = M <= kPackedMaxWorkers;
  if (!select_clears_counter(L)) {
    if (packed) S3GD_TRY(cudaMemsetAsync(counter, 0x80, (size_t)((d + 3) / 4) * 4, st));
    else S3GD_TRY(cudaMemsetAsync(counter, 0, (size_t)d * sizeof(int32_t), st));
  }
  if (opt_signbits) S3GD_TRY(cudaMemsetAsync(opt_signbits, 0, (size_t)M * ((K + 31) / 32) * sizeof(uint32_t), st));
  S3GD_TRY(launch_select(sel, L, ws, opt_idx, opt_signbits, counter, packed, err_to_clear, ef_raw, eta, st));
  cudaError_t e = v ? launch_counter_apply_momentum(counter, packed, x, v, d, mu, lr, opt_vote, st)
                    : launch_counter_apply(counter, packed, x, d, lr, opt_vote, (uint64_t)M * K, st);
  prof_mark(kPhaseApplied, st);
  return from_cuda(e);
}

s3gd_status check_step_args(const float* x, const float* grads, uint32_t* opt_idx, uint32_t* opt_signbits) {
  if (x == nullptr || grads == nullptr || !aligned(x, 4) || !aligned(grads, 4)) return S3GD_ERR_INVALID_ARG;
  if ((opt_idx == nullptr) != (opt_signbits == nullptr)) return S3GD_ERR_INVALID_ARG;
  if (opt_idx != nullptr && (!aligned(opt_idx, 4) || !aligned(opt_signbits, 4))) return S3GD_ERR_INVALID_ARG;
  return S3GD_OK;
}

}  // namespace

namespace {
s3gd_status plain_step(float* x, const float* grads, int M, uint64_t d, uint64_t K, float lr, uint32_t* opt_idx,
                       uint32_t* opt_signbits, int8_t* opt_vote, void* ws, size_t ws_bytes, void* stream,
                       uint32_t sample_rank, uint32_t prevote_rank) {
  Layout L;
  if (!make_layout(M, d, K, &L)) return S3GD_ERR_INVALID_ARG;
  override_sample_rank(&L, sample_rank, prevote_rank);
  s3gd_status s = check_step_args(x, grads, opt_idx, opt_signbits);
  if (s != S3GD_OK) return s;
  s = check_ws(L, ws, ws_bytes);
  if (s != S3GD_OK) return s;
  return step_impl(x, grads, nullptr, nullptr, 0.f, M, d, K, lr, opt_idx, opt_signbits, opt_vote, L, ws,
                   static_cast<cudaStream_t>(stream));
}
}  // namespace

s3gd_status s3gd_step(float* x, const float* grads, int M, uint64_t d, uint64_t K, float lr, uint32_t* opt_idx,
                      uint32_t* opt_signbits, int8_t* opt_vote, void* ws, size_t ws_bytes, void* stream) {
  return plain_step(x, grads, M, d, K, lr, opt_idx, opt_signbits, opt_vote, ws, ws_bytes, stream, 0u, 0u);
}

s3gd_status s3gd_debug_step(float* x, const float* grads, int M, uint64_t d, uint64_t K, float lr, uint32_t* opt_idx,
                            uint32_t* opt_signbits, int8_t* opt_vote, void* ws, size_t ws_bytes, void* stream,
                            uint32_t sample_rank, uint32_t prevote_rank) {
  return plain_step(x, grads, M, d, K, lr, opt_idx, opt_signbits, opt_vote, ws, ws_bytes, stream, sample_rank,
                    prevote_rank);
}

s3gd_status s3gd_step_ex(float* x, const float* grads, float* opt_err, float eta, float* opt_v, float mu, int M,
                         uint64_t d, uint64_t K, float lr, uint32_t* opt_idx, uint32_t* opt_signbits,
                         int8_t* opt_vote, void* ws, size_t ws_bytes, void* stream) {
  Layout L;
  if (!make_layout(M, d, K, &L)) return S3GD_ERR_INVALID_ARG;
  s3gd_status s = check_step_args(x, grads, opt_idx, opt_signbits);
  if (s != S3GD_OK) return s;
  if ((opt_err != nullptr && !aligned(opt_err, 4)) || (opt_v != nullptr && !aligned(opt_v, 4))) return S3GD_ERR_INVALID_ARG;
  s = check_ws(L, ws, ws_bytes);
  if (s != S3GD_OK) return s;
  cudaStream_t st = static_cast<cudaStream_t>(stream);
  const float* sel = grads;
  prof_mark(kPhaseStart, st);                  // the accumulation counts into the first phase
  const float* ef_raw = nullptr;
  if (opt_err != nullptr) {                    // g = g~ + eta * e, kept in the error memory
    // The filter pass can form g itself while it streams (one read of g~ and e, one write of g)
    // when there is a filter pass and both buffers allow the same 16-byte accesses.
    const bool fused = L.cap > 0 && K != 0 && K != d &&
                       ((reinterpret_cast<uintptr_t>(opt_err) ^ reinterpret_cast<uintptr_t>(grads)) & 15u) == 0;
    if (fused) ef_raw = grads;
    else S3GD_TRY(launch_ef_accumulate(opt_err, grads, eta, (uint64_t)M * d, st));
    sel = opt_err;
  }
  return step_impl(x, sel, opt_err, opt_v, mu, M, d, K, lr, opt_idx, opt_signbits, opt_vote, L, ws, st, false, ef_raw,
                   eta);
}

s3gd_status s3gd_apply_momentum(float* x, float* v, const int8_t* vote, uint64_t d, float mu, float lr,
                                void* stream) {
  if (x == nullptr || v == nullptr || vote == nullptr || d == 0 || d >= (1ull << 32) || !aligned(x, 4) || !aligned(v, 4))
    return S3GD_ERR_INVALID_ARG;
  return from_cuda(launch_apply_momentum(x, v, vote, d, mu, lr, static_cast<cudaStream_t>(stream)));
}

s3gd_status s3gd_randk_sign(const float* grads, int M, uint64_t d, uint64_t K, uint32_t seed, uint32_t step,
                            uint32_t* out_idx, uint32_t* out_signbits, void* ws, size_t ws_bytes, void* stream) {
  Layout L;
  if (!make_layout(M, d, K, &L) || grads == nullptr || !aligned(grads, 4)) return S3GD_ERR_INVALID_ARG;
  if (K > 0 && (out_idx == nullptr || out_signbits == nullptr || !aligned(out_idx, 4) || !aligned(out_signbits, 4)))
    return S3GD_ERR_INVALID_ARG;
  s3gd_status s = check_ws(L, ws, ws_bytes);
  if (s != S3GD_OK) return s;
  cudaStream_t st = static_cast<cudaStream_t>(stream);
  uint32_t* hdr = reinterpret_cast<uint32_t*>(static_cast<char*>(ws) + L.off_hdr);
  S3GD_TRY(cudaMemsetAsync(hdr, 0, kHdrWords * sizeof(uint32_t), st));
  return from_cuda(launch_randk(grads, M, d, K, seed, step, out_idx, out_signbits, nullptr, false, hdr, st));
}

s3gd_status s3gd_step_randk(float* x, const float* grads, int M, uint64_t d, uint64_t K, float lr, uint32_t seed,
                            uint32_t step, uint32_t* opt_idx, uint32_t* opt_signbits, int8_t* opt_vote, void* ws,
                            size_t ws_bytes, void* stream) {
  Layout L;
  if (!make_layout(M, d, K, &L)) return S3GD_ERR_INVALID_ARG;
  s3gd_status s = check_step_args(x, grads, opt_idx, opt_signbits);
  if (s != S3GD_OK) return s;
  s = check_ws(L, ws, ws_bytes);
  if (s != S3GD_OK) return s;
  cudaStream_t st = static_cast<cudaStream_t>(stream);
  char* base = static_cast<char*>(ws);
  uint32_t* hdr = reinterpret_cast<uint32_t*>(base + L.off_hdr);
  int32_t* counter = reinterpret_cast<int32_t*>(base + L.off_counter);
  prof_mark(kPhaseStart, st);
  S3GD_TRY(cudaMemsetAsync(hdr, 0, kHdrWords * sizeof(uint32_t), st));
  const bool packed = M <= kPackedMaxWorkers;     // a permutation: one vote per worker and coordinate
  if (packed) S3GD_TRY(cudaMemsetAsync(counter, 0x80, (size_t)((d + 3) / 4) * 4, st));
  else S3GD_TRY(cudaMemsetAsync(counter, 0, (size_t)d * sizeof(int32_t), st));
  for (int ph = kPhaseSampled; ph <= kPhaseThreshold; ++ph) prof_mark(ph, st);
  S3GD_TRY(launch_randk(grads, M, d, K, seed, step, opt_idx, opt_signbits, counter, packed, hdr, st));
  prof_mark(kPhaseEmitted, st);
  cudaError_t e = launch_counter_apply(counter, packed, x, d, lr, opt_vote, (uint64_t)M * K, st);
  prof_mark(kPhaseApplied, st);
  return from_cuda(e);
}

namespace {
s3gd_status profile_begin(int max_steps, bool filter_only, int every);
}

s3gd_status s3gd_profile_begin(int max_steps) { return profile_begin(max_steps, false, 1); }
s3gd_status s3gd_profile_begin_filter(int max_steps) { return profile_begin(max_steps, true, 1); }
s3gd_status s3gd_profile_begin_filter_every(int max_steps, int every) { return profile_begin(max_steps, true, every); }

namespace {
s3gd_status profile_begin(int max_steps, bool filter_only, int every) {
  if (max_steps <= 0 || max_steps > (1 << 20) || every < 1 || g_prof.on) return S3GD_ERR_INVALID_ARG;
  const size_t n = (size_t)max_steps * kPhaseMarks;
  g_prof.ev = new cudaEvent_t[n];
  for (size_t i = 0; i < n; ++i) {
    if (cudaEventCreate(&g_prof.ev[i]) != cudaSuccess) {
      for (size_t k = 0; k < i; ++k) cudaEventDestroy(g_prof.ev[k]);
      delete[] g_prof.ev;
      g_prof.ev = nullptr;
      return S3GD_ERR_CUDA;
    }
  }
  g_prof.max_steps = max_steps;
  g_prof.n_steps = 0;
  g_prof.every = every;
  g_prof.n_calls = 0;
  g_launches.store(0);
  g_prof.filter_only = filter_only;
  g_prof.on = true;
  return S3GD_OK;
}
}  // namespace

s3gd_status s3gd_profile_end(float* out_ms, int* n_steps, uint64_t* launches) {
  if (!g_prof.on) return S3GD_ERR_INVALID_ARG;
  s3gd_status ret = S3GD_OK;
  if (cudaDeviceSynchronize() != cudaSuccess) ret = S3GD_ERR_CUDA;
  for (int s = 0; s < g_prof.n_steps && ret == S3GD_OK && out_ms != nullptr; ++s) {
    for (int ph = 0; ph + 1 < kPhaseMarks; ++ph) {
      float ms = 0.f;
      if (g_prof.filter_only && ph != kPhaseSampled) {
        out_ms[(size_t)s * (kPhaseMarks - 1) + ph] = 0.f;
        continue;
      }
      if (cudaEventElapsedTime(&ms, g_prof.ev[(size_t)s * kPhaseMarks + ph],
                               g_prof.ev[(size_t)s * kPhaseMarks + ph + 1]) != cudaSuccess)
        ret = S3GD_ERR_CUDA;
      out_ms[(size_t)s * (kPhaseMarks - 1) + ph] = ms;
    }
  }
  if (n_steps) *n_steps = g_prof.n_steps;
  if (launches) *launches = g_launches.load();
  for (size_t i = 0; i < (size_t)g_prof.max_steps * kPhaseMarks; ++i) cudaEventDestroy(g_prof.ev[i]);
  delete[] g_prof.ev;
  g_prof = Profiler();
  return ret;
}

s3gd_status s3gd_device_status(const void* ws, void* stream, uint32_t* info) {
  if (ws == nullptr) return S3GD_ERR_WORKSPACE;
  cudaStream_t st = static_cast<cudaStream_t>(stream);
  uint32_t h[8] = {0, 0, 0, 0, 0, 0, 0, 0};
  if (cudaStreamSynchronize(st) != cudaSuccess) return S3GD_ERR_CUDA;
  if (cudaMemcpy(h, ws, sizeof(h), cudaMemcpyDeviceToHost) != cudaSuccess) return S3GD_ERR_CUDA;
  h[5] = h[6] = h[7] = 0;
  if (info) for (int i = 0; i < 8; ++i) info[i] = h[i];
  if (h[kHdrStatus] & kFlagInternal) return S3GD_ERR_INTERNAL;
  if (h[kHdrStatus] & kFlagIndexRange) return S3GD_ERR_INDEX_RANGE;
  return S3GD_OK;
}

s3gd_status s3gd_last_device_status(const void* ws, void* stream) { return s3gd_device_status(ws, stream, nullptr); }

}  // extern "C"

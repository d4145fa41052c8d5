// Host side of the C ABI declared in include/cocodc.h: argument validation,
// the context, and kernel launches.  Every arithmetic step runs in the kernels
// of outer.cuh / select.cuh / plan.cuh; nothing here computes on parameter data.

#include "../../include/cocodc.h"

#include <cuda_runtime.h>

#include <algorithm>
#include <cmath>
#include <cstdint>
#include <new>
#include <utility>
#include <vector>

#include "outer.cuh"
#include "outer_ring.cuh"
#include "plan.cuh"
#include "select.cuh"

using namespace cocodc;

struct cocodc_ctx {
  int device = 0;
  int sm_count = 0;
  int K = 0;
  int n_segments = 0;
  long long N = 0;
  int max_M = 0;
  int max_grid = 0;
  // device copies of the fragment table
  int* d_frag_seg_ptr = nullptr;
  long long* d_seg_off = nullptr;
  long long* d_seg_len = nullptr;
  long long* d_frag_size = nullptr;
  long long* d_frag_first_off = nullptr;   // native offset of every fragment's first segment
  // launch scratch
  SegPlan* d_plan = nullptr;
  PlanHeader* d_hdr = nullptr;
  double* d_partial = nullptr;
  int* d_status = nullptr;
  int* d_ticket = nullptr;                  // arrival counter of the in-kernel score epilogue (zero between launches)
  unsigned char* in_flight = nullptr;       // caller's in-flight mask (cocodc_bind_in_flight), or nullptr
  // a completion launched with COCODC_STAGE_DEFER whose scores no call has formed yet (host view of d_pending->n)
  PendingScores* d_pending = nullptr;
  bool pending = false;
  float* pend_norms = nullptr;
  float* pend_scores = nullptr;
  long long* pend_last = nullptr;
  int pend_grid = 0;                         // CTAs of the deferred completion's launch
  FragTable table{};                        // the fragment table as a kernel argument, when it is small enough
  bool inline_plan = false;                 // the streaming kernels expand the id list themselves (no k_plan launch)
  long long launches = 0;
  std::vector<std::pair<const void*, int>> occupancy;  // kernel -> resident CTAs per SM
  std::vector<std::pair<const void*, unsigned>> smem_opted_in;   // kernels opted in to large shared memory, with the size
  // host copy of the fragment table (host-buffer entry point walks it on the host)
  std::vector<int> h_frag_seg_ptr;
  std::vector<long long> h_seg_off, h_seg_len;
  // host-buffer entry point: copy streams, pipeline events, K-sized device staging
  static constexpr int kSlots = 3;
  cudaStream_t s_h2d = nullptr, s_d2h = nullptr;
  cudaEvent_t ev_h2d[kSlots] = {}, ev_comp[kSlots] = {}, ev_d2h[kSlots] = {};
  double* d_frag_sumsq = nullptr;   // [K]
  int* d_k_ids = nullptr;           // [K]
  long long* d_k_last = nullptr;    // [K]
  float* d_k_norms = nullptr;       // [K]
  float* d_k_scores = nullptr;      // [K]
};

namespace {

struct DeviceGuard {
  int prev = -1;
  bool switched = false;
  explicit DeviceGuard(int dev) {
    if (cudaGetDevice(&prev) == cudaSuccess && prev != dev) switched = (cudaSetDevice(dev) == cudaSuccess);
  }
  ~DeviceGuard() { if (switched) cudaSetDevice(prev); }
};

inline bool aligned16(const void* p) { return (reinterpret_cast<uintptr_t>(p) & 15u) == 0; }

struct Range { uintptr_t lo, hi; };
inline Range range_of(const void* p, long long elems) {
  uintptr_t b = reinterpret_cast<uintptr_t>(p);
  return Range{b, b + (uintptr_t)elems * sizeof(float)};
}
inline bool overlap(Range a, Range b) { return a.lo < b.hi && b.lo < a.hi; }

int grid_for(cocodc_ctx* c, const void* kernel) {
  for (auto& kv : c->occupancy) if (kv.first == kernel) return kv.second * c->sm_count;
  int per_sm = 0;
  if (cudaOccupancyMaxActiveBlocksPerMultiprocessor(&per_sm, kernel, kThreads, 0) != cudaSuccess || per_sm < 1)
    per_sm = 1;
  per_sm = std::min(per_sm, 8);
  c->occupancy.emplace_back(kernel, per_sm);
  return per_sm * c->sm_count;
}

cocodc_status launch_plan(cocodc_ctx* c, const int32_t* ids, const int32_t* n_ids,
                          const int64_t* snap_offset, long long snap_row_len, int lanes_per_tile, cudaStream_t st) {
  k_plan<<<1, kPlanThreads, 0, st>>>(ids, n_ids, c->K, c->d_frag_seg_ptr, c->d_seg_off, c->d_seg_len,
                                     reinterpret_cast<const long long*>(snap_offset), snap_row_len, lanes_per_tile,
                                     c->n_segments, c->d_plan, c->d_hdr, c->d_status,
                                     (int)COCODC_ERR_INVALID_ARG);
  c->launches++;
  return cudaGetLastError() == cudaSuccess ? COCODC_OK : COCODC_ERR_CUDA;
}

// Scores that a deferred completion left unformed are formed now (one small launch), before a call that reads or
// writes the schedule arrays, or the scratch the CTAs' sums sit in, without being the selection that consumes them.
cocodc_status flush_pending(cocodc_ctx* c, cudaStream_t st) {
  if (!c->pending) return COCODC_OK;
  k_flush_pending<<<1, 256, 0, st>>>(c->d_pending, c->d_partial, c->K, c->pend_norms, c->pend_scores, c->pend_last,
                                     c->in_flight, c->d_status, (int)COCODC_ERR_NONFINITE);
  c->launches++;
  c->pending = false;
  return cudaGetLastError() == cudaSuccess ? COCODC_OK : COCODC_ERR_CUDA;
}

// One way to run the streaming step: which kernel, with how many threads and how much dynamic
// shared memory, on how many CTAs, over tiles of how many lanes.  Every variant has eight accumulating
// warps, so the score epilogue does not depend on the choice; the plan is built for the variant's tile.
struct Variant {
  void (*kernel)(const OuterArgs, const FragTable);
  int threads;
  unsigned smem;
  bool one_cta_per_sm;   // staged kernel: persistent, one CTA per SM; otherwise sized by occupancy
  int ring_slots = 0;    // k_outer_ring only
  int lanes_per_tile = kThreads;   // 16-byte lanes of one tile: what the plan of this launch is built with
};

// Worker counts without a compile-time instance: the slot-ring kernel, or, when even the recorded values of
// one tile do not fit its ring, the element loop.
template <int MODE, bool SAME>
Variant runtime_variant(int M) {
  const int chunks = ring_chunks_for(MODE, M);
  if (chunks == 0) return Variant{k_outer_generic<MODE, SAME>, kThreads, 0u, false};
  return Variant{k_outer_ring<MODE, SAME>, kRingThreads, (unsigned)chunks * kChunkBytes, true, chunks};
}

// The staged kernel with the tile width its number of streams calls for (tile_width()).
template <int M, int MODE, bool SAME>
Variant staged_variant() {
  constexpr int U = tile_width(StageLayout<M, MODE, SAME, 1>::kLoaded);
  using L = StageLayout<M, MODE, SAME, U>;
  return Variant{k_outer_tma<M, MODE, SAME, U>, tma_threads(M), L::kSmemBytes, true, 0, kThreads * U};
}

// More than 48 KB of dynamic shared memory needs a one-time opt-in per kernel and device (the
// caller has made the context's device current).
void opt_in_shared_memory(cocodc_ctx* c, const void* kernel, unsigned bytes) {
  if (bytes <= 24u * 1024u) return;   // static shared memory (up to 18 KB: plan, selection state) counts towards the 48 KB a kernel gets without opting in
  for (auto& k : c->smem_opted_in) {
    if (k.first != kernel) continue;
    if (k.second >= bytes) return;
    cudaFuncSetAttribute(kernel, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)bytes);
    k.second = bytes;
    return;
  }
  cudaFuncSetAttribute(kernel, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)bytes);
  c->smem_opted_in.emplace_back(kernel, bytes);
}

// Worker counts 1..8 have compile-time instances of the staged kernel; larger M take the chunk-ring kernel
// (or the element loop when one tile of recorded values does not fit its ring): runtime_variant().
template <int MODE, bool SAME>
Variant pick_variant(int M) {
  switch (M) {
    case 1: return staged_variant<1, MODE, SAME>();
    case 2: return staged_variant<2, MODE, SAME>();
    case 3: return staged_variant<3, MODE, SAME>();
    case 4: return staged_variant<4, MODE, SAME>();
    case 5: return staged_variant<5, MODE, SAME>();
    case 6: return staged_variant<6, MODE, SAME>();
    case 7: return staged_variant<7, MODE, SAME>();
    case 8: return staged_variant<8, MODE, SAME>();
    default: return runtime_variant<MODE, SAME>(M);
  }
}

template <int M>
Variant inplace_variant() {
  return Variant{k_outer_inplace<M>, kInplaceThreads, InplaceLayout<M>::kSmemBytes, true};
}

// The fused step with zero delay (every stream read is also written).  Measured per worker count on 100 M-parameter
// launches, in-place pipeline against the staged kernel with register stores, GB/s for M = 1..8:
// 5940 / 6330 / 6390 / 6480 / 6460 / 6330 / 6170 / 6230 against 6120 / 6450 / 6310 / 6260 / 6150 / 6510 / 6430 / 6360,
// so M = 3, 4, 5 take the in-place pipeline and the other staged worker counts the staged kernel.
Variant pick_zero_delay_variant(int M) {
  switch (M) {
    case 3: return inplace_variant<3>();
    case 4: return inplace_variant<4>();
    case 5: return inplace_variant<5>();
    default: return pick_variant<MODE_FUSED, true>(M);
  }
}

// received-sum mode: n_recv more streams per stage, ring sized at run time; staged up to four local workers
template <int M>
Variant received_variant(int n_recv) {
  const int loaded = StageLayout<M, MODE_FUSED_RECV, false>::kLoaded + n_recv;
  return Variant{k_outer_tma<M, MODE_FUSED_RECV, false>, tma_threads(M),
                 (unsigned)(stages_for(loaded) * loaded) * kTileBytes, true};
}

Variant pick_variant(int M, int mode, bool same, int n_recv = 0) {
  if (mode == MODE_FUSED_RECV) {
    switch (M) {
      case 1: return received_variant<1>(n_recv);
      case 2: return received_variant<2>(n_recv);
      case 3: return received_variant<3>(n_recv);
      case 4: return received_variant<4>(n_recv);
      default: return runtime_variant<MODE_FUSED_RECV, false>(M);
    }
  }
  if (mode == MODE_OUTER_ONLY) return pick_variant<MODE_OUTER_ONLY, false>(M);
  if (mode == MODE_PSEUDO_SUM) return pick_variant<MODE_PSEUDO_SUM, false>(M);
  if (mode == MODE_MERGE_ONLY) return same ? pick_variant<MODE_MERGE_ONLY, true>(M) : pick_variant<MODE_MERGE_ONLY, false>(M);
  return same ? pick_zero_delay_variant(M) : pick_variant<MODE_FUSED, false>(M);
}

int variant_grid(cocodc_ctx* c, const Variant& v) {
  return v.one_cta_per_sm ? c->sm_count : grid_for(c, reinterpret_cast<const void*>(v.kernel));
}

// What a launch is to work on, as the kernels take it; with a fragment table too large to be a kernel argument
// the plan is first written to global memory by k_plan.
cocodc_status prepare_plan(cocodc_ctx* c, const int32_t* ids, const int32_t* n_ids, const int64_t* snap_offset,
                           long long snap_row_len, int lanes_per_tile, cudaStream_t st, PlanRequest* rq,
                           const SegPlan** gplan, const PlanHeader** ghdr) {
  rq->ids = ids;
  rq->n_ids = n_ids;
  rq->snap_offset = reinterpret_cast<const long long*>(snap_offset);
  rq->snap_row_len = snap_row_len;
  rq->lanes_per_tile = lanes_per_tile;
  rq->err_invalid = (int)COCODC_ERR_INVALID_ARG;
  if (c->inline_plan) {
    *gplan = nullptr;
    *ghdr = nullptr;
    return COCODC_OK;
  }
  *gplan = c->d_plan;
  *ghdr = c->d_hdr;
  return launch_plan(c, ids, n_ids, snap_offset, snap_row_len, lanes_per_tile, st);
}

// (plan +) streaming kernel for a device-resident id list
cocodc_status launch_outer(cocodc_ctx* c, const OuterArgs& A, int mode, bool same, const int32_t* ids,
                           const int32_t* n_ids, const int64_t* snap_offset, cudaStream_t st) {
  const Variant v = pick_variant(A.M, mode, same, A.n_recv);
  const int grid = variant_grid(c, v);
  opt_in_shared_memory(c, reinterpret_cast<const void*>(v.kernel), v.smem);
  OuterArgs args = A;
  cocodc_status s = prepare_plan(c, ids, n_ids, snap_offset, A.snap_stride, v.lanes_per_tile, st, &args.rq,
                                 &args.plan, &args.hdr);
  if (s != COCODC_OK) return s;
  args.ring_slots = v.ring_slots;
  v.kernel<<<grid, v.threads, v.smem, st>>>(args, c->table);
  c->launches++;
  if (A.fin.defer) c->pend_grid = grid;
  return cudaGetLastError() == cudaSuccess ? COCODC_OK : COCODC_ERR_CUDA;
}

// Shared checks of the three entry points that stream worker buffers.
cocodc_status check_hyper(const cocodc_ctx* c, const cocodc_hyper* h) {
  if (!c || !h) return COCODC_ERR_INVALID_ARG;
  if (h->M < 1 || h->M > c->max_M) return COCODC_ERR_INVALID_ARG;
  if (h->H < 1 || h->tau < 0) return COCODC_ERR_INVALID_ARG;
  if (h->comp_mode != COCODC_COMP_NONE && h->comp_mode != COCODC_COMP_TAYLOR) return COCODC_ERR_INVALID_ARG;
  if (h->sign_mode < COCODC_SIGN_FORWARD || h->sign_mode > COCODC_SIGN_DESCENT) return COCODC_ERR_INVALID_ARG;
  if (!std::isfinite(h->outer_lr) || !std::isfinite(h->momentum) || !std::isfinite(h->lambda) ||
      !std::isfinite(h->alpha))
    return COCODC_ERR_INVALID_ARG;
  return COCODC_OK;
}

// Eq. 6-7 folded into two scalars (computed in double, rounded once).
void fold_coefficients(const cocodc_hyper* h, bool zero_delay, OuterArgs* A) {
  double c1 = 0.0, c2 = 0.0;
  if (h->comp_mode == COCODC_COMP_TAYLOR && h->tau > 0 && !zero_delay) {
    const double c = (double)h->lambda / ((double)h->tau * (double)h->H);
    switch (h->sign_mode) {
      case COCODC_SIGN_FORWARD: c1 = 1.0; c2 = c; break;
      case COCODC_SIGN_PRINTED: c1 = -1.0; c2 = c; break;
      default: c1 = 1.0; c2 = -c; break;
    }
  }
  A->c1 = (float)c1;
  A->c2 = (float)c2;
  A->alpha = h->alpha;
  A->one_minus_alpha = (float)(1.0 - (double)h->alpha);
  A->eta = h->outer_lr;
  A->mu = h->momentum;
  A->M = h->M;
  A->Mf = (float)h->M;
  A->inv_M = 1.0f / (float)h->M;
  A->M_pow2 = ((h->M & (h->M - 1)) == 0) ? 1 : 0;
}

// elements of fragment p (host copy of the table)
long long fragment_elems(const cocodc_ctx* c, int p) {
  long long n = 0;
  for (int s = c->h_frag_seg_ptr[p]; s < c->h_frag_seg_ptr[p + 1]; ++s) n += c->h_seg_len[s];
  return n;
}

void set_status_sink(const cocodc_ctx* c, OuterArgs* A) {
  A->status = c->d_status;
  A->err_timeout = (int)COCODC_ERR_TIMEOUT;
}

}  // namespace

extern "C" {

const char* cocodc_status_string(cocodc_status s) {
  switch (s) {
    case COCODC_OK: return "ok";
    case COCODC_ERR_INVALID_ARG: return "invalid argument";
    case COCODC_ERR_ALIGNMENT: return "buffer not 16-byte aligned or stride not a multiple of 4 elements";
    case COCODC_ERR_ALIAS: return "buffers overlap";
    case COCODC_ERR_NONFINITE: return "non-finite value";
    case COCODC_ERR_TIMEOUT: return "bounded wait ran out";
    case COCODC_ERR_CUDA: return "CUDA error";
    case COCODC_ERR_NOMEM: return "out of memory";
  }
  return "unknown status";
}

cocodc_status cocodc_sync_budget(int32_t K, int64_t H, double gamma, double Tc, double Ts,
                                 int64_t* N_out, int64_t* h_out) {
  if (!N_out || !h_out || K < 1 || H < 1) return COCODC_ERR_INVALID_ARG;
  if (!(gamma > 0.0 && gamma <= 1.0) || !(Tc > 0.0) || !(Ts > 0.0)) return COCODC_ERR_INVALID_ARG;
  const double cap = std::floor(gamma * (double)H * Tc / Ts);
  if (!std::isfinite(cap)) return COCODC_ERR_INVALID_ARG;
  int64_t N = (cap >= 9.0e18) ? INT64_MAX : (int64_t)cap;   // Eq. 8
  if (N < K) N = K;
  int64_t h = H / N;                                         // Eq. 9
  if (h < 1) h = 1;
  *N_out = N;
  *h_out = h;
  return COCODC_OK;
}

cocodc_status cocodc_create(cocodc_ctx** ctx_out, const cocodc_partition* part, int32_t max_M, int32_t device) {
  if (!ctx_out) return COCODC_ERR_INVALID_ARG;
  *ctx_out = nullptr;
  if (!part || !part->frag_seg_ptr || !part->seg_offset || !part->seg_len) return COCODC_ERR_INVALID_ARG;
  if (part->K < 1 || part->K > kMaxK || part->n_segments < part->K || part->N < 1) return COCODC_ERR_INVALID_ARG;
  if (max_M < 1 || max_M > 64) return COCODC_ERR_INVALID_ARG;
  const int K = part->K, S = part->n_segments;
  if (part->frag_seg_ptr[0] != 0 || part->frag_seg_ptr[K] != S) return COCODC_ERR_INVALID_ARG;
  std::vector<long long> frag_size(K, 0);
  std::vector<std::pair<long long, long long>> segs;
  segs.reserve(S);
  for (int p = 0; p < K; ++p) {
    if (part->frag_seg_ptr[p + 1] <= part->frag_seg_ptr[p]) return COCODC_ERR_INVALID_ARG;  // empty fragment
    if (part->frag_seg_ptr[p + 1] > S) return COCODC_ERR_INVALID_ARG;   // would read past the segment arrays
    for (int s = part->frag_seg_ptr[p]; s < part->frag_seg_ptr[p + 1]; ++s) {
      const long long o = part->seg_offset[s], l = part->seg_len[s];
      if (o < 0 || l < 1 || o > part->N - l) return COCODC_ERR_INVALID_ARG;
      frag_size[p] += l;
      segs.emplace_back(o, l);
    }
  }
  std::sort(segs.begin(), segs.end());
  for (size_t i = 1; i < segs.size(); ++i)
    if (segs[i].first < segs[i - 1].first + segs[i - 1].second) return COCODC_ERR_INVALID_ARG;  // overlap

  int n_dev = 0;
  if (cudaGetDeviceCount(&n_dev) != cudaSuccess) return COCODC_ERR_CUDA;
  if (device < 0 || device >= n_dev) return COCODC_ERR_INVALID_ARG;
  DeviceGuard guard(device);
  cocodc_ctx* c = new (std::nothrow) cocodc_ctx();
  if (!c) return COCODC_ERR_NOMEM;
  c->device = device;
  c->K = K;
  c->n_segments = S;
  c->N = part->N;
  c->max_M = max_M;
  cudaDeviceProp prop;
  if (cudaGetDeviceProperties(&prop, device) != cudaSuccess) { delete c; return COCODC_ERR_CUDA; }
  c->sm_count = prop.multiProcessorCount;
  c->max_grid = c->sm_count * 8;

  std::vector<long long> off(S), len(S);
  for (int s = 0; s < S; ++s) { off[s] = part->seg_offset[s]; len[s] = part->seg_len[s]; }
  const size_t partial_elems = (size_t)K * c->max_grid * (kThreads / 32);
  bool ok = true;
  ok = ok && cudaMalloc(&c->d_frag_seg_ptr, sizeof(int) * (K + 1)) == cudaSuccess;
  ok = ok && cudaMalloc(&c->d_seg_off, sizeof(long long) * S) == cudaSuccess;
  ok = ok && cudaMalloc(&c->d_seg_len, sizeof(long long) * S) == cudaSuccess;
  ok = ok && cudaMalloc(&c->d_frag_size, sizeof(long long) * K) == cudaSuccess;
  ok = ok && cudaMalloc(&c->d_frag_first_off, sizeof(long long) * K) == cudaSuccess;
  ok = ok && cudaMalloc(&c->d_plan, sizeof(SegPlan) * S) == cudaSuccess;
  ok = ok && cudaMalloc(&c->d_hdr, sizeof(PlanHeader)) == cudaSuccess;
  ok = ok && cudaMalloc(&c->d_partial, sizeof(double) * partial_elems) == cudaSuccess;
  ok = ok && cudaMalloc(&c->d_status, sizeof(int)) == cudaSuccess;
  ok = ok && cudaMalloc(&c->d_ticket, sizeof(int)) == cudaSuccess;
  ok = ok && cudaMalloc(&c->d_pending, sizeof(PendingScores)) == cudaSuccess;
  ok = ok && cudaMalloc(&c->d_frag_sumsq, sizeof(double) * K) == cudaSuccess;
  ok = ok && cudaMalloc(&c->d_k_ids, sizeof(int) * K) == cudaSuccess;
  ok = ok && cudaMalloc(&c->d_k_last, sizeof(long long) * K) == cudaSuccess;
  ok = ok && cudaMalloc(&c->d_k_norms, sizeof(float) * K) == cudaSuccess;
  ok = ok && cudaMalloc(&c->d_k_scores, sizeof(float) * K) == cudaSuccess;
  if (!ok) { cudaGetLastError(); cocodc_destroy(c); return COCODC_ERR_NOMEM; }
  ok = ok && cudaStreamCreateWithFlags(&c->s_h2d, cudaStreamNonBlocking) == cudaSuccess;
  ok = ok && cudaStreamCreateWithFlags(&c->s_d2h, cudaStreamNonBlocking) == cudaSuccess;
  for (int i = 0; i < cocodc_ctx::kSlots && ok; ++i) {
    ok = ok && cudaEventCreateWithFlags(&c->ev_h2d[i], cudaEventDisableTiming) == cudaSuccess;
    ok = ok && cudaEventCreateWithFlags(&c->ev_comp[i], cudaEventDisableTiming) == cudaSuccess;
    ok = ok && cudaEventCreateWithFlags(&c->ev_d2h[i], cudaEventDisableTiming) == cudaSuccess;
  }
  if (!ok) { cudaGetLastError(); cocodc_destroy(c); return COCODC_ERR_CUDA; }
  c->h_frag_seg_ptr.assign(part->frag_seg_ptr, part->frag_seg_ptr + K + 1);
  c->h_seg_off = off;
  c->h_seg_len = len;
  ok = ok && cudaMemcpy(c->d_frag_seg_ptr, part->frag_seg_ptr, sizeof(int) * (K + 1), cudaMemcpyHostToDevice) == cudaSuccess;
  ok = ok && cudaMemcpy(c->d_seg_off, off.data(), sizeof(long long) * S, cudaMemcpyHostToDevice) == cudaSuccess;
  ok = ok && cudaMemcpy(c->d_seg_len, len.data(), sizeof(long long) * S, cudaMemcpyHostToDevice) == cudaSuccess;
  ok = ok && cudaMemcpy(c->d_frag_size, frag_size.data(), sizeof(long long) * K, cudaMemcpyHostToDevice) == cudaSuccess;
  {
    std::vector<long long> first_off(K);
    for (int p = 0; p < K; ++p) first_off[p] = part->seg_offset[part->frag_seg_ptr[p]];
    ok = ok && cudaMemcpy(c->d_frag_first_off, first_off.data(), sizeof(long long) * K, cudaMemcpyHostToDevice) == cudaSuccess;
  }
  ok = ok && cudaMemset(c->d_status, 0, sizeof(int)) == cudaSuccess;
  ok = ok && cudaMemset(c->d_ticket, 0, sizeof(int)) == cudaSuccess;
  ok = ok && cudaMemset(c->d_pending, 0, sizeof(PendingScores)) == cudaSuccess;
  ok = ok && cudaMemset(c->d_hdr, 0, sizeof(PlanHeader)) == cudaSuccess;
  c->inline_plan = (S <= kInlineSegs);
  if (c->inline_plan) {
    c->table.K = K;
    c->table.n_seg = S;
    for (int p = 0; p <= K; ++p) c->table.seg_ptr[p] = part->frag_seg_ptr[p];
    for (int sg = 0; sg < S; ++sg) { c->table.off[sg] = off[sg]; c->table.len[sg] = len[sg]; }
  }
  if (!ok) { cudaGetLastError(); cocodc_destroy(c); return COCODC_ERR_CUDA; }
  *ctx_out = c;
  return COCODC_OK;
}

cocodc_status cocodc_destroy(cocodc_ctx* c) {
  if (!c) return COCODC_OK;
  DeviceGuard guard(c->device);
  cudaFree(c->d_frag_seg_ptr);
  cudaFree(c->d_seg_off);
  cudaFree(c->d_seg_len);
  cudaFree(c->d_frag_size);
  cudaFree(c->d_frag_first_off);
  cudaFree(c->d_plan);
  cudaFree(c->d_hdr);
  cudaFree(c->d_partial);
  cudaFree(c->d_status);
  cudaFree(c->d_ticket);
  cudaFree(c->d_pending);
  cudaFree(c->d_frag_sumsq);
  cudaFree(c->d_k_ids);
  cudaFree(c->d_k_last);
  cudaFree(c->d_k_norms);
  cudaFree(c->d_k_scores);
  for (int i = 0; i < cocodc_ctx::kSlots; ++i) {
    if (c->ev_h2d[i]) cudaEventDestroy(c->ev_h2d[i]);
    if (c->ev_comp[i]) cudaEventDestroy(c->ev_comp[i]);
    if (c->ev_d2h[i]) cudaEventDestroy(c->ev_d2h[i]);
  }
  if (c->s_h2d) cudaStreamDestroy(c->s_h2d);
  if (c->s_d2h) cudaStreamDestroy(c->s_d2h);
  delete c;
  return COCODC_OK;
}

int64_t cocodc_launch_count(const cocodc_ctx* c) { return c ? c->launches : 0; }

cocodc_status cocodc_poll_status(cocodc_ctx* c, void* stream) {
  if (!c) return COCODC_ERR_INVALID_ARG;
  DeviceGuard guard(c->device);
  cudaStream_t st = static_cast<cudaStream_t>(stream);
  int word = 0;
  if (cudaMemcpyAsync(&word, c->d_status, sizeof(int), cudaMemcpyDeviceToHost, st) != cudaSuccess) return COCODC_ERR_CUDA;
  if (cudaMemsetAsync(c->d_status, 0, sizeof(int), st) != cudaSuccess) return COCODC_ERR_CUDA;
  if (cudaStreamSynchronize(st) != cudaSuccess) return COCODC_ERR_CUDA;
  // a launch that gave up on a bounded wait leaves the arrival counter of its score epilogue behind
  if (word != 0 && cudaMemsetAsync(c->d_ticket, 0, sizeof(int), st) != cudaSuccess) return COCODC_ERR_CUDA;
  // ... and a deferred completion that failed leaves nothing worth forming
  if (word != 0 && c->pending) {
    if (cudaMemsetAsync(c->d_pending, 0, sizeof(int), st) != cudaSuccess) return COCODC_ERR_CUDA;
    c->pending = false;
  }
  return static_cast<cocodc_status>(word);
}

cocodc_status cocodc_fragment_scores(cocodc_ctx* c, const float* delta_g, const int64_t* interval,
                                     float* norms, float* scores, double* sumsq_out, void* stream) {
  if (!c || !delta_g) return COCODC_ERR_INVALID_ARG;
  if ((norms == nullptr) != (scores == nullptr) || (!norms && !sumsq_out)) return COCODC_ERR_INVALID_ARG;
  if (!aligned16(delta_g)) return COCODC_ERR_ALIGNMENT;
  DeviceGuard guard(c->device);
  cudaStream_t st = static_cast<cudaStream_t>(stream);
  if (flush_pending(c, st) != COCODC_OK) return COCODC_ERR_CUDA;
  constexpr int U = 4;
  auto kernel = k_sumsq<U>;
  const int grid = grid_for(c, reinterpret_cast<const void*>(kernel));
  PlanRequest rq{};
  const SegPlan* gplan = nullptr;
  const PlanHeader* ghdr = nullptr;
  cocodc_status s = prepare_plan(c, nullptr, nullptr, nullptr, 0, kThreads * U, st, &rq, &gplan, &ghdr);
  if (s != COCODC_OK) return s;
  Finalize fin{};
  fin.ticket = c->d_ticket;
  fin.mode = 1;
  fin.write_scores = norms ? 1 : 0;
  fin.interval = reinterpret_cast<const long long*>(interval);
  fin.norms = norms;
  fin.scores = scores;
  fin.sumsq_out = sumsq_out;
  fin.err_nonfinite = (int)COCODC_ERR_NONFINITE;
  kernel<<<grid, kThreads, 0, st>>>(delta_g, gplan, ghdr, rq, fin, c->d_partial, c->d_status, c->table);
  c->launches++;
  return cudaGetLastError() == cudaSuccess ? COCODC_OK : COCODC_ERR_CUDA;
}

cocodc_status cocodc_scores_from_sumsq(cocodc_ctx* c, const double* sumsq, const int32_t* ids, const int32_t* n_ids,
                                       const int64_t* interval, int64_t t_p, int64_t t_l, int64_t* last_sync,
                                       float* norms, float* scores, void* stream) {
  if (!c || !sumsq || !norms || !scores) return COCODC_ERR_INVALID_ARG;
  const bool completion = (ids != nullptr);
  if (completion && (!n_ids || !last_sync || interval || t_l < t_p)) return COCODC_ERR_INVALID_ARG;
  if (!completion && n_ids) return COCODC_ERR_INVALID_ARG;
  DeviceGuard guard(c->device);
  if (flush_pending(c, static_cast<cudaStream_t>(stream)) != COCODC_OK) return COCODC_ERR_CUDA;
  k_scores_from_sumsq<<<1, kFinalizeThreads, 0, static_cast<cudaStream_t>(stream)>>>(
      sumsq, 0, ids, n_ids, 0, c->K, completion ? 0 : 1, reinterpret_cast<const long long*>(interval), t_p, t_l,
      reinterpret_cast<long long*>(last_sync), norms, scores, completion ? c->in_flight : nullptr, c->d_status,
      (int)COCODC_ERR_NONFINITE, (int)COCODC_ERR_INVALID_ARG);
  c->launches++;
  return cudaGetLastError() == cudaSuccess ? COCODC_OK : COCODC_ERR_CUDA;
}

cocodc_status cocodc_bind_in_flight(cocodc_ctx* c, uint8_t* in_flight) {
  if (!c) return COCODC_ERR_INVALID_ARG;
  c->in_flight = in_flight;
  return COCODC_OK;
}

cocodc_status cocodc_flush_scores(cocodc_ctx* c, void* stream) {
  if (!c) return COCODC_ERR_INVALID_ARG;
  DeviceGuard guard(c->device);
  return flush_pending(c, static_cast<cudaStream_t>(stream));
}

}  // extern "C"

namespace {
cocodc_status select_impl(cocodc_ctx* c, const float* scores, const int64_t* last_sync,
                          const uint8_t* ineligible, int64_t t_now, const int64_t* t_now_dev, int64_t H,
                          int32_t budget_kind, int64_t budget,
                          uint8_t* mask, int32_t* ids, int32_t* n_sel,
                          int64_t* pool_offset, void* stream) {
  if (!c || !scores || !last_sync || !mask || !ids || !n_sel) return COCODC_ERR_INVALID_ARG;
  if (H < 1 || budget < 0) return COCODC_ERR_INVALID_ARG;
  if (budget_kind != COCODC_BUDGET_COUNT && budget_kind != COCODC_BUDGET_PARAMS &&
      budget_kind != COCODC_BUDGET_PARAMS_EXACT)
    return COCODC_ERR_INVALID_ARG;
  DeviceGuard guard(c->device);
  cudaStream_t st = static_cast<cudaStream_t>(stream);
  if (flush_pending(c, st) != COCODC_OK) return COCODC_ERR_CUDA;
  k_select<<<1, kSelectThreads, 0, st>>>(c->K, scores, reinterpret_cast<const long long*>(last_sync), ineligible,
                                         c->d_frag_size, c->d_frag_first_off, t_now, reinterpret_cast<const long long*>(t_now_dev), H, budget_kind, budget, mask, ids, n_sel,
                                         reinterpret_cast<long long*>(pool_offset), c->in_flight, c->d_status, (int)COCODC_ERR_NONFINITE,
                                         (int)COCODC_ERR_INVALID_ARG);
  c->launches++;
  return cudaGetLastError() == cudaSuccess ? COCODC_OK : COCODC_ERR_CUDA;
}

// cocodc_outer_step and cocodc_outer_step_received: the latter passes the all-reduced sum of every
// worker's pseudo-gradients (delta_sum) and the total worker count it is to be divided by.
cocodc_status outer_step_impl(cocodc_ctx* c, const cocodc_hyper* h,
                              float* w_now, const float* w_snap,
                              int64_t now_stride, int64_t snap_stride, const int64_t* snap_offset,
                              float* theta_g, float* momentum, float* delta_g_out,
                              const int32_t* ids, const int32_t* n_ids,
                              int64_t t_p, int64_t t_l, int64_t* last_sync,
                              float* norms, float* scores, double* sumsq_out, uint32_t stages, void* stream,
                              const float* const* delta_sums, int32_t n_sums, int32_t M_total,
                              const int64_t* t_p_dev = nullptr, const int64_t* t_l_dev = nullptr) {
  cocodc_status s = check_hyper(c, h);
  if (s != COCODC_OK) return s;
  const bool received = n_sums > 0;
  if (received && (M_total < h->M || stages != COCODC_STAGE_ALL || n_sums > kMaxRecv)) return COCODC_ERR_INVALID_ARG;
  for (int r = 0; r < n_sums; ++r) {
    if (!delta_sums[r]) return COCODC_ERR_INVALID_ARG;
    if (!aligned16(delta_sums[r])) return COCODC_ERR_ALIGNMENT;
  }
  if (!(stages & COCODC_STAGE_OUTER) || (stages & ~(COCODC_STAGE_ALL | COCODC_STAGE_SUMSQ | COCODC_STAGE_DEFER)))
    return COCODC_ERR_INVALID_ARG;
  const bool do_merge = (stages & COCODC_STAGE_MERGE) != 0;
  const bool do_score = (stages & COCODC_STAGE_SCORE) != 0;
  const bool defer = (stages & COCODC_STAGE_DEFER) != 0;
  // deferring is a way of running the SCORE stage; the sums of squares themselves are then not handed out
  if (defer && (!do_score || (stages & COCODC_STAGE_SUMSQ) || sumsq_out)) return COCODC_ERR_INVALID_ARG;
  const bool do_sums = do_score || (stages & COCODC_STAGE_SUMSQ) != 0;
  if ((stages & COCODC_STAGE_SUMSQ) && !sumsq_out) return COCODC_ERR_INVALID_ARG;
  if (!w_snap || !theta_g || !momentum || !ids || !n_ids) return COCODC_ERR_INVALID_ARG;
  if (do_merge && !w_now) return COCODC_ERR_INVALID_ARG;
  if (do_score && (!last_sync || !norms || !scores)) return COCODC_ERR_INVALID_ARG;
  if (t_l < t_p) return COCODC_ERR_INVALID_ARG;
  if ((t_p_dev == nullptr) != (t_l_dev == nullptr)) return COCODC_ERR_INVALID_ARG;
  const long long N = c->N;
  if (snap_stride < (snap_offset ? 1 : N) || (do_merge && now_stride < N)) return COCODC_ERR_INVALID_ARG;
  const bool same = do_merge && (w_snap == w_now) && (snap_stride == now_stride) && (snap_offset == nullptr);
  if (received && same) return COCODC_ERR_INVALID_ARG;   // the received sum belongs to recorded snapshots
  if (h->tau == 0 && h->comp_mode == COCODC_COMP_TAYLOR && do_merge && !same) return COCODC_ERR_INVALID_ARG;
  if (!aligned16(w_snap) || !aligned16(theta_g) || !aligned16(momentum) || (snap_stride & 3)) return COCODC_ERR_ALIGNMENT;
  if (do_merge && (!aligned16(w_now) || (now_stride & 3))) return COCODC_ERR_ALIGNMENT;
  if (delta_g_out && !aligned16(delta_g_out)) return COCODC_ERR_ALIGNMENT;
  // aliasing: every output range must be disjoint from every other buffer
  {
    const int M = h->M;
    Range r[4];
    int nr = 0;
    r[nr++] = range_of(theta_g, N);
    r[nr++] = range_of(momentum, N);
    if (delta_g_out) r[nr++] = range_of(delta_g_out, N);
    if (do_merge) r[nr++] = range_of(w_now, (long long)(M - 1) * now_stride + N);
    for (int i = 0; i < nr; ++i)
      for (int j = i + 1; j < nr; ++j)
        if (overlap(r[i], r[j])) return COCODC_ERR_ALIAS;
    if (!same) {
      const Range rs = range_of(w_snap, (long long)(M - 1) * snap_stride + (snap_offset ? snap_stride : N));
      for (int i = 0; i < nr; ++i) if (overlap(rs, r[i])) return COCODC_ERR_ALIAS;
    }
    // delta_g_out may be the same buffer as one of the sums (updated in place), nothing else may
    for (int q = 0; q < n_sums; ++q) {
      const Range rd = range_of(delta_sums[q], N);
      for (int i = 0; i < nr; ++i)
        if (overlap(rd, r[i]) && !(delta_g_out == delta_sums[q] && r[i].lo == rd.lo)) return COCODC_ERR_ALIAS;
    }
  }
  DeviceGuard guard(c->device);
  cudaStream_t st = static_cast<cudaStream_t>(stream);
  if (flush_pending(c, st) != COCODC_OK) return COCODC_ERR_CUDA;
  OuterArgs A{};
  A.w_now = w_now;
  A.w_snap = w_snap;
  A.now_stride = now_stride;
  A.snap_stride = snap_stride;
  A.theta_g = theta_g;
  A.momentum = momentum;
  A.delta_out = delta_g_out;
  for (int r = 0; r < n_sums; ++r) A.delta_in[r] = delta_sums[r];
  A.n_recv = n_sums;
  A.partial = do_sums ? c->d_partial : nullptr;
  if (do_sums) {   // Eq. 10 is formed by the last warp of the same launch
    A.fin.ticket = c->d_ticket;
    A.fin.mode = 0;
    A.fin.write_scores = do_score ? 1 : 0;
    A.fin.ids = ids;
    A.fin.t_p = t_p;
    A.fin.t_l = t_l;
    A.fin.t_p_dev = reinterpret_cast<const long long*>(t_p_dev);
    A.fin.t_l_dev = reinterpret_cast<const long long*>(t_l_dev);
    A.fin.last_sync = reinterpret_cast<long long*>(last_sync);
    A.fin.norms = norms;
    A.fin.scores = scores;
    A.fin.sumsq_out = sumsq_out;
    A.fin.in_flight = do_score ? c->in_flight : nullptr;
    A.fin.err_nonfinite = (int)COCODC_ERR_NONFINITE;
    A.fin.defer = defer ? c->d_pending : nullptr;
  }
  fold_coefficients(h, same, &A);
  if (received) {   // Eq. 1 divides the received sum by the number of workers that contributed to it
    A.Mf = (float)M_total;
    A.inv_M = 1.0f / (float)M_total;
    A.M_pow2 = ((M_total & (M_total - 1)) == 0) ? 1 : 0;
  }
  set_status_sink(c, &A);
  const int mode = received ? MODE_FUSED_RECV : (do_merge ? MODE_FUSED : MODE_OUTER_ONLY);
  s = launch_outer(c, A, mode, same, ids, n_ids, snap_offset, st);
  if (s == COCODC_OK && defer) {
    c->pending = true;
    c->pend_norms = norms;
    c->pend_scores = scores;
    c->pend_last = reinterpret_cast<long long*>(last_sync);
  }
  return s;
}

}  // namespace

extern "C" {

cocodc_status cocodc_outer_step(cocodc_ctx* c, const cocodc_hyper* h,
                                float* w_now, const float* w_snap,
                                int64_t now_stride, int64_t snap_stride, const int64_t* snap_offset,
                                float* theta_g, float* momentum, float* delta_g_out,
                                const int32_t* ids, const int32_t* n_ids,
                                int64_t t_p, int64_t t_l, int64_t* last_sync,
                                float* norms, float* scores, double* sumsq_out, uint32_t stages, void* stream) {
  return outer_step_impl(c, h, w_now, w_snap, now_stride, snap_stride, snap_offset, theta_g, momentum, delta_g_out,
                         ids, n_ids, t_p, t_l, last_sync, norms, scores, sumsq_out, stages, stream, nullptr, 0, 0);
}

cocodc_status cocodc_outer_step_received(cocodc_ctx* c, const cocodc_hyper* h, int32_t M_total,
                                         float* w_now, const float* w_snap,
                                         int64_t now_stride, int64_t snap_stride, const int64_t* snap_offset,
                                         float* theta_g, float* momentum, const float* delta_sum,
                                         float* delta_g_out, const int32_t* ids, const int32_t* n_ids,
                                         int64_t t_p, int64_t t_l, int64_t* last_sync,
                                         float* norms, float* scores, void* stream) {
  if (!delta_sum) return COCODC_ERR_INVALID_ARG;
  return outer_step_impl(c, h, w_now, w_snap, now_stride, snap_stride, snap_offset, theta_g, momentum, delta_g_out,
                         ids, n_ids, t_p, t_l, last_sync, norms, scores, nullptr, COCODC_STAGE_ALL, stream, &delta_sum, 1,
                         M_total);
}

cocodc_status cocodc_outer_step_received_peers(cocodc_ctx* c, const cocodc_hyper* h, int32_t M_total,
                                               float* w_now, const float* w_snap,
                                               int64_t now_stride, int64_t snap_stride, const int64_t* snap_offset,
                                               float* theta_g, float* momentum,
                                               const float* const* delta_sums, int32_t n_sums,
                                               float* delta_g_out, const int32_t* ids, const int32_t* n_ids,
                                               int64_t t_p, int64_t t_l, int64_t* last_sync,
                                               float* norms, float* scores, void* stream) {
  if (!delta_sums || n_sums < 1) return COCODC_ERR_INVALID_ARG;
  return outer_step_impl(c, h, w_now, w_snap, now_stride, snap_stride, snap_offset, theta_g, momentum, delta_g_out,
                         ids, n_ids, t_p, t_l, last_sync, norms, scores, nullptr, COCODC_STAGE_ALL, stream, delta_sums,
                         n_sums, M_total);
}

cocodc_status cocodc_select_fragments(cocodc_ctx* c, const float* scores, const int64_t* last_sync,
                                      const uint8_t* ineligible, int64_t t_now, int64_t H,
                                      int32_t budget_kind, int64_t budget,
                                      uint8_t* mask, int32_t* ids, int32_t* n_sel,
                                      int64_t* pool_offset, void* stream) {
  return select_impl(c, scores, last_sync, ineligible, t_now, nullptr, H, budget_kind, budget, mask, ids, n_sel,
                     pool_offset, stream);
}

cocodc_status cocodc_select_fragments_at(cocodc_ctx* c, const float* scores, const int64_t* last_sync,
                                         const uint8_t* ineligible, const int64_t* t_now, int64_t H,
                                         int32_t budget_kind, int64_t budget,
                                         uint8_t* mask, int32_t* ids, int32_t* n_sel,
                                         int64_t* pool_offset, void* stream) {
  if (!t_now) return COCODC_ERR_INVALID_ARG;
  return select_impl(c, scores, last_sync, ineligible, 0, t_now, H, budget_kind, budget, mask, ids, n_sel,
                     pool_offset, stream);
}

cocodc_status cocodc_outer_step_at(cocodc_ctx* c, const cocodc_hyper* h,
                                   float* w_now, const float* w_snap,
                                   int64_t now_stride, int64_t snap_stride, const int64_t* snap_offset,
                                   float* theta_g, float* momentum, float* delta_g_out,
                                   const int32_t* ids, const int32_t* n_ids,
                                   const int64_t* t_p, const int64_t* t_l, int64_t* last_sync,
                                   float* norms, float* scores, double* sumsq_out, uint32_t stages, void* stream) {
  if (!t_p || !t_l) return COCODC_ERR_INVALID_ARG;
  return outer_step_impl(c, h, w_now, w_snap, now_stride, snap_stride, snap_offset, theta_g, momentum, delta_g_out,
                         ids, n_ids, 0, 0, last_sync, norms, scores, sumsq_out, stages, stream, nullptr, 0, 0, t_p,
                         t_l);
}

cocodc_status cocodc_pseudo_gradient_sum(cocodc_ctx* c, const float* w_snap, int64_t snap_stride,
                                         const int64_t* snap_offset, const float* theta_g, int32_t M,
                                         float* sum_out, const int32_t* ids, const int32_t* n_ids, void* stream) {
  if (!c || !w_snap || !theta_g || !sum_out || !ids || !n_ids) return COCODC_ERR_INVALID_ARG;
  if (M < 1 || M > c->max_M) return COCODC_ERR_INVALID_ARG;
  const long long N = c->N;
  if (snap_stride < (snap_offset ? 1 : N)) return COCODC_ERR_INVALID_ARG;
  if (!aligned16(w_snap) || !aligned16(theta_g) || !aligned16(sum_out) || (snap_stride & 3)) return COCODC_ERR_ALIGNMENT;
  const Range ro = range_of(sum_out, N);
  if (overlap(ro, range_of(theta_g, N)) ||
      overlap(ro, range_of(w_snap, (long long)(M - 1) * snap_stride + (snap_offset ? snap_stride : N))))
    return COCODC_ERR_ALIAS;
  DeviceGuard guard(c->device);
  cudaStream_t st = static_cast<cudaStream_t>(stream);
  OuterArgs A{};
  A.w_snap = w_snap; A.snap_stride = snap_stride; A.now_stride = N;
  A.theta_g = const_cast<float*>(theta_g);   // read only in this mode
  A.delta_out = sum_out;
  A.partial = nullptr;
  A.status = c->d_status; A.err_timeout = COCODC_ERR_TIMEOUT;
  A.M = M;
  return launch_outer(c, A, MODE_PSEUDO_SUM, false, ids, n_ids, snap_offset, st);
}

cocodc_status cocodc_merge(cocodc_ctx* c, const cocodc_hyper* h,
                           float* w_now, const float* w_snap,
                           int64_t now_stride, int64_t snap_stride, const int64_t* snap_offset,
                           const float* theta_g_new, const int32_t* ids, const int32_t* n_ids, void* stream) {
  cocodc_status s = check_hyper(c, h);
  if (s != COCODC_OK) return s;
  if (!w_now || !w_snap || !theta_g_new || !ids || !n_ids) return COCODC_ERR_INVALID_ARG;
  const long long N = c->N;
  if (now_stride < N || snap_stride < (snap_offset ? 1 : N)) return COCODC_ERR_INVALID_ARG;
  const bool same = (w_snap == w_now) && (snap_stride == now_stride) && (snap_offset == nullptr);
  if (h->tau == 0 && h->comp_mode == COCODC_COMP_TAYLOR && !same) return COCODC_ERR_INVALID_ARG;
  if (!aligned16(w_now) || !aligned16(w_snap) || !aligned16(theta_g_new) || (now_stride & 3) || (snap_stride & 3))
    return COCODC_ERR_ALIGNMENT;
  {
    const int M = h->M;
    const Range rn = range_of(w_now, (long long)(M - 1) * now_stride + N);
    if (overlap(rn, range_of(theta_g_new, N))) return COCODC_ERR_ALIAS;
    if (!same && overlap(rn, range_of(w_snap, (long long)(M - 1) * snap_stride + (snap_offset ? snap_stride : N))))
      return COCODC_ERR_ALIAS;
  }
  DeviceGuard guard(c->device);
  cudaStream_t st = static_cast<cudaStream_t>(stream);
  OuterArgs A{};
  A.w_now = w_now;
  A.w_snap = w_snap;
  A.now_stride = now_stride;
  A.snap_stride = snap_stride;
  A.theta_g = const_cast<float*>(theta_g_new);  // read only in this mode
  fold_coefficients(h, same, &A);
  set_status_sink(c, &A);
  return launch_outer(c, A, MODE_MERGE_ONLY, same, ids, n_ids, snap_offset, st);
}

cocodc_status cocodc_snapshot(cocodc_ctx* c, const float* w_now, float* w_snap,
                              int64_t now_stride, int64_t snap_stride, const int64_t* snap_offset,
                              int32_t M, const int32_t* ids, const int32_t* n_ids, void* stream) {
  if (!c || !w_now || !w_snap || !ids || !n_ids) return COCODC_ERR_INVALID_ARG;
  if (M < 1 || M > c->max_M) return COCODC_ERR_INVALID_ARG;
  const long long N = c->N;
  if (now_stride < N || snap_stride < (snap_offset ? 1 : N)) return COCODC_ERR_INVALID_ARG;
  if (!aligned16(w_now) || !aligned16(w_snap) || (now_stride & 3) || (snap_stride & 3)) return COCODC_ERR_ALIGNMENT;
  if (overlap(range_of(w_now, (long long)(M - 1) * now_stride + N),
              range_of(w_snap, (long long)(M - 1) * snap_stride + (snap_offset ? snap_stride : N))))
    return COCODC_ERR_ALIAS;
  DeviceGuard guard(c->device);
  cudaStream_t st = static_cast<cudaStream_t>(stream);
  opt_in_shared_memory(c, reinterpret_cast<const void*>(k_snapshot_tma), kSnapSmemBytes);
  PlanRequest rq{};
  const SegPlan* gplan = nullptr;
  const PlanHeader* ghdr = nullptr;
  cocodc_status s = prepare_plan(c, ids, n_ids, snap_offset, snap_stride, kThreads * kSnapU, st, &rq, &gplan, &ghdr);
  if (s != COCODC_OK) return s;
  k_snapshot_tma<<<c->sm_count, kThreads, kSnapSmemBytes, st>>>(w_now, w_snap, now_stride, snap_stride, M, gplan, ghdr,
                                                                rq, c->d_status, (int)COCODC_ERR_TIMEOUT, c->table,
                                                                SelectRequest{});
  c->launches++;
  return cudaGetLastError() == cudaSuccess ? COCODC_OK : COCODC_ERR_CUDA;
}

}  // extern "C"

namespace {
cocodc_status initiate_impl(cocodc_ctx* c, const float* scores, const int64_t* last_sync, const uint8_t* ineligible,
                            int64_t t_now, const int64_t* t_now_dev, int64_t H, int32_t budget_kind, int64_t budget,
                            uint8_t* mask, int32_t* ids, int32_t* n_sel, int64_t* pool_offset,
                            const float* w_now, float* w_snap, int64_t now_stride, int64_t snap_stride, int32_t M,
                            void* stream) {
  if (!c || !scores || !last_sync || !mask || !ids || !n_sel || !w_now || !w_snap) return COCODC_ERR_INVALID_ARG;
  if (H < 1 || budget < 0 || M < 1 || M > c->max_M) return COCODC_ERR_INVALID_ARG;
  if (budget_kind != COCODC_BUDGET_COUNT && budget_kind != COCODC_BUDGET_PARAMS &&
      budget_kind != COCODC_BUDGET_PARAMS_EXACT)
    return COCODC_ERR_INVALID_ARG;
  const long long N = c->N;
  if (now_stride < N || snap_stride < (pool_offset ? 1 : N)) return COCODC_ERR_INVALID_ARG;
  if (!aligned16(w_now) || !aligned16(w_snap) || (now_stride & 3) || (snap_stride & 3)) return COCODC_ERR_ALIGNMENT;
  if (overlap(range_of(w_now, (long long)(M - 1) * now_stride + N),
              range_of(w_snap, (long long)(M - 1) * snap_stride + (pool_offset ? snap_stride : N))))
    return COCODC_ERR_ALIAS;
  if (!c->inline_plan || budget_kind == COCODC_BUDGET_PARAMS_EXACT) {
    // a table too large to be a kernel argument, or the enumerating budget: the two calls one after the other
    // (select_impl forms the scores of a deferred completion first)
    cocodc_status s = select_impl(c, scores, last_sync, ineligible, t_now, t_now_dev, H, budget_kind, budget, mask,
                                  ids, n_sel, pool_offset, stream);
    if (s != COCODC_OK) return s;
    return cocodc_snapshot(c, w_now, w_snap, now_stride, snap_stride, pool_offset, M, ids, n_sel, stream);
  }
  DeviceGuard guard(c->device);
  cudaStream_t st = static_cast<cudaStream_t>(stream);
  // A deferred completion is consumed by this launch if it was given the arrays this selection reads; otherwise
  // its scores are formed first, where it said.
  if (c->pending && (c->pend_scores != scores || c->pend_last != reinterpret_cast<const long long*>(last_sync)) &&
      flush_pending(c, st) != COCODC_OK)
    return COCODC_ERR_CUDA;
  opt_in_shared_memory(c, reinterpret_cast<const void*>(k_snapshot_tma), kSnapSmemBytes);
  PlanRequest rq{};
  rq.snap_row_len = snap_stride;
  rq.lanes_per_tile = kThreads * kSnapU;
  rq.err_invalid = (int)COCODC_ERR_INVALID_ARG;
  SelectRequest q{};
  q.scores = scores;
  q.last_sync = reinterpret_cast<const long long*>(last_sync);
  q.ineligible = ineligible;
  q.in_flight = c->in_flight;
  q.t_now = t_now;
  q.t_now_dev = reinterpret_cast<const long long*>(t_now_dev);
  q.H = H;
  q.budget_kind = budget_kind;
  q.budget = budget;
  q.mask = mask;
  q.ids = ids;
  q.n_sel = n_sel;
  q.pool_offset = reinterpret_cast<long long*>(pool_offset);
  q.ticket = c->d_ticket;
  q.err_nonfinite = (int)COCODC_ERR_NONFINITE;
  if (c->pending) {
    q.pending = c->d_pending;
    q.partial = c->d_partial;
    q.norms = c->pend_norms;
    q.scores_out = c->pend_scores;
    q.last_sync_out = c->pend_last;
    q.pend_grid = c->pend_grid;
    q.pend_warps = kThreads / 32;
    c->pending = false;
  }
  k_snapshot_tma<<<c->sm_count, kThreads, kSnapSmemBytes, st>>>(w_now, w_snap, now_stride, snap_stride, M, nullptr,
                                                                nullptr, rq, c->d_status, (int)COCODC_ERR_TIMEOUT,
                                                                c->table, q);
  c->launches++;
  return cudaGetLastError() == cudaSuccess ? COCODC_OK : COCODC_ERR_CUDA;
}
}  // namespace

extern "C" {

cocodc_status cocodc_initiate(cocodc_ctx* c, const float* scores, const int64_t* last_sync, const uint8_t* ineligible,
                              int64_t t_now, int64_t H, int32_t budget_kind, int64_t budget,
                              uint8_t* mask, int32_t* ids, int32_t* n_sel, int64_t* pool_offset,
                              const float* w_now, float* w_snap, int64_t now_stride, int64_t snap_stride, int32_t M,
                              void* stream) {
  return initiate_impl(c, scores, last_sync, ineligible, t_now, nullptr, H, budget_kind, budget, mask, ids, n_sel,
                       pool_offset, w_now, w_snap, now_stride, snap_stride, M, stream);
}

cocodc_status cocodc_initiate_at(cocodc_ctx* c, const float* scores, const int64_t* last_sync,
                                 const uint8_t* ineligible, const int64_t* t_now, int64_t H, int32_t budget_kind,
                                 int64_t budget, uint8_t* mask, int32_t* ids, int32_t* n_sel, int64_t* pool_offset,
                                 const float* w_now, float* w_snap, int64_t now_stride, int64_t snap_stride, int32_t M,
                                 void* stream) {
  if (!t_now) return COCODC_ERR_INVALID_ARG;
  return initiate_impl(c, scores, last_sync, ineligible, 0, t_now, H, budget_kind, budget, mask, ids, n_sel,
                       pool_offset, w_now, w_snap, now_stride, snap_stride, M, stream);
}

cocodc_status cocodc_outer_step_host(cocodc_ctx* c, const cocodc_hyper* h,
                                     float* w_now, const float* w_snap,
                                     int64_t now_stride, int64_t snap_stride, const int64_t* snap_offset,
                                     float* theta_g, float* momentum, float* delta_g_out,
                                     const int32_t* ids, int32_t n_ids,
                                     int64_t t_p, int64_t t_l, int64_t* last_sync,
                                     float* norms, float* scores, int32_t snap_on_device,
                                     void* workspace, uint64_t workspace_bytes, void* stream) {
  cocodc_status s = check_hyper(c, h);
  if (s != COCODC_OK) return s;
  if (!w_now || !w_snap || !theta_g || !momentum || !ids || !last_sync || !norms || !scores || !workspace)
    return COCODC_ERR_INVALID_ARG;
  if (n_ids < 0 || n_ids > c->K || t_l < t_p) return COCODC_ERR_INVALID_ARG;
  const long long N = c->N;
  const int M = h->M, K = c->K;
  if (now_stride < N || snap_stride < (snap_offset ? 1 : N)) return COCODC_ERR_INVALID_ARG;
  const bool same = !snap_on_device && (w_snap == w_now) && (snap_stride == now_stride) && (snap_offset == nullptr);
  if (h->tau == 0 && h->comp_mode == COCODC_COMP_TAYLOR && !same) return COCODC_ERR_INVALID_ARG;
  if (!aligned16(workspace)) return COCODC_ERR_ALIGNMENT;
  if (snap_on_device && (!aligned16(w_snap) || (snap_stride & 3))) return COCODC_ERR_ALIGNMENT;
  {
    char seen[kMaxK] = {};
    for (int j = 0; j < n_ids; ++j) {
      const int p = ids[j];
      if (p < 0 || p >= K || seen[p]) return COCODC_ERR_INVALID_ARG;
      if (snap_offset && (snap_offset[p] < 0 || snap_offset[p] + fragment_elems(c, p) > snap_stride))
        return COCODC_ERR_INVALID_ARG;   // no place, or not inside one row of the pool
      seen[p] = 1;
    }
    Range r[4];
    int nr = 0;
    r[nr++] = range_of(theta_g, N);
    r[nr++] = range_of(momentum, N);
    if (delta_g_out) r[nr++] = range_of(delta_g_out, N);
    r[nr++] = range_of(w_now, (long long)(M - 1) * now_stride + N);
    for (int i = 0; i < nr; ++i)
      for (int j = i + 1; j < nr; ++j)
        if (overlap(r[i], r[j])) return COCODC_ERR_ALIAS;
    if (!same && !snap_on_device) {
      const Range rs = range_of(w_snap, (long long)(M - 1) * snap_stride + (snap_offset ? snap_stride : N));
      for (int i = 0; i < nr; ++i) if (overlap(rs, r[i])) return COCODC_ERR_ALIAS;
    }
  }
  // staging slots: [snap M][now M][theta_g][momentum][delta] chunks of C elements each
  const long long per_elem = 2LL * M + 3;
  long long C = (long long)(workspace_bytes / sizeof(float)) / (cocodc_ctx::kSlots * per_elem);
  C &= ~1023LL;
  if (C < 4096) return COCODC_ERR_INVALID_ARG;
  if (C > (1LL << 28)) C = 1LL << 28;

  DeviceGuard guard(c->device);
  cudaStream_t st = static_cast<cudaStream_t>(stream);
  if (flush_pending(c, st) != COCODC_OK) return COCODC_ERR_CUDA;
  const Variant v = pick_variant(M, MODE_FUSED, same);
  const int grid = variant_grid(c, v);
  opt_in_shared_memory(c, reinterpret_cast<const void*>(v.kernel), v.smem);
  const int entries = grid * (kThreads / 32);
  bool ok = true;
  auto CK = [&](cudaError_t e) { ok = ok && (e == cudaSuccess); };
  CK(cudaMemsetAsync(c->d_frag_sumsq, 0, sizeof(double) * K, st));
  CK(cudaMemcpyAsync(c->d_k_ids, ids, sizeof(int) * n_ids, cudaMemcpyHostToDevice, st));
  CK(cudaMemcpyAsync(c->d_k_last, last_sync, sizeof(long long) * K, cudaMemcpyHostToDevice, st));
  CK(cudaMemcpyAsync(c->d_k_norms, norms, sizeof(float) * K, cudaMemcpyHostToDevice, st));
  CK(cudaMemcpyAsync(c->d_k_scores, scores, sizeof(float) * K, cudaMemcpyHostToDevice, st));

  OuterArgs A{};
  A.now_stride = C;
  A.snap_stride = C;
  A.plan = c->d_plan;
  A.hdr = c->d_hdr;
  A.partial = c->d_partial;
  fold_coefficients(h, same, &A);
  set_status_sink(c, &A);
  const size_t B4 = sizeof(float);
  long long chunk = 0;
  for (int j = 0; j < n_ids && ok; ++j) {
    const int p = ids[j];
    long long pos = 0;
    for (int sgi = c->h_frag_seg_ptr[p]; sgi < c->h_frag_seg_ptr[p + 1] && ok; ++sgi) {
      const long long off = c->h_seg_off[sgi], len = c->h_seg_len[sgi];
      const long long sbase = snap_offset ? snap_offset[p] + pos : off;
      for (long long lo = 0; lo < len && ok; lo += C, ++chunk) {
        const long long cnt = std::min(C, len - lo);
        const int slot = (int)(chunk % cocodc_ctx::kSlots);
        float* base = static_cast<float*>(workspace) + (size_t)slot * per_elem * C;
        float* d_snap = base;
        float* d_now = base + (size_t)M * C;
        float* d_thg = base + (size_t)2 * M * C;
        float* d_u = d_thg + C;
        float* d_delta = d_u + C;
        // host -> device, once the slot's previous results have left it
        if (chunk >= cocodc_ctx::kSlots) CK(cudaStreamWaitEvent(c->s_h2d, c->ev_d2h[slot], 0));
        for (int m = 0; m < M; ++m) {
          if (!same && !snap_on_device)
            CK(cudaMemcpyAsync(d_snap + (size_t)m * C, w_snap + (size_t)m * snap_stride + sbase + lo, cnt * B4,
                               cudaMemcpyHostToDevice, c->s_h2d));
          CK(cudaMemcpyAsync(d_now + (size_t)m * C, w_now + (size_t)m * now_stride + off + lo, cnt * B4,
                             cudaMemcpyHostToDevice, c->s_h2d));
        }
        CK(cudaMemcpyAsync(d_thg, theta_g + off + lo, cnt * B4, cudaMemcpyHostToDevice, c->s_h2d));
        CK(cudaMemcpyAsync(d_u, momentum + off + lo, cnt * B4, cudaMemcpyHostToDevice, c->s_h2d));
        CK(cudaEventRecord(c->ev_h2d[slot], c->s_h2d));
        // compute on the caller's stream
        CK(cudaStreamWaitEvent(st, c->ev_h2d[slot], 0));
        A.w_now = d_now;
        A.w_snap = same ? d_now : (snap_on_device ? w_snap : d_snap);
        A.snap_stride = snap_on_device ? snap_stride : C;
        A.theta_g = d_thg;
        A.momentum = d_u;
        A.delta_out = delta_g_out ? d_delta : nullptr;
        A.ring_slots = v.ring_slots;
        k_plan_chunk<<<1, 1, 0, st>>>(cnt, snap_on_device ? sbase + lo : 0, v.lanes_per_tile, c->d_plan, c->d_hdr);
        v.kernel<<<grid, v.threads, v.smem, st>>>(A, c->table);
        k_accumulate_chunk<<<1, kFinalizeThreads, 0, st>>>(c->d_partial, entries, c->d_frag_sumsq + j);
        c->launches += 3;
        CK(cudaEventRecord(c->ev_comp[slot], st));
        // device -> host
        CK(cudaStreamWaitEvent(c->s_d2h, c->ev_comp[slot], 0));
        for (int m = 0; m < M; ++m)
          CK(cudaMemcpyAsync(w_now + (size_t)m * now_stride + off + lo, d_now + (size_t)m * C, cnt * B4,
                             cudaMemcpyDeviceToHost, c->s_d2h));
        CK(cudaMemcpyAsync(theta_g + off + lo, d_thg, cnt * B4, cudaMemcpyDeviceToHost, c->s_d2h));
        CK(cudaMemcpyAsync(momentum + off + lo, d_u, cnt * B4, cudaMemcpyDeviceToHost, c->s_d2h));
        if (delta_g_out)
          CK(cudaMemcpyAsync(delta_g_out + off + lo, d_delta, cnt * B4, cudaMemcpyDeviceToHost, c->s_d2h));
        CK(cudaEventRecord(c->ev_d2h[slot], c->s_d2h));
      }
      pos += len;
    }
  }
  if (ok && n_ids > 0) {
    k_scores_from_sumsq<<<1, kFinalizeThreads, 0, st>>>(c->d_frag_sumsq, 1, c->d_k_ids, nullptr, n_ids, K, 0, nullptr,
                                                        t_p, t_l, c->d_k_last, c->d_k_norms, c->d_k_scores, nullptr,
                                                        c->d_status, (int)COCODC_ERR_NONFINITE,
                                                        (int)COCODC_ERR_INVALID_ARG);
    c->launches++;
  }
  CK(cudaMemcpyAsync(last_sync, c->d_k_last, sizeof(long long) * K, cudaMemcpyDeviceToHost, st));
  CK(cudaMemcpyAsync(norms, c->d_k_norms, sizeof(float) * K, cudaMemcpyDeviceToHost, st));
  CK(cudaMemcpyAsync(scores, c->d_k_scores, sizeof(float) * K, cudaMemcpyDeviceToHost, st));
  // the call is synchronous: results are in host memory when it returns
  cudaError_t e1 = cudaStreamSynchronize(c->s_h2d);
  cudaError_t e2 = cudaStreamSynchronize(st);
  cudaError_t e3 = cudaStreamSynchronize(c->s_d2h);
  if (!ok || e1 != cudaSuccess || e2 != cudaSuccess || e3 != cudaSuccess || cudaGetLastError() != cudaSuccess)
    return COCODC_ERR_CUDA;
  return COCODC_OK;
}

cocodc_status cocodc_snapshot_host(cocodc_ctx* c, const float* w_now, float* w_snap,
                                   int64_t now_stride, int64_t snap_stride, const int64_t* snap_offset,
                                   int32_t M, const int32_t* ids, int32_t n_ids, void* stream) {
  if (!c || !w_now || !w_snap || !ids) return COCODC_ERR_INVALID_ARG;
  if (M < 1 || M > c->max_M || n_ids < 0 || n_ids > c->K) return COCODC_ERR_INVALID_ARG;
  if (now_stride < c->N || snap_stride < (snap_offset ? 1 : c->N)) return COCODC_ERR_INVALID_ARG;
  for (int j = 0; j < n_ids; ++j) {
    if (ids[j] < 0 || ids[j] >= c->K) return COCODC_ERR_INVALID_ARG;
    if (snap_offset && (snap_offset[ids[j]] < 0 || snap_offset[ids[j]] + fragment_elems(c, ids[j]) > snap_stride))
      return COCODC_ERR_INVALID_ARG;
  }
  DeviceGuard guard(c->device);
  cudaStream_t st = static_cast<cudaStream_t>(stream);
  bool ok = true;
  for (int j = 0; j < n_ids; ++j) {
    const int p = ids[j];
    long long pos = 0;
    for (int sgi = c->h_frag_seg_ptr[p]; sgi < c->h_frag_seg_ptr[p + 1]; ++sgi) {
      const long long off = c->h_seg_off[sgi], len = c->h_seg_len[sgi];
      const long long sbase = snap_offset ? snap_offset[p] + pos : off;
      for (int m = 0; m < M; ++m)
        ok = ok && cudaMemcpyAsync(w_snap + (size_t)m * snap_stride + sbase, w_now + (size_t)m * now_stride + off,
                                   (size_t)len * sizeof(float), cudaMemcpyHostToDevice, st) == cudaSuccess;
      pos += len;
    }
  }
  return ok ? COCODC_OK : COCODC_ERR_CUDA;
}

cocodc_status cocodc_selftest_bounded_wait(cocodc_ctx* c, int32_t polls, void* stream) {
  if (!c || polls < 1 || polls > kWaitLimit) return COCODC_ERR_INVALID_ARG;
  DeviceGuard guard(c->device);
  k_selftest_bounded_wait<<<1, 32, 0, static_cast<cudaStream_t>(stream)>>>(polls, c->d_status, (int)COCODC_ERR_TIMEOUT);
  c->launches++;
  return cudaGetLastError() == cudaSuccess ? COCODC_OK : COCODC_ERR_CUDA;
}

}  // extern "C"

// cocodc_fragment_scores_noalloc: the stand-alone fragment scores (Eq. 10) for callers that must
// not allocate device memory.
//
// Who needs this: code that runs where cudaMalloc is off limits - inside a framework's memory-pool
// callback or an allocator hook (allocating there re-enters the allocator), in a process whose
// device memory was handed out up front by a supervisor and whose runtime heap is capped at zero,
// or on a latency-critical path where an allocation's implicit device synchronisation is not
// acceptable.  Such callers cannot create a cocodc context either (cocodc_create allocates), so
// this entry point takes the fragment table directly and keeps its scratch in a fixed array that
// is part of the library image.
//
// The scratch is the per-CTA, per-warp partial sums of squares that the regular
// cocodc_fragment_scores keeps in context memory.  Here it is a file-scope __device__ array of
// kNoallocScratchBytes (592 KiB); every GPU that loads the library holds it until the process
// exits.  Limits that follow from its size: at most COCODC_NOALLOC_MAX_K fragments and
// COCODC_NOALLOC_MAX_SEGMENTS segments.
#include "../../include/cocodc.h"

#include <cuda_runtime.h>

#include <algorithm>
#include <mutex>
#include <utility>
#include <vector>

#include "outer.cuh"

using namespace cocodc;

namespace {

constexpr int kNoallocMaxK = COCODC_NOALLOC_MAX_K;
constexpr int kNoallocMaxSeg = COCODC_NOALLOC_MAX_SEGMENTS;
constexpr int kGrid = 1184;                // fixed launch width (8 CTAs on each of 148 SMs): the scratch is sized for it
constexpr int kWarps = kThreads / 32;
constexpr int kU = 4;                      // 16-byte lanes per thread and tile
constexpr size_t kScratchDoubles = (size_t)kNoallocMaxK * kGrid;   // one double per (fragment, CTA)
constexpr size_t kNoallocScratchBytes = kScratchDoubles * sizeof(double);
static_assert(kNoallocScratchBytes <= (2u << 20), "the fixed scratch is meant to stay modest");

// The scratch itself.  In host code this name is only a handle for the runtime's symbol calls, not
// an address a kernel could use: the device address is looked up once per device below.
static __device__ __align__(256) double g_noalloc_scratch[kScratchDoubles];

// The whole launch plan travels as a kernel argument (about 3 KB), so no device table is needed.
struct PlanTable {
  PlanHeader hdr;
  SegPlan seg[kNoallocMaxSeg];
};

// Per-CTA running sum of squares of the current fragment.  When the fragment changes (the same tile, hence
// the same moment, for every thread of the CTA) the warps reduce, thread 0 adds the warp sums in warp order
// and writes partial[fragment * gridDim.x + CTA]; fragments the CTA never touched get an explicit zero.
struct CtaAccumulator {
  double acc = 0.0;
  int slot = 0;
  double* warp_sums;   // shared, one per warp

  __device__ __forceinline__ explicit CtaAccumulator(double* shared_warp_sums) : warp_sums(shared_warp_sums) {}
  __device__ __forceinline__ void flush_to(int new_slot, double* __restrict__ partial) {
    const double v = warp_sum(acc);
    if ((threadIdx.x & 31) == 0) warp_sums[threadIdx.x >> 5] = v;
    __syncthreads();
    if (threadIdx.x == 0) {
      double s = 0.0;
      for (int w = 0; w < kWarps; ++w) s += warp_sums[w];
      partial[(size_t)slot * gridDim.x + blockIdx.x] = s;
      for (int z = slot + 1; z < new_slot; ++z) partial[(size_t)z * gridDim.x + blockIdx.x] = 0.0;
    }
    __syncthreads();
    acc = 0.0;
    slot = new_slot;
  }
  __device__ __forceinline__ void advance(int new_slot, double* __restrict__ partial) {
    if (new_slot != slot) flush_to(new_slot, partial);
  }
  __device__ __forceinline__ void finish(int n_ids, double* __restrict__ partial) {
    if (slot < n_ids) flush_to(n_ids, partial);
  }
};

// Variant of k_sumsq that reads its plan from the argument block and writes its partial sums to
// the scratch array.  Every (fragment, CTA) entry that the finalize kernel reads is written
// by this kernel in the same call (untouched ones with an explicit zero), so what an earlier call
// left in the array is never read and nothing has to be cleared.
__global__ void __launch_bounds__(kThreads)
k_sumsq_table(const float* __restrict__ x, const __grid_constant__ PlanTable plan, double* __restrict__ partial) {
  constexpr int LPT = kThreads * kU;
  __shared__ double warp_sums[kWarps];
  CtaAccumulator sa(warp_sums);
  int seg = 0;
  for (int tile = blockIdx.x; tile < plan.hdr.total_tiles; tile += gridDim.x) {
    while (seg + 1 < plan.hdr.n_seg && tile >= plan.seg[seg + 1].first_tile) ++seg;
    const SegPlan& sp = plan.seg[seg];
    sa.advance(sp.slot, partial);
    const long long e_tile = sp.abase + 4LL * (long long)(tile - sp.first_tile) * LPT;
    const long long seg_end = sp.off + sp.len;
    if (e_tile >= sp.off && e_tile + 4LL * LPT <= seg_end) {
      float4 v[kU];
#pragma unroll
      for (int j = 0; j < kU; ++j) v[j] = ld4(x + e_tile + 4LL * (j * kThreads + threadIdx.x));
#pragma unroll
      for (int j = 0; j < kU; ++j) {
        float sq = __fmul_rn(v[j].x, v[j].x);
        sq = __fmaf_rn(v[j].y, v[j].y, sq);
        sq = __fmaf_rn(v[j].z, v[j].z, sq);
        sq = __fmaf_rn(v[j].w, v[j].w, sq);
        sa.acc += (double)sq;
      }
    } else {
      for (int j = 0; j < kU; ++j) {
        const long long e = e_tile + 4LL * (j * kThreads + threadIdx.x);
        if (e >= seg_end) break;
        for (int k = 0; k < 4; ++k) {
          const long long ee = e + k;
          if (ee >= sp.off && ee < seg_end) { const float t = ld1(x + ee); sa.acc += (double)__fmul_rn(t, t); }
        }
      }
    }
  }
  sa.finish(plan.hdr.n_ids, partial);
}

// One block per fragment: fixed-order sum of the fragment's partials, norm and score (Eq. 10).
__global__ void __launch_bounds__(kFinalizeThreads)
k_finalize_table(const double* __restrict__ partial, int entries_per_slot, const long long* __restrict__ interval,
                 float* __restrict__ norms, float* __restrict__ scores) {
  __shared__ double red[kFinalizeThreads];
  const int p = blockIdx.x;
  const double* src = partial + (size_t)p * entries_per_slot;
  double s = 0.0;
  for (int i = threadIdx.x; i < entries_per_slot; i += kFinalizeThreads) s += src[i];
  red[threadIdx.x] = s;
  __syncthreads();
#pragma unroll
  for (int w = kFinalizeThreads / 2; w > 0; w >>= 1) {
    if (threadIdx.x < w) red[threadIdx.x] += red[threadIdx.x + w];
    __syncthreads();
  }
  if (threadIdx.x != 0) return;
  const double norm = sqrt(red[0]);
  long long I = interval ? interval[p] : 1;
  if (I < 1) I = 1;
  norms[p] = (float)norm;
  scores[p] = (float)(norm / (double)I);
}

// Device address of the scratch array, looked up once per device with that device current.
constexpr int kMaxDevices = 64;
std::mutex g_setup_mutex;
double* g_scratch_ptr[kMaxDevices] = {};

cocodc_status scratch_for_device(int device, double** out) {
  std::lock_guard<std::mutex> lock(g_setup_mutex);
  if (g_scratch_ptr[device] == nullptr) {
    int prev = -1;
    if (cudaGetDevice(&prev) != cudaSuccess) return COCODC_ERR_CUDA;
    if (prev != device && cudaSetDevice(device) != cudaSuccess) return COCODC_ERR_CUDA;
    void* p = nullptr;
    const cudaError_t e = cudaGetSymbolAddress(&p, g_noalloc_scratch);
    if (prev != device) cudaSetDevice(prev);
    if (e != cudaSuccess || p == nullptr) { cudaGetLastError(); return COCODC_ERR_CUDA; }
    g_scratch_ptr[device] = static_cast<double*>(p);
  }
  *out = g_scratch_ptr[device];
  return COCODC_OK;
}

}  // namespace

extern "C" cocodc_status cocodc_fragment_scores_noalloc(const cocodc_partition* part, const float* delta_g,
                                                        const int64_t* interval, float* norms, float* scores,
                                                        int32_t device, void* stream) {
  if (!part || !part->frag_seg_ptr || !part->seg_offset || !part->seg_len || !delta_g || !norms || !scores)
    return COCODC_ERR_INVALID_ARG;
  const int K = part->K, S = part->n_segments;
  if (K < 1 || S < K || part->N < 1) return COCODC_ERR_INVALID_ARG;
  if (K > kNoallocMaxK || S > kNoallocMaxSeg) return COCODC_ERR_INVALID_ARG;   // beyond what the fixed scratch and plan hold
  if (device < 0 || device >= kMaxDevices) return COCODC_ERR_INVALID_ARG;
  if ((reinterpret_cast<uintptr_t>(delta_g) & 15u) != 0) return COCODC_ERR_ALIGNMENT;
  if (part->frag_seg_ptr[0] != 0 || part->frag_seg_ptr[K] != S) return COCODC_ERR_INVALID_ARG;

  PlanTable table;
  long long tiles = 0;
  int ns = 0;
  constexpr int LPT = kThreads * kU;
  std::pair<long long, long long> sorted[kNoallocMaxSeg];
  for (int p = 0; p < K; ++p) {
    if (part->frag_seg_ptr[p + 1] <= part->frag_seg_ptr[p]) return COCODC_ERR_INVALID_ARG;
    if (part->frag_seg_ptr[p + 1] > S) return COCODC_ERR_INVALID_ARG;   // a pointer past the S segments the arrays hold
    for (int s = part->frag_seg_ptr[p]; s < part->frag_seg_ptr[p + 1]; ++s) {
      const long long o = part->seg_offset[s], l = part->seg_len[s];
      if (o < 0 || l < 1 || o > part->N - l) return COCODC_ERR_INVALID_ARG;
      SegPlan sp;
      sp.off = o; sp.len = l; sp.snap_off = o; sp.abase = o & ~3LL;
      sp.first_tile = (int)tiles; sp.slot = p; sp.frag = p; sp.vec_ok = 1;
      sorted[ns] = {o, l};
      table.seg[ns++] = sp;
      const long long lanes = (o - sp.abase + l + 3) >> 2;
      tiles += (lanes + LPT - 1) / LPT;
      if (tiles > 0x3fffffffLL) return COCODC_ERR_INVALID_ARG;
    }
  }
  std::sort(sorted, sorted + ns);
  for (int i = 1; i < ns; ++i)
    if (sorted[i].first < sorted[i - 1].first + sorted[i - 1].second) return COCODC_ERR_INVALID_ARG;
  table.hdr.total_tiles = (int)tiles;
  table.hdr.n_seg = ns;
  table.hdr.n_ids = K;
  table.hdr.pad = 0;

  double* scratch = nullptr;
  cocodc_status st = scratch_for_device(device, &scratch);
  if (st != COCODC_OK) return st;
  int prev = -1;
  if (cudaGetDevice(&prev) != cudaSuccess) return COCODC_ERR_CUDA;
  if (prev != device && cudaSetDevice(device) != cudaSuccess) return COCODC_ERR_CUDA;
  cudaStream_t cs = static_cast<cudaStream_t>(stream);
  k_sumsq_table<<<kGrid, kThreads, 0, cs>>>(delta_g, table, scratch);
  k_finalize_table<<<K, kFinalizeThreads, 0, cs>>>(scratch, kGrid,
                                                   reinterpret_cast<const long long*>(interval), norms, scores);
  const cudaError_t e = cudaGetLastError();
  if (prev != device) cudaSetDevice(prev);
  return e == cudaSuccess ? COCODC_OK : COCODC_ERR_CUDA;
}

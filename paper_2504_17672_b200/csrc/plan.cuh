// Launch plan: which tiles of which segments one call processes.
//
// A call works on a list of fragment ids that lives in device memory (it is
// usually written by the selection kernel, and the host never reads it).  A
// one-block kernel expands that list into a table of segments with a running
// tile count; the streaming kernels then map a tile index to (segment, lane
// range) without any host round-trip.
//
// Geometry.  Every segment [off, off+len) is covered by 16-byte "lanes" of four
// elements that start at abase = off rounded down to a multiple of 4, so lane
// addresses are aligned in every N-sized buffer whose base is aligned.  A tile
// is `lanes_per_tile` consecutive lanes of one segment.  Only the first and the
// last lane of a segment can be partial; partial lanes take a scalar path.
#pragma once

#include <cuda_runtime.h>
#include <stdint.h>

namespace cocodc {

struct SegPlan {
  long long off;       // element offset of the segment in every N-sized buffer
  long long len;       // elements
  long long snap_off;  // element offset of the segment inside a row of w_snap
  long long abase;     // off & ~3
  int first_tile;      // index of the segment's first tile in this launch
  int slot;            // position of the owning fragment in the id list
  int frag;            // fragment id
  int vec_ok;          // 1 if w_snap lanes are 16-byte aligned together with the native lanes
};

struct PlanHeader {
  int total_tiles;
  int n_seg;
  int n_ids;
  int pad;
};

// Status word helper: keep the first error recorded since the last poll.
__device__ __forceinline__ void record_status(int* status, int code) {
  atomicCAS(status, 0, code);
}

constexpr int kPlanThreads = 256;
constexpr int kMaxK = 1024;

// ids == nullptr means "all K fragments in index order" (stand-alone scoring).
static __global__ void __launch_bounds__(kPlanThreads)
k_plan(const int* __restrict__ ids, const int* __restrict__ n_ids_p, int K,
       const int* __restrict__ frag_seg_ptr, const long long* __restrict__ seg_off,
       const long long* __restrict__ seg_len, const long long* __restrict__ snap_offset,
       long long snap_row_len, int lanes_per_tile, int plan_capacity, SegPlan* __restrict__ plan,
       PlanHeader* __restrict__ hdr, int* __restrict__ status, int err_invalid) {
  // Three steps, so that the chains of dependent global loads (id -> segment range -> segment) run side by side
  // for all listed fragments instead of one fragment after the other: (1) every thread sizes its fragments,
  // (2) one thread turns the sizes into running segment and tile counts, (3) every thread writes its
  // fragments' table entries.
  __shared__ int seen[kMaxK];
  __shared__ int s_frag[kMaxK];            // fragment id of list position j
  __shared__ int s_seg_base[kMaxK];        // first table entry of position j (after step 2)
  __shared__ long long s_tiles[kMaxK];     // tiles of position j, then (after step 2) its first tile
  __shared__ int bad;
  const int tid = threadIdx.x;
  int n = (ids == nullptr) ? K : *n_ids_p;
  if (tid == 0) bad = (n < 0 || n > K) ? 1 : 0;
  for (int i = tid; i < K; i += blockDim.x) seen[i] = 0;
  __syncthreads();
  auto tiles_of = [&](long long off, long long len) -> long long {
    const long long lanes = (off - (off & ~3LL) + len + 3) >> 2;
    return (lanes + lanes_per_tile - 1) / lanes_per_tile;
  };
  if (!bad) {
    for (int j = tid; j < n; j += blockDim.x) {
      const int p = (ids == nullptr) ? j : ids[j];
      if (p < 0 || p >= K) { bad = 1; continue; }
      if (ids != nullptr && atomicAdd(&seen[p], 1) != 0) { bad = 1; continue; }
      if (snap_offset != nullptr && snap_offset[p] < 0) { bad = 1; continue; }   // no slot in the snapshot pool
      long long t = 0;
      for (int sg = frag_seg_ptr[p]; sg < frag_seg_ptr[p + 1]; ++sg) t += tiles_of(seg_off[sg], seg_len[sg]);
      s_frag[j] = p;
      s_seg_base[j] = frag_seg_ptr[p + 1] - frag_seg_ptr[p];
      s_tiles[j] = t;
    }
  }
  __syncthreads();
  if (tid == 0 && !bad) {
    long long tiles = 0;
    int ns = 0;
    for (int j = 0; j < n; ++j) {
      const int cnt = s_seg_base[j];
      const long long t = s_tiles[j];
      s_seg_base[j] = ns;
      s_tiles[j] = tiles;
      ns += cnt;
      tiles += t;
      if (ns > plan_capacity || tiles > 0x3fffffffLL) { bad = 1; break; }   // tile + gridDim.x must not wrap
    }
    if (!bad) {
      hdr->total_tiles = (int)tiles;
      hdr->n_seg = ns;
      hdr->n_ids = n;
      hdr->pad = 0;
    }
  }
  __syncthreads();
  if (!bad) {
    for (int j = tid; j < n; j += blockDim.x) {
      const int p = s_frag[j];
      int ns = s_seg_base[j];
      long long tiles = s_tiles[j];
      long long pos = 0;  // elements of the fragment placed so far (packed snapshot layout)
      for (int sg = frag_seg_ptr[p]; sg < frag_seg_ptr[p + 1]; ++sg) {
        SegPlan sp;
        sp.off = seg_off[sg];
        sp.len = seg_len[sg];
        sp.snap_off = (snap_offset != nullptr) ? snap_offset[p] + pos : sp.off;
        sp.abase = sp.off & ~3LL;
        sp.first_tile = (int)tiles;
        sp.slot = j;
        sp.frag = p;
        sp.vec_ok = (((sp.snap_off - sp.off) & 3LL) == 0) ? 1 : 0;
        // a packed snapshot must lie inside one row of the pool the caller described
        if (snap_offset != nullptr && sp.snap_off + sp.len > snap_row_len) bad = 1;
        plan[ns++] = sp;
        tiles += tiles_of(sp.off, sp.len);
        pos += sp.len;
      }
    }
  }
  __syncthreads();
  if (tid == 0 && bad) {
    hdr->total_tiles = 0; hdr->n_seg = 0; hdr->n_ids = 0; hdr->pad = 0;
    record_status(status, err_invalid);
  }
}

// ---------------------------------------------------------------------------
// Per-CTA accumulation of sums of squares, one slot per listed fragment.
//
// A persistent CTA walks its tiles in increasing order, so the fragment slot it
// works on never decreases.  Every thread keeps a double accumulator for the
// current slot; when the slot changes the warp reduces it and lane 0 writes
// partial[(slot*gridDim.x + blockIdx.x)*warps + warp] (warps = accumulating warps per CTA).  Slots a CTA never
// touched get an explicit zero, so the finalize kernel can sum every entry
// without the buffer being cleared first.  The tile-to-CTA map is static,
// hence the summation order - and the rounded result - is the same every run.
// ---------------------------------------------------------------------------
__device__ __forceinline__ double warp_sum(double v) {
#pragma unroll
  for (int o = 16; o > 0; o >>= 1) v += __shfl_xor_sync(0xffffffffu, v, o);
  return v;
}

struct SlotAccumulator {
  double acc = 0.0;
  int slot = 0;
  int warps;   // accumulating warps per CTA (warps 0 .. warps-1 must all call the methods below)

  __device__ __forceinline__ explicit SlotAccumulator(int accumulating_warps) : warps(accumulating_warps) {}

  __device__ __forceinline__ void flush_to(int new_slot, double* __restrict__ partial) {
    const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
    double v = warp_sum(acc);
    if (lane == 0) {
      partial[((size_t)slot * gridDim.x + blockIdx.x) * warps + warp] = v;
      for (int s = slot + 1; s < new_slot; ++s)
        partial[((size_t)s * gridDim.x + blockIdx.x) * warps + warp] = 0.0;
    }
    acc = 0.0;
    slot = new_slot;
  }
  __device__ __forceinline__ void advance(int new_slot, double* __restrict__ partial) {
    if (new_slot != slot) flush_to(new_slot, partial);
  }
  // after the last tile: write the current slot and zero the rest up to n_ids
  __device__ __forceinline__ void finish(int n_ids, double* __restrict__ partial) {
    if (slot < n_ids) flush_to(n_ids, partial);
  }
};

constexpr int kFinalizeThreads = 256;

// One block per listed fragment: sum its partials in a fixed order, take the
// square root, form the score of Eq. 10 and (for a completion) stamp last_sync.
//   mode 0: completion - I_p = max(1, t_p - last_sync[p]); last_sync[p] = t_l
//   mode 1: stand-alone scoring - I_p = max(1, interval[p]) or 1; last_sync untouched
static __global__ void __launch_bounds__(kFinalizeThreads)
k_finalize_scores(const PlanHeader* __restrict__ hdr, const int* __restrict__ ids,
                  const double* __restrict__ partial, int entries_per_slot,
                  int mode, long long t_p, long long t_l, const long long* __restrict__ t_p_dev,
                  const long long* __restrict__ t_l_dev, const long long* __restrict__ interval,
                  long long* __restrict__ last_sync, float* __restrict__ norms,
                  float* __restrict__ scores, int* __restrict__ status, int err_nonfinite) {
  __shared__ double red[kFinalizeThreads];
  const int j = blockIdx.x;
  if (j >= hdr->n_ids) return;
  const double* src = partial + (size_t)j * entries_per_slot;
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
  const int p = (ids == nullptr) ? j : ids[j];
  const double norm = sqrt(red[0]);
  long long I = 1;
  if (mode == 0) {
    // step numbers kept in device memory (graph replay) take precedence over the launch arguments
    if (t_p_dev) t_p = *t_p_dev;
    if (t_l_dev) t_l = *t_l_dev;
    I = t_p - last_sync[p];
    last_sync[p] = t_l;
  } else if (interval != nullptr) {
    I = interval[p];
  }
  if (I < 1) I = 1;
  norms[p] = (float)norm;
  scores[p] = (float)(norm / (double)I);
  if (!isfinite(norm)) record_status(status, err_nonfinite);
}

// ---------------------------------------------------------------------------
// Helpers of the host-buffer entry point, which streams a fragment through
// device staging in chunks: each chunk is a one-segment plan, and the chunk's
// sum of squares is added to its fragment's running total in chunk order.
// ---------------------------------------------------------------------------
static __global__ void k_plan_chunk(long long len, long long snap_off, int lanes_per_tile,
                             SegPlan* __restrict__ plan, PlanHeader* __restrict__ hdr) {
  SegPlan sp;
  sp.off = 0; sp.len = len; sp.snap_off = snap_off; sp.abase = 0;
  sp.first_tile = 0; sp.slot = 0; sp.frag = 0; sp.vec_ok = ((snap_off & 3LL) == 0) ? 1 : 0;
  plan[0] = sp;
  const long long lanes = (len + 3) >> 2;
  hdr->total_tiles = (int)((lanes + lanes_per_tile - 1) / lanes_per_tile);
  hdr->n_seg = 1; hdr->n_ids = 1; hdr->pad = 0;
}

static __global__ void __launch_bounds__(kFinalizeThreads)
k_accumulate_chunk(const double* __restrict__ partial, int entries, double* __restrict__ total) {
  __shared__ double red[kFinalizeThreads];
  double s = 0.0;
  for (int i = threadIdx.x; i < entries; i += kFinalizeThreads) s += partial[i];
  red[threadIdx.x] = s;
  __syncthreads();
#pragma unroll
  for (int w = kFinalizeThreads / 2; w > 0; w >>= 1) {
    if (threadIdx.x < w) red[threadIdx.x] += red[threadIdx.x + w];
    __syncthreads();
  }
  if (threadIdx.x == 0) *total += red[0];
}

static __global__ void k_finalize_from_sums(const double* __restrict__ sums, const int* __restrict__ ids, int n,
                                     long long t_p, long long t_l, long long* __restrict__ last_sync,
                                     float* __restrict__ norms, float* __restrict__ scores,
                                     int* __restrict__ status, int err_nonfinite) {
  for (int j = threadIdx.x; j < n; j += blockDim.x) {
    const int p = ids[j];
    const double norm = sqrt(sums[j]);
    long long I = t_p - last_sync[p];
    if (I < 1) I = 1;
    last_sync[p] = t_l;
    norms[p] = (float)norm;
    scores[p] = (float)(norm / (double)I);
    if (!isfinite(norm)) record_status(status, err_nonfinite);
  }
}

}  // namespace cocodc

// Launch plan: which tiles of which segments one call processes.
//
// A call works on a list of fragment ids that lives in device memory (it is
// usually written by the selection kernel, and the host never reads it).  The
// list is expanded into a table of segments with a running tile count, from
// which the streaming kernels map a tile index to (segment, lane range) without
// any host round-trip.  Two ways to get that table:
//   - fragment tables of up to kInlineSegs segments travel as a kernel argument
//     (FragTable) and every CTA of the streaming kernel expands the id list
//     itself, into shared memory, in its prologue (acquire_plan): one launch
//     per call, and the only dependent global loads are n_ids -> ids[j] ->
//     snap_offset[ids[j]];
//   - larger tables stay in device memory and a one-block kernel (k_plan)
//     writes the plan to global memory before the streaming kernel runs.
// The per-fragment norms and scores are likewise formed by the streaming kernel
// itself: the last warp to finish adds up the partial sums (finalize_epilogue).
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

// Fragment table small enough to be a kernel argument (CSR over segments, as cocodc_partition).
constexpr int kInlineSegs = 128;
struct FragTable {
  int K;
  int n_seg;
  int seg_ptr[kInlineSegs + 1];
  int pad;
  long long off[kInlineSegs];
  long long len[kInlineSegs];
};

// What a launch is to work on.
struct PlanRequest {
  const int* ids;                // device id list; nullptr: all K fragments in index order
  const int* n_ids;              // device, its length
  const long long* snap_offset;  // device [K] places in a packed snapshot pool, or nullptr
  long long snap_row_len;        // elements of one row of that pool
  int lanes_per_tile;
  int err_invalid;               // status code for a bad id list
};

// A completion whose scores are left to the next selection (COCODC_STAGE_DEFER): the launch ends with every CTA's
// sum of squares per list position in `partial` and this record in device memory; the launch that next decides
// which fragments to synchronise adds the CTAs' sums up in its prologue, where the boundary between the two
// launches has already done the grid-wide hand-off that the ticket counter otherwise provides.
constexpr int kMaxK = 1024;
struct PendingScores {
  int n;                         // list positions waiting; 0: nothing pending
  int grid, warps;               // shape of `partial` as the completion wrote it: [n][grid][warps], first entry per CTA
  int pad;
  long long t_p, t_l;            // step numbers of the completion
  int ids[kMaxK];                // fragment of list position j
};

// What the last warp of a launch does with the fragments' sums of squares (Eq. 10).
struct Finalize {
  int* ticket;                   // device counter, zero between launches; nullptr: no epilogue
  int mode;                      // 0 completion: I_p = t_p - last_sync[p], last_sync[p] = t_l; 1 stand-alone: I_p = interval[p] or 1
  int write_scores;              // 0: only sumsq_out is written
  const int* ids;                // the id list (nullptr: fragment j is list position j)
  long long t_p, t_l;
  const long long* t_p_dev;      // step numbers kept in device memory take precedence (graph replay)
  const long long* t_l_dev;
  const long long* interval;
  long long* last_sync;
  float* norms;
  float* scores;
  double* sumsq_out;             // [K] per-fragment sums of squares before the square root, or nullptr
  unsigned char* in_flight;      // [K] cleared for completed fragments, or nullptr
  int err_nonfinite;
  PendingScores* defer;          // non-null: stop after the CTAs' sums and leave this record (mode 0 only)
};

// Status word helper: keep the first error recorded since the last poll.
__device__ __forceinline__ void record_status(int* status, int code) {
  atomicCAS(status, 0, code);
}

constexpr int kPlanThreads = 256;

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
// touched get an explicit zero, so the score epilogue can sum every entry
// without the buffer being cleared first.  The tile-to-CTA map is static,
// hence the summation order - and the rounded result - is the same every run.
// ---------------------------------------------------------------------------
__device__ __forceinline__ double warp_sum(double v) {
#pragma unroll
  for (int o = 16; o > 0; o >>= 1) v += __shfl_xor_sync(0xffffffffu, v, o);
  return v;
}

// Arrival counters of the epilogues.  An acq_rel read-modify-write orders the arriving thread's earlier writes
// (and, through the warp or CTA barrier before it, those of the threads it speaks for) before the count, and
// the count before the reads of whoever arrives last; this is cheaper than a sequentially consistent fence
// (what __threadfence() compiles to) on each side of a relaxed atomic.
__device__ __forceinline__ int arrive_cta(int* shared_counter) {
  int old;
  asm volatile("atom.acq_rel.gpu.shared::cta.add.u32 %0, [%1], 1;"
               : "=r"(old) : "r"((unsigned)__cvta_generic_to_shared(shared_counter)) : "memory");
  return old;
}
// the same when both the data and its readers stay inside the CTA (shared memory)
__device__ __forceinline__ int arrive_cta_local(int* shared_counter) {
  int old;
  asm volatile("atom.acq_rel.cta.shared::cta.add.u32 %0, [%1], 1;"
               : "=r"(old) : "r"((unsigned)__cvta_generic_to_shared(shared_counter)) : "memory");
  return old;
}
__device__ __forceinline__ int arrive_gpu(int* global_counter) {
  int old;
  asm volatile("atom.acq_rel.gpu.global.add.u32 %0, [%1], 1;" : "=r"(old) : "l"(global_counter) : "memory");
  return old;
}

constexpr int kFastSlots = 32;   // id lists up to this long keep the per-warp sums of a CTA in shared memory

struct SlotAccumulator {
  double acc = 0.0;
  int slot = 0;
  int warps;   // accumulating warps per CTA (warps 0 .. warps-1 must all call the methods below)
  double* cta_part = nullptr;   // shared [kFastSlots][warps]: the warps' sums stay in the CTA (the score epilogue
                                // adds them there and writes one entry per slot); nullptr: one global entry per warp

  __device__ __forceinline__ explicit SlotAccumulator(int accumulating_warps) : warps(accumulating_warps) {}

  __device__ __forceinline__ void flush_to(int new_slot, double* __restrict__ partial) {
    const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
    double v = warp_sum(acc);
    if (lane == 0) {
      if (cta_part != nullptr) {
        cta_part[slot * warps + warp] = v;
        for (int s = slot + 1; s < new_slot; ++s) cta_part[s * warps + warp] = 0.0;
      } else {
        partial[((size_t)slot * gridDim.x + blockIdx.x) * warps + warp] = v;
        for (int s = slot + 1; s < new_slot; ++s)
          partial[((size_t)s * gridDim.x + blockIdx.x) * warps + warp] = 0.0;
      }
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

// ---------------------------------------------------------------------------
// The plan in shared memory, built by every CTA in its prologue.
// ---------------------------------------------------------------------------
struct InlinePlan {
  SegPlan seg[kInlineSegs];
  PlanHeader hdr;
  long long tiles[kInlineSegs];   // tiles of list position j, then its first tile
  int frag[kInlineSegs];          // fragment id of list position j
  int cnt[kInlineSegs];           // segments of position j, then its first table entry
  int seen[kInlineSegs];
  long long place[kInlineSegs];   // pool place of every fragment (fetched beside the id list, not after it)
  double warp_part[kFastSlots * 8];   // per-warp sums of squares of short id lists (SlotAccumulator::cta_part)
  int bad;
  int done_warps;                 // accumulating warps of this CTA that have written their partial sums
};

struct PlanView {
  const SegPlan* seg;
  PlanHeader hdr;
};

__device__ __forceinline__ long long tiles_of_segment(long long off, long long len, int lanes_per_tile) {
  const long long lanes = (off - (off & ~3LL) + len + 3) >> 2;
  return (lanes + lanes_per_tile - 1) / lanes_per_tile;
}

// Called by EVERY thread of the CTA before the roles split.  (Out of line, like the epilogue: prologue and
// epilogue run once per CTA, and the streaming loops between them are sensitive to what is compiled around them.)  With a plan in global memory (gplan != nullptr,
// written by k_plan or k_plan_chunk earlier on the stream) it only returns that; otherwise the CTA expands the
// id list itself.  Every CTA reaches the same verdict on a bad list (an id out of range or listed twice, a
// listed fragment without a place in the pool or not inside one row of it): nothing is processed and CTA 0
// records the error.
static __device__ __noinline__ PlanView acquire_plan(InlinePlan& ip, const FragTable& T, const PlanRequest& rq,
                                                 const SegPlan* gplan, const PlanHeader* ghdr, int* status) {
  const int tid = threadIdx.x, nt = blockDim.x;
  PlanView pv;
  if (gplan != nullptr) {
    if (tid == 0) ip.done_warps = 0;
    __syncthreads();
    pv.seg = gplan;
    pv.hdr = *ghdr;
    return pv;
  }
  const int K = T.K;
  // the pool places of all K fragments are fetched alongside the list length and the ids, so that the chain of
  // dependent global loads is two long, not three
  for (int i = tid; i < K; i += nt) {
    ip.seen[i] = 0;
    ip.place[i] = (rq.snap_offset != nullptr) ? rq.snap_offset[i] : 0;
  }
  int n = (rq.ids == nullptr) ? K : *rq.n_ids;
  if (tid == 0) { ip.bad = (n < 0 || n > K) ? 1 : 0; ip.done_warps = 0; }
  __syncthreads();
  if (n < 0 || n > K) n = 0;
  const int lpt = rq.lanes_per_tile;
  for (int j = tid; j < n; j += nt) {
    const int p = (rq.ids == nullptr) ? j : rq.ids[j];
    bool ok = (p >= 0 && p < K);
    if (ok && rq.ids != nullptr && atomicAdd(&ip.seen[p], 1) != 0) ok = false;
    if (ok && rq.snap_offset != nullptr && ip.place[p] < 0) ok = false;   // no place in the snapshot pool
    long long t = 0;
    int c = 0;
    if (ok) {
      for (int sg = T.seg_ptr[p]; sg < T.seg_ptr[p + 1]; ++sg) t += tiles_of_segment(T.off[sg], T.len[sg], lpt);
      c = T.seg_ptr[p + 1] - T.seg_ptr[p];
    } else {
      ip.bad = 1;
    }
    ip.frag[j] = ok ? p : 0;
    ip.cnt[j] = c;
    ip.tiles[j] = t;
  }
  __syncthreads();
  // running segment and tile counts over the list: warp 0, four positions per lane
  if (tid < 32) {
    int c[4];
    long long tl[4];
    int csum = 0;
    long long tsum = 0;
#pragma unroll
    for (int q = 0; q < 4; ++q) {
      const int j = 4 * tid + q;
      c[q] = (j < n) ? ip.cnt[j] : 0;
      tl[q] = (j < n) ? ip.tiles[j] : 0;
      csum += c[q];
      tsum += tl[q];
    }
    int cinc = csum;
    long long tinc = tsum;
#pragma unroll
    for (int o = 1; o < 32; o <<= 1) {
      const int cv = __shfl_up_sync(0xffffffffu, cinc, o);
      const long long tv = __shfl_up_sync(0xffffffffu, tinc, o);
      if (tid >= o) { cinc += cv; tinc += tv; }
    }
    int cbase = cinc - csum;
    long long tbase = tinc - tsum;
#pragma unroll
    for (int q = 0; q < 4; ++q) {
      const int j = 4 * tid + q;
      if (j < n) { ip.cnt[j] = cbase; ip.tiles[j] = tbase; }
      cbase += c[q];
      tbase += tl[q];
    }
    if (tid == 31) {
      if (cinc > kInlineSegs || tinc > 0x3fffffffLL) ip.bad = 1;   // tile + gridDim.x must not wrap
      ip.hdr.total_tiles = (int)tinc;
      ip.hdr.n_seg = cinc;
      ip.hdr.n_ids = n;
      ip.hdr.pad = 0;
    }
  }
  __syncthreads();
  if (!ip.bad) {
    for (int j = tid; j < n; j += nt) {
      const int p = ip.frag[j];
      int ns = ip.cnt[j];
      long long tiles = ip.tiles[j];
      long long pos = 0;   // elements of the fragment placed so far (packed snapshot layout)
      for (int sg = T.seg_ptr[p]; sg < T.seg_ptr[p + 1]; ++sg) {
        SegPlan sp;
        sp.off = T.off[sg];
        sp.len = T.len[sg];
        sp.snap_off = (rq.snap_offset != nullptr) ? ip.place[p] + pos : sp.off;
        sp.abase = sp.off & ~3LL;
        sp.first_tile = (int)tiles;
        sp.slot = j;
        sp.frag = p;
        sp.vec_ok = (((sp.snap_off - sp.off) & 3LL) == 0) ? 1 : 0;
        // a packed snapshot must lie inside one row of the pool the caller described
        if (rq.snap_offset != nullptr && sp.snap_off + sp.len > rq.snap_row_len) ip.bad = 1;
        ip.seg[ns++] = sp;
        tiles += tiles_of_segment(sp.off, sp.len, lpt);
        pos += sp.len;
      }
    }
  }
  __syncthreads();
  pv.seg = ip.seg;
  if (ip.bad) {
    pv.hdr.total_tiles = 0; pv.hdr.n_seg = 0; pv.hdr.n_ids = 0; pv.hdr.pad = 0;
    if (tid == 0 && blockIdx.x == 0) record_status(status, rq.err_invalid);
  } else {
    pv.hdr = ip.hdr;
  }
  return pv;
}

// ---------------------------------------------------------------------------
// Norms and scores from the partial sums, inside the launch that produced them.
//
// Called by every accumulating warp (all 32 lanes) after SlotAccumulator::finish.  The last warp of a CTA to
// arrive adds that CTA's per-warp sums, slot by slot, into the CTA's first global entry of the slot (the
// per-warp sums come from shared memory when the id list has at most kFastSlots fragments - in_shared - and from
// the warps' global entries otherwise; the order of the additions is the same); the last CTA of the launch to
// get there (a ticket counter in global memory) adds the CTAs' entries of every slot in a fixed order, takes
// the square root, forms Eq. 10's score and stamps last_sync.  Which warp does the adding varies from run to
// run, the order of the additions does not, so the rounded result is the same every run.  The ticket counter
// is left at zero for the next launch.  A warp that gave up on a bounded wait never arrives: the launch then
// writes no norms (the status word says why) and the counter is reset by the next status poll.
// ---------------------------------------------------------------------------

__device__ __forceinline__ void write_fragment_score(const Finalize& F, int p, long long last, double total,
                                                     long long t_p, long long t_l, int* status);

// Deferred completion: CTA 0 leaves the record from which the next selection forms the scores (called by one warp).
__device__ __forceinline__ void leave_pending_record(const Finalize& F, const PlanHeader& h, int warps) {
  const int lane = threadIdx.x & 31;
  PendingScores* P = F.defer;
  for (int j = lane; j < h.n_ids; j += 32) P->ids[j] = (F.ids == nullptr) ? j : F.ids[j];
  if (lane == 0) {
    P->t_p = F.t_p_dev ? *F.t_p_dev : F.t_p;
    P->t_l = F.t_l_dev ? *F.t_l_dev : F.t_l;
    P->grid = (int)gridDim.x;
    P->warps = warps;
    P->n = h.n_ids;
  }
}

// Sum over the CTAs' entries of list position j, by one warp: lane l adds the entries of CTAs l, l + 32, ... in that
// order, then the lanes' sums meet in the shuffle tree - the order finalize_epilogue uses, hence the same bits.
__device__ __forceinline__ double pending_slot_total(const double* __restrict__ partial, int j, int grid, int warps) {
  const int lane = threadIdx.x & 31;
  double s = 0.0;
  for (int i0 = lane; i0 < grid; i0 += 32 * 8) {
    double x[8];
#pragma unroll
    for (int r = 0; r < 8; ++r) {
      const int i = i0 + 32 * r;
      x[r] = (i < grid) ? __ldcg(partial + ((size_t)j * grid + i) * warps) : 0.0;
    }
#pragma unroll
    for (int r = 0; r < 8; ++r) if (i0 + 32 * r < grid) s += x[r];
  }
  return warp_sum(s);
}

static __device__ __noinline__ void finalize_epilogue(InlinePlan& ip, const Finalize& F, const PlanHeader& h,
                                                  double* __restrict__ partial, int warps, int* status,
                                                  bool in_shared = false) {
  if (F.ticket == nullptr) return;
  const int lane = threadIdx.x & 31;
  const int grid = gridDim.x, cta = blockIdx.x;
  int t = 0;
  __syncwarp();
  if (lane == 0) t = in_shared ? arrive_cta_local(&ip.done_warps) : arrive_cta(&ip.done_warps);
  t = __shfl_sync(0xffffffffu, t, 0);
  if (t != warps - 1) return;
  // (loads first, additions after: the additions keep their order, the loads overlap)
  for (int j = lane; j < h.n_ids; j += 32) {
    double* e = partial + ((size_t)j * grid + cta) * warps;
    double v = 0.0;
    if (in_shared) {
      for (int w = 0; w < warps; ++w) v += ip.warp_part[j * warps + w];
    } else {
      for (int w0 = 0; w0 < warps; w0 += 8) {
        double x[8];
#pragma unroll
        for (int q = 0; q < 8; ++q) x[q] = (w0 + q < warps) ? __ldcg(e + w0 + q) : 0.0;
#pragma unroll
        for (int q = 0; q < 8; ++q) if (w0 + q < warps) v += x[q];
      }
    }
    __stcg(e, v);
  }
  __syncwarp();
  if (F.defer) {                 // the next selection adds the CTAs' entries up
    if (cta == 0) leave_pending_record(F, h, warps);
    return;
  }
  if (lane == 0) t = arrive_gpu(F.ticket);
  t = __shfl_sync(0xffffffffu, t, 0);
  if (t != grid - 1) return;
  long long t_p = F.t_p, t_l = F.t_l;
  if (F.t_p_dev) t_p = *F.t_p_dev;
  if (F.t_l_dev) t_l = *F.t_l_dev;
  // Four slots at a time, so that their loads are in flight together.  Per slot: lane l adds the entries of
  // CTAs l, l + 32, ... in that order, then the lanes' sums meet in the shuffle tree.  The fragment ids and their
  // last_sync entries are fetched by lanes 0-3 beside those loads, not after the sums.
  constexpr int kBatch = 4, kPerLane = 5;       // 32 * 5 = 160 entries per pass: one pass for a grid of 148
  for (int j0 = 0; j0 < h.n_ids; j0 += kBatch) {
    int my_p = 0;
    long long my_last = 0;
    if (lane < kBatch && j0 + lane < h.n_ids) {
      my_p = (F.ids == nullptr) ? j0 + lane : F.ids[j0 + lane];
      if (F.write_scores && F.mode == 0) my_last = F.last_sync[my_p];
    }
    double s[kBatch];
#pragma unroll
    for (int q = 0; q < kBatch; ++q) s[q] = 0.0;
    for (int i0 = lane; i0 < grid; i0 += 32 * kPerLane) {
      double x[kBatch][kPerLane];
#pragma unroll
      for (int q = 0; q < kBatch; ++q)
#pragma unroll
        for (int r = 0; r < kPerLane; ++r) {
          const int i = i0 + 32 * r;
          x[q][r] = (j0 + q < h.n_ids && i < grid) ? __ldcg(partial + ((size_t)(j0 + q) * grid + i) * warps) : 0.0;
        }
#pragma unroll
      for (int q = 0; q < kBatch; ++q)
#pragma unroll
        for (int r = 0; r < kPerLane; ++r)
          if (j0 + q < h.n_ids && i0 + 32 * r < grid) s[q] += x[q][r];
    }
#pragma unroll
    for (int q = 0; q < kBatch; ++q) {
      const int j = j0 + q;
      if (j >= h.n_ids) break;
      const double total = warp_sum(s[q]);
      const int p = __shfl_sync(0xffffffffu, my_p, q);
      const long long last = __shfl_sync(0xffffffffu, my_last, q);
      if (lane == 0) write_fragment_score(F, p, last, total, t_p, t_l, status);
    }
  }
  __syncwarp();
  if (lane == 0) *F.ticket = 0;
}

// Last steps of Eq. 10 for fragment p (last = last_sync[p] as read before), by lane 0 of the warp that holds
// the fragment's total.
__device__ __forceinline__ void write_fragment_score(const Finalize& F, int p, long long last, double total,
                                                     long long t_p, long long t_l, int* status) {
  if (F.sumsq_out) F.sumsq_out[p] = total;
  if (!F.write_scores) return;
  const double norm = sqrt(total);
  long long I = 1;
  if (F.mode == 0) {
    I = t_p - last;
    F.last_sync[p] = t_l;
    if (F.in_flight) F.in_flight[p] = 0;
  } else if (F.interval != nullptr) {
    I = F.interval[p];
  }
  if (I < 1) I = 1;
  F.norms[p] = (float)norm;
  F.scores[p] = (float)(norm / (double)I);
  if (!isfinite(norm)) record_status(status, F.err_nonfinite);
}

// The same epilogue for kernels in which every thread of the CTA is an accumulating thread that reaches the
// end of the kernel (no producer warps, no abandoned waits), so the CTA can meet at a barrier: the CTA's
// entries are added by its threads side by side, and in the last CTA of the launch every warp takes slots.
// The order of the additions is the one finalize_epilogue uses, hence the same bits.
static __device__ __noinline__ void finalize_epilogue_cta(InlinePlan& ip, const Finalize& F, const PlanHeader& h,
                                                      double* __restrict__ partial, int warps, int* status) {
  if (F.ticket == nullptr) return;
  const int tid = threadIdx.x, lane = tid & 31, warp = tid >> 5;
  const int grid = gridDim.x, cta = blockIdx.x;
  __syncthreads();     // every warp's entries are written
  for (int j = tid; j < h.n_ids; j += blockDim.x) {
    double* e = partial + ((size_t)j * grid + cta) * warps;
    double v = 0.0;
    for (int w0 = 0; w0 < warps; w0 += 8) {
      double x[8];
#pragma unroll
      for (int q = 0; q < 8; ++q) x[q] = (w0 + q < warps) ? __ldcg(e + w0 + q) : 0.0;
#pragma unroll
      for (int q = 0; q < 8; ++q) if (w0 + q < warps) v += x[q];
    }
    __stcg(e, v);
  }
  if (F.defer) {
    if (cta == 0 && warp == 0) leave_pending_record(F, h, warps);
    return;
  }
  __syncthreads();
  if (tid == 0) ip.done_warps = (arrive_gpu(F.ticket) == grid - 1) ? 1 : 0;
  __syncthreads();
  if (!ip.done_warps) return;
  long long t_p = F.t_p, t_l = F.t_l;
  if (F.t_p_dev) t_p = *F.t_p_dev;
  if (F.t_l_dev) t_l = *F.t_l_dev;
  for (int j = warp; j < h.n_ids; j += warps) {
    double s = 0.0;
    for (int i0 = lane; i0 < grid; i0 += 32 * 8) {
      double x[8];
#pragma unroll
      for (int r = 0; r < 8; ++r) {
        const int i = i0 + 32 * r;
        x[r] = (i < grid) ? __ldcg(partial + ((size_t)j * grid + i) * warps) : 0.0;
      }
#pragma unroll
      for (int r = 0; r < 8; ++r) if (i0 + 32 * r < grid) s += x[r];
    }
    const double total = warp_sum(s);
    if (lane == 0) {
      const int p = (F.ids == nullptr) ? j : F.ids[j];
      const long long last = (F.write_scores && F.mode == 0) ? F.last_sync[p] : 0;
      write_fragment_score(F, p, last, total, t_p, t_l, status);
    }
  }
  if (tid == 0) *F.ticket = 0;
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

// Eq. 10 from per-fragment sums of squares that already exist (added up chunk by chunk by the host-buffer entry
// point, or all-reduced over the devices that each hold a slice of every fragment).
//   completion (interval_mode == 0): fragments ids[0 .. n), sums indexed as `by_position` says,
//       I_p = max(1, t_p - last_sync[p]), last_sync[p] = t_l, in_flight[p] = 0
//   stand-alone (interval_mode == 1): all K fragments, I_p = max(1, interval[p]) (1 without intervals)
static __global__ void k_scores_from_sumsq(const double* __restrict__ sums, int by_position, const int* __restrict__ ids,
                                    const int* __restrict__ n_ids_dev, int n_host, int K, int interval_mode,
                                    const long long* __restrict__ interval, long long t_p, long long t_l,
                                    long long* __restrict__ last_sync, float* __restrict__ norms,
                                    float* __restrict__ scores, unsigned char* __restrict__ in_flight,
                                    int* __restrict__ status, int err_nonfinite, int err_invalid) {
  int n = interval_mode ? K : (n_ids_dev ? *n_ids_dev : n_host);
  if (n < 0 || n > K) {
    if (threadIdx.x == 0) record_status(status, err_invalid);
    return;
  }
  for (int j = threadIdx.x; j < n; j += blockDim.x) {
    const int p = interval_mode ? j : ids[j];
    if (p < 0 || p >= K) { record_status(status, err_invalid); continue; }
    const double norm = sqrt(sums[by_position ? j : p]);
    long long I = 1;
    if (interval_mode) {
      if (interval != nullptr) I = interval[p];
    } else {
      I = t_p - last_sync[p];
      last_sync[p] = t_l;
      if (in_flight) in_flight[p] = 0;
    }
    if (I < 1) I = 1;
    norms[p] = (float)norm;
    scores[p] = (float)(norm / (double)I);
    if (!isfinite(norm)) record_status(status, err_nonfinite);
  }
}

}  // namespace cocodc

// Fragment selection on the device (Algorithm 2 and Eq. 11, walked under a budget).
//
// K is at most 1024, so one block does it: every thread ranks one fragment by
// counting the fragments that precede it in the priority order, the order is
// scattered into shared memory, and one thread walks it with the budget.  The
// result stays on the device, where the next launch reads it.
#pragma once

#include "plan.cuh"

namespace cocodc {

constexpr int kSelectThreads = 1024;
constexpr int kExactMaxFree = 24;    // knapsack candidates enumerated at most (2^24 subsets)

__global__ void __launch_bounds__(kSelectThreads)
k_select(int K, const float* __restrict__ scores, const long long* __restrict__ last_sync,
         const unsigned char* __restrict__ ineligible, const long long* __restrict__ frag_size,
         const long long* __restrict__ frag_first_off,
         long long t_now, const long long* __restrict__ t_now_dev, long long H, int budget_kind, long long budget,
         unsigned char* __restrict__ mask, int* __restrict__ ids, int* __restrict__ n_sel,
         long long* __restrict__ pool_offset, unsigned char* __restrict__ in_flight,
         int* __restrict__ status, int err_nonfinite, int err_too_many) {
  __shared__ float s_score[kMaxK];
  __shared__ unsigned char s_class[kMaxK];  // 0 = ineligible, 1 = ordinary, 2 = overdue
  __shared__ int s_order[kMaxK];
  __shared__ long long s_fsize[kMaxK];      // fragment sizes, so that the walk below reads no global memory
  __shared__ unsigned char s_falign[kMaxK]; // native offset of the fragment's first segment, mod 4 (see place())
  __shared__ int s_nan;
  __shared__ int s_count;
  const int p = threadIdx.x;
  if (t_now_dev) t_now = *t_now_dev;   // step number kept in device memory (graph replay)
  if (p == 0) { s_nan = 0; s_count = 0; }
  __syncthreads();
  if (p < K) {
    const float r = scores[p];
    // a fragment whose synchronisation is in flight cannot be chosen again before it completes
    const bool elig = ((ineligible == nullptr) || (ineligible[p] == 0)) &&
                      ((in_flight == nullptr) || (in_flight[p] == 0));
    const bool overdue = (t_now - last_sync[p]) >= H;   // Algorithm 2's staleness test
    s_score[p] = r;
    s_fsize[p] = frag_size[p];
    s_falign[p] = (unsigned char)(frag_first_off[p] & 3);
    s_class[p] = elig ? (overdue ? 2 : 1) : 0;
    if (r != r) s_nan = 1;
    mask[p] = 0;
    ids[p] = -1;
    if (pool_offset) pool_offset[p] = -1;
  }
  __syncthreads();
  if (s_nan) {
    if (p == 0) { *n_sel = 0; record_status(status, err_nonfinite); }
    return;
  }
  if (p < K && s_class[p] != 0) {
    const float r = s_score[p];
    const int cls = s_class[p];
    int rank = 0;
    for (int q = 0; q < K; ++q) {
      const int cq = s_class[q];
      if (cq == 0 || q == p) continue;
      bool before;
      if (cq != cls) before = cq > cls;                 // overdue fragments come first
      else if (cls == 2) before = q < p;                // among overdue: by index
      else {
        const float rq = s_score[q];
        before = (rq > r) || (rq == r && q < p);        // by score, ties to the lower index
      }
      rank += before ? 1 : 0;
    }
    s_order[rank] = p;
    atomicAdd(&s_count, 1);
  }
  __syncthreads();
  // ---- the walk under the budget ---------------------------------------------------------------
  // COUNT and PARAMS budgets: thread 0 walks the whole order.  EXACT (not in the paper): it walks only the
  // fragments that must go first -- the overdue ones and those never synchronised (score +inf) -- and the
  // rest of the order becomes a knapsack that all threads solve by enumeration below.
  __shared__ long long s_remaining;
  __shared__ long long s_pool_pos;   // next free element of the snapshot pool (kept a multiple of 4)
  // A fragment's place in the pool starts at the next multiple of 4 plus its native offset mod 4: recorded and
  // native values then share their 16-byte alignment, and the streaming kernels can move the fragment as
  // vectors staged by bulk copies (a place that breaks the congruence leaves only 4-byte accesses for the
  // recorded values, at half to two thirds of the bandwidth).
  auto place = [&](int f, long long& pool_pos) {
    const long long start = pool_pos + s_falign[f];
    pool_offset[f] = start;
    pool_pos = (start + s_fsize[f] + 3) & ~3LL;
  };
  __shared__ int s_n;                // fragments admitted so far
  __shared__ int s_free_begin;       // first position of the order that belongs to the knapsack
  const int n_elig = s_count;
  const bool exact = (budget_kind == 2);
  if (p == 0) {
    long long remaining = budget, pool_pos = 0;
    int n = 0, j = 0;
    for (; j < n_elig; ++j) {
      const int f = s_order[j];
      if (exact && s_class[f] != 2 && s_score[f] != INFINITY) break;
      const long long cost = (budget_kind == 0) ? 1 : s_fsize[f];
      if (j == 0 || cost <= remaining) {   // the head of the order is always taken
        mask[f] = 1;
        if (in_flight) in_flight[f] = 1;
        ids[n++] = f;
        remaining -= cost;
        if (pool_offset) place(f, pool_pos);
      }
    }
    s_remaining = remaining; s_pool_pos = pool_pos; s_n = n; s_free_begin = j;
  }
  __syncthreads();
  const int n_free = n_elig - s_free_begin;
  if (!exact || n_free == 0) {
    if (p == 0) *n_sel = s_n;
    return;
  }
  if (n_free > kExactMaxFree) {      // too many candidates to enumerate: report it, select nothing
    if (p < K) {
      if (in_flight && mask[p]) in_flight[p] = 0;   // taken back: marked by the walk above in this call
      mask[p] = 0; ids[p] = -1; if (pool_offset) pool_offset[p] = -1;
    }
    if (p == 0) { *n_sel = 0; record_status(status, err_too_many); }
    return;
  }
  // ---- knapsack over the remaining order by enumeration ------------------------------------------
  // Subset m has bit j set when the j-th remaining fragment (in priority order) is in it.  Its value is the
  // sum of the scores, added in double in that order; the best feasible subset wins, equal values go to
  // the smaller m (which prefers fragments earlier in the order).
  __shared__ double s_val[kExactMaxFree];
  __shared__ long long s_size[kExactMaxFree];
  __shared__ double s_best_val[kSelectThreads];
  __shared__ unsigned s_best_mask[kSelectThreads];
  if (p < n_free) {
    const int f = s_order[s_free_begin + p];
    s_val[p] = (double)s_score[f];
    s_size[p] = s_fsize[f];
  }
  __syncthreads();
  const long long room = s_remaining;
  double best_val = -1.0;            // below every feasible value only when scores are non-negative ...
  unsigned best_mask = 0xffffffffu;  // ... so feasibility is tracked by the mask: all ones = none found
  const unsigned total = 1u << n_free;
  for (unsigned m = p; m < total; m += kSelectThreads) {
    long long size = 0;
    double val = 0.0;
    for (int j = 0; j < n_free; ++j)
      if ((m >> j) & 1u) { size += s_size[j]; val += s_val[j]; }
    if (size <= room && (best_mask == 0xffffffffu || val > best_val)) { best_val = val; best_mask = m; }
  }
  s_best_val[p] = best_val;
  s_best_mask[p] = best_mask;
  __syncthreads();
  for (int w = kSelectThreads / 2; w > 0; w >>= 1) {
    if (p < w) {
      const double v = s_best_val[p + w];
      const unsigned m = s_best_mask[p + w];
      const unsigned mine = s_best_mask[p];
      if (m != 0xffffffffu && (mine == 0xffffffffu || v > s_best_val[p] || (v == s_best_val[p] && m < mine))) {
        s_best_val[p] = v;
        s_best_mask[p] = m;
      }
    }
    __syncthreads();
  }
  if (p != 0) return;
  unsigned chosen = s_best_mask[0];
  if (chosen == 0xffffffffu) chosen = 0;             // nothing fits (the budget is already overdrawn)
  if (chosen == 0 && s_n == 0) chosen = 1;           // a decision always returns a fragment (Algorithm 2)
  int n = s_n;
  long long pool_pos = s_pool_pos;
  for (int j = 0; j < n_free; ++j) {
    if (!((chosen >> j) & 1u)) continue;
    const int f = s_order[s_free_begin + j];
    mask[f] = 1;
    if (in_flight) in_flight[f] = 1;
    ids[n++] = f;
    if (pool_offset) place(f, pool_pos);
  }
  *n_sel = n;
}

// ---------------------------------------------------------------------------------------------------
// The same decision inside another kernel's prologue (cocodc_initiate: Algorithm 2 and the snapshot of what it
// picks are one event, at t_p, so they are one launch).  For fragment tables that travel as a kernel argument
// (K <= kInlineSegs) and the budgets that are walked (COUNT, PARAMS), every CTA of the snapshot kernel works out
// the selection for itself - it is a deterministic function of the schedule state - and keeps the id list and
// the pool places in shared memory, where the plan is then built from; CTA 0 also writes them to the caller's
// arrays.  The in-flight marks are written by whichever CTA finishes its selection last (a ticket, select_commit):
// no CTA may see them before it has read the mask itself.
// ---------------------------------------------------------------------------------------------------
struct SelectRequest {
  const float* scores;                 // nullptr: no selection in this launch
  const long long* last_sync;
  const unsigned char* ineligible;
  unsigned char* in_flight;
  long long t_now;
  const long long* t_now_dev;          // the step number kept in device memory takes precedence (graph replay)
  long long H;
  int budget_kind;                     // 0 COUNT, 1 PARAMS
  long long budget;
  unsigned char* mask;
  int* ids;
  int* n_sel;
  long long* pool_offset;              // nullptr: the snapshot keeps the native layout
  int* ticket;                         // zero between launches
  int err_nonfinite;
  // A completion whose scores were left to this selection (PendingScores): the record, the CTAs' sums it describes,
  // and the arrays the completion was given (scores and last_sync above are the same arrays, read-only there).
  PendingScores* pending;              // nullptr: nothing can be pending
  const double* partial;
  int pend_grid, pend_warps;           // shape of `partial` as the host remembers it (the record has the last word)
  float* norms;
  float* scores_out;
  long long* last_sync_out;
};

struct InlineSelect {
  float score[kInlineSegs];
  int order[kInlineSegs];
  int ids[kInlineSegs];
  long long fsize[kInlineSegs];
  long long pool[kInlineSegs];         // by fragment id; -1: not selected
  unsigned char cls[kInlineSegs];      // 0 = ineligible, 1 = ordinary, 2 = overdue
  unsigned char falign[kInlineSegs];
  long long last[kInlineSegs];         // last_sync as this selection sees it (pending completions applied)
  unsigned char infl[kInlineSegs];     // the in-flight marks likewise
  int pend_id[kInlineSegs];            // pending list position -> fragment
  float pend_norm[kInlineSegs];
  int n;
  int n_elig;
  int nan;
  int bad_norm;
  int n_pend;
};

// Eq. 10 for the fragments of a pending completion, into the selection's shared-memory view of the schedule state.
// One warp per list position adds the CTAs' sums; the arithmetic after the sum is write_fragment_score's.  The
// loads are issued in two parts so that they cost no round trip of their own: fetch() runs before the barrier at
// which the schedule arrays arrive and already adds up list position `warp` with the shape the host remembers of
// the completion's launch; apply() runs after it, uses that sum when the record confirms the shape, and takes any
// further positions (lists longer than the CTA has warps) with plain loads.
struct PendingFetch {
  int n, grid, warps, frag;      // the record's fields; frag = ids[warp]
  long long t_p, t_l;
  double total;                  // sum of list position `warp`, formed with the host's shape
};

__device__ __forceinline__ PendingFetch fetch_pending_scores(const PendingScores* P, const double* __restrict__ partial,
                                                             int K, int host_grid, int host_warps) {
  PendingFetch f{};
  if (P == nullptr) return f;
  const int warp = threadIdx.x >> 5;
  f.n = P->n; f.grid = P->grid; f.warps = P->warps; f.t_p = P->t_p; f.t_l = P->t_l;
  if (warp < K) {
    f.frag = P->ids[warp];
    f.total = pending_slot_total(partial, warp, host_grid, host_warps);
  }
  if (f.n < 0 || f.n > K) f.n = 0;   // (cannot happen: the completion's list was validated)
  return f;
}

__device__ __forceinline__ void apply_pending_scores(const PendingFetch& pf, const PendingScores* P,
                                                     const double* __restrict__ partial, int host_grid, int host_warps,
                                                     float* score, long long* last, unsigned char* infl,
                                                     int* pend_id, float* pend_norm, int* bad_norm) {
  const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31, nw = blockDim.x >> 5;
  const bool shape_ok = (pf.grid == host_grid && pf.warps == host_warps);
  for (int j = warp; j < pf.n; j += nw) {
    const bool fetched = (j == warp) && shape_ok;
    const int f = fetched ? pf.frag : P->ids[j];
    const double total = fetched ? pf.total : pending_slot_total(partial, j, pf.grid, pf.warps);
    if (lane == 0) {
      const double norm = sqrt(total);
      long long I = pf.t_p - last[f];
      if (I < 1) I = 1;
      pend_id[j] = f;
      pend_norm[j] = (float)norm;
      score[f] = (float)(norm / (double)I);
      last[f] = pf.t_l;
      infl[f] = 0;
      if (!isfinite(norm)) *bad_norm = 1;
    }
  }
}

// Called by every thread of the CTA (at least K threads).
static __device__ __noinline__ void select_in_cta(InlineSelect& is, const SelectRequest& q, const FragTable& T,
                                                  int* status) {
  const int p = threadIdx.x;
  const int K = T.K;
  const bool writer = (blockIdx.x == 0);
  const long long t_now = q.t_now_dev ? *q.t_now_dev : q.t_now;
  if (p == 0) { is.n = 0; is.n_elig = 0; is.nan = 0; is.bad_norm = 0; }
  if (p < K) {
    is.score[p] = q.scores[p];
    is.last[p] = q.last_sync[p];
    is.infl[p] = (q.in_flight != nullptr) ? q.in_flight[p] : (unsigned char)0;
  }
  const PendingFetch pf = fetch_pending_scores(q.pending, q.partial, K, q.pend_grid, q.pend_warps);
  const int n_pend = pf.n;
  __syncthreads();
  if (n_pend > 0) {   // a completion left its scores to this selection: form them first (the same on every CTA)
    apply_pending_scores(pf, q.pending, q.partial, q.pend_grid, q.pend_warps, is.score, is.last, is.infl, is.pend_id,
                         is.pend_norm, &is.bad_norm);
    __syncthreads();
  }
  if (p < K) {
    const float r = is.score[p];
    const bool elig = ((q.ineligible == nullptr) || (q.ineligible[p] == 0)) && (is.infl[p] == 0);
    const bool overdue = (t_now - is.last[p]) >= q.H;         // Algorithm 2's staleness test
    long long size = 0;
    for (int sg = T.seg_ptr[p]; sg < T.seg_ptr[p + 1]; ++sg) size += T.len[sg];
    is.fsize[p] = size;
    is.falign[p] = (unsigned char)(T.off[T.seg_ptr[p]] & 3);
    is.cls[p] = elig ? (overdue ? 2 : 1) : 0;
    is.pool[p] = -1;
    if (r != r) is.nan = 1;
    if (writer) {
      q.mask[p] = 0;
      q.ids[p] = -1;
      if (q.pool_offset) q.pool_offset[p] = -1;
    }
  }
  __syncthreads();
  if (is.nan) {
    if (p == 0 && writer) { *q.n_sel = 0; record_status(status, q.err_nonfinite); }
  } else {
    if (p < K && is.cls[p] != 0) {
      const float r = is.score[p];
      const int cls = is.cls[p];
      int rank = 0;
      for (int o = 0; o < K; ++o) {
        const int co = is.cls[o];
        if (co == 0 || o == p) continue;
        bool before;
        if (co != cls) before = co > cls;                 // overdue fragments come first
        else if (cls == 2) before = o < p;                // among overdue: by index
        else {
          const float ro = is.score[o];
          before = (ro > r) || (ro == r && o < p);        // by score, ties to the lower index
        }
        rank += before ? 1 : 0;
      }
      is.order[rank] = p;
      atomicAdd(&is.n_elig, 1);
    }
    __syncthreads();
    if (p == 0) {
      long long remaining = q.budget, pool_pos = 0;
      int n = 0;
      for (int j = 0; j < is.n_elig; ++j) {
        const int f = is.order[j];
        const long long cost = (q.budget_kind == 0) ? 1 : is.fsize[f];
        if (j == 0 || cost <= remaining) {                // the head of the order is always taken
          is.ids[n++] = f;
          remaining -= cost;
          const long long start = pool_pos + is.falign[f];   // same placement rule as k_select
          is.pool[f] = start;
          pool_pos = (start + is.fsize[f] + 3) & ~3LL;
          if (writer) {
            q.mask[f] = 1;
            q.ids[n - 1] = f;
            if (q.pool_offset) q.pool_offset[f] = start;
          }
        }
      }
      is.n = n;
      if (writer) *q.n_sel = n;
    }
  }
  if (p == 0) is.n_pend = n_pend;
  __syncthreads();
}

// What a selection writes to the schedule state, by one thread per CTA once its CTA has finished select_in_cta
// and at a point where waiting for the counter's answer delays nothing (the snapshot kernel calls it from a copy
// warp that has run out of work, long before the DMA thread is done).  Every CTA has read the schedule state
// once the last one gets here: only then is it written - the pending completion's norms, scores, last_sync and
// cleared in-flight marks first, then the marks of what was selected.
__device__ __forceinline__ void select_commit(InlineSelect& is, const SelectRequest& q, int* status) {
  const int n_pend = is.n_pend;
  if (q.in_flight == nullptr && n_pend == 0) return;
  if (arrive_gpu(q.ticket) != (int)gridDim.x - 1) return;
  for (int j = 0; j < n_pend; ++j) {
    const int f = is.pend_id[j];
    q.norms[f] = is.pend_norm[j];
    q.scores_out[f] = is.score[f];
    q.last_sync_out[f] = is.last[f];
    if (q.in_flight != nullptr) q.in_flight[f] = 0;
  }
  if (n_pend > 0) {
    q.pending->n = 0;
    if (is.bad_norm) record_status(status, q.err_nonfinite);
  }
  if (q.in_flight != nullptr)
    for (int j = 0; j < is.n; ++j) q.in_flight[is.ids[j]] = 1;
  *q.ticket = 0;
}

// The same for a pending completion that no selection is about to consume (one block).
static __global__ void __launch_bounds__(256)
k_flush_pending(PendingScores* P, const double* __restrict__ partial, int K, float* __restrict__ norms,
                float* __restrict__ scores, long long* __restrict__ last_sync, unsigned char* __restrict__ in_flight,
                int* __restrict__ status, int err_nonfinite) {
  const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31, nw = blockDim.x >> 5;
  const int n_pend = P->n;
  if (n_pend <= 0 || n_pend > K) return;
  const int grid = P->grid, warps = P->warps;
  const long long t_p = P->t_p, t_l = P->t_l;
  for (int j = warp; j < n_pend; j += nw) {
    const int f = P->ids[j];
    const double total = pending_slot_total(partial, j, grid, warps);
    if (lane == 0) {
      const double norm = sqrt(total);
      long long I = t_p - last_sync[f];
      if (I < 1) I = 1;
      norms[f] = (float)norm;
      scores[f] = (float)(norm / (double)I);
      last_sync[f] = t_l;
      if (in_flight != nullptr) in_flight[f] = 0;
      if (!isfinite(norm)) record_status(status, err_nonfinite);
    }
  }
  __syncthreads();
  if (threadIdx.x == 0) P->n = 0;
}

}  // namespace cocodc

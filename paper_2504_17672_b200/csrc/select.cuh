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

__global__ void __launch_bounds__(kSelectThreads)
k_select(int K, const float* __restrict__ scores, const long long* __restrict__ last_sync,
         const unsigned char* __restrict__ ineligible, const long long* __restrict__ frag_size,
         long long t_now, const long long* __restrict__ t_now_dev, long long H, int budget_kind, long long budget,
         unsigned char* __restrict__ mask, int* __restrict__ ids, int* __restrict__ n_sel,
         long long* __restrict__ pool_offset, int* __restrict__ status, int err_nonfinite) {
  __shared__ float s_score[kMaxK];
  __shared__ unsigned char s_class[kMaxK];  // 0 = ineligible, 1 = ordinary, 2 = overdue
  __shared__ int s_order[kMaxK];
  __shared__ int s_nan;
  __shared__ int s_count;
  const int p = threadIdx.x;
  if (t_now_dev) t_now = *t_now_dev;   // step number kept in device memory (graph replay)
  if (p == 0) { s_nan = 0; s_count = 0; }
  __syncthreads();
  if (p < K) {
    const float r = scores[p];
    const bool elig = (ineligible == nullptr) || (ineligible[p] == 0);
    const bool overdue = (t_now - last_sync[p]) >= H;   // Algorithm 2's staleness test
    s_score[p] = r;
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
  if (p != 0) return;
  long long remaining = budget;
  long long pool_pos = 0;   // next free element of the snapshot pool (kept a multiple of 4)
  int n = 0;
  const int n_elig = s_count;
  for (int j = 0; j < n_elig; ++j) {
    const int f = s_order[j];
    const long long cost = (budget_kind == 0) ? 1 : frag_size[f];
    if (j == 0 || cost <= remaining) {   // the head of the order is always taken
      mask[f] = 1;
      ids[n++] = f;
      remaining -= cost;
      if (pool_offset) {
        pool_offset[f] = pool_pos;
        pool_pos = (pool_pos + frag_size[f] + 3) & ~3LL;
      }
    }
  }
  *n_sel = n;
}

}  // namespace cocodc

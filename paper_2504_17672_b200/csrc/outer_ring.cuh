// The outer-step kernel for worker counts that are not instantiated at compile time (M > 8, or more than
// four local workers in the received-sum mode): the same arithmetic and the same TMA staging as
// k_outer_tma, with the worker count a run-time value.
//
// Shared memory is a ring of 4 KB slots, each one tile of ONE stream, each with its own "full" and "empty"
// barrier.  The producer thread walks the tiles and, per tile, issues the streams in the order the
// arithmetic needs them:
//     theta_g, momentum, received sums,            (what the mode reads of them)
//     recorded values of workers 0 .. M-1,         (modes that form the local pseudo-gradient sum)
//     then per worker its current values           (modes that merge; preceded by the recorded values of that
//                                                   worker when they were not loaded above)
// The consumers take the slots in the same order.  Slots are released as soon as their lane is in a register,
// except the recorded values in the fused mode: they are needed twice (Eq. 1's sum, then Eq. 5-7 per worker),
// so they stay in the ring until their worker has been merged, and the ring is sized M slots larger for it.
// About 80 KB of slots beyond those held are what the producer can have in flight.
//
// Waits are bounded and verdicts are taken per warp, as in k_outer_tma.  Only this GPU's memory and mapped
// peer buffers of received sums are read, with plain one-CTA bulk copies.
#pragma once

#include "outer_tma.cuh"

namespace cocodc {

constexpr int kRingMaxSlots = 54;      // 216 KB of the 227 KB a CTA may use
constexpr int kRingFreeSlots = 20;     // slots beyond the held ones: what may be in flight (80 KB)

__host__ __device__ constexpr bool mode_sums_locally(int mode) {
  return mode == MODE_FUSED || mode == MODE_OUTER_ONLY || mode == MODE_PSEUDO_SUM;
}
// recorded values stay in the ring from the sum to the merge
__host__ __device__ constexpr int ring_held_slots(int mode, int M) {
  return (mode_sums_locally(mode) && mode_merges(mode)) ? M : 0;
}
// 0: the worker count does not fit the ring (the caller falls back to the element loop)
__host__ __device__ constexpr int ring_slots_for(int mode, int M) {
  const int held = ring_held_slots(mode, M);
  const int want = held + kRingFreeSlots;
  const int slots = want > kRingMaxSlots ? kRingMaxSlots : want;
  return slots >= held + 6 ? slots : 0;
}

constexpr int kRingProducers = 4;      // producer threads (one per warp), taking the slots in turn
constexpr int kRingThreads = kThreads + 32 * kRingProducers;

template <int MODE, bool SAME>
__global__ void __launch_bounds__(kRingThreads, 1)
k_outer_ring(const OuterArgs A) {
  static_assert(SAME ? (MODE == MODE_FUSED || MODE == MODE_MERGE_ONLY) : true, "zero delay needs the merge");
  constexpr bool kUpdates = mode_updates_global(MODE);
  constexpr bool kMerges = mode_merges(MODE);
  constexpr bool kLocalSum = mode_sums_locally(MODE);
  constexpr bool kRecv = (MODE == MODE_FUSED_RECV);
  extern __shared__ __align__(128) unsigned char smem_raw[];
  float* const ring = reinterpret_cast<float*>(smem_raw);
  __shared__ __align__(8) unsigned long long full_bar[kRingMaxSlots];
  __shared__ __align__(8) unsigned long long empty_bar[kRingMaxSlots];
  __shared__ volatile int s_fail;
  const int tid = threadIdx.x;
  const int M = A.M;
  const unsigned R = (unsigned)A.ring_slots;
  const int n_recv = kRecv ? A.n_recv : 0;
  const PlanHeader h = *A.hdr;
  if (tid == 0) {
    for (unsigned s = 0; s < R; ++s) {
      mbar_init(smem_u32(&full_bar[s]), 1);
      mbar_init(smem_u32(&empty_bar[s]), kThreads / 32);   // one arrival per consumer warp
    }
    s_fail = 0;
    asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory");
  }
  __syncthreads();

  // ------------------------------------------------------------------ producers
  // One thread issues a 4 KB copy (wait for the slot, arm its barrier, start the copy) every few hundred
  // cycles, less than a tile of many workers needs; so kRingProducers threads share the slots round robin.
  // Every slot has its own barriers, hence the order in which the threads get to issue does not matter.
  if (tid >= kThreads) {
    if ((tid & 31) != 0) return;
    const unsigned me = (unsigned)(tid - kThreads) >> 5;
    TileWalker tw(A.plan, h.n_seg);
    unsigned s = 0, lap = 0;   // next slot of the ring, and how often the ring has been filled
    unsigned turn = 0;         // whose slot the next one is
    bool ok = true;
    auto issue = [&](const float* src) {
      if (!ok) return;
      if (turn == me) {
        if (lap > 0 && (s_fail || !mbar_wait_bounded(smem_u32(&empty_bar[s]), (lap - 1) & 1))) {
          record_status(A.status, A.err_timeout);
          s_fail = 1;
          ok = false;
          return;
        }
        const unsigned bar = smem_u32(&full_bar[s]);
        mbar_expect_tx(bar, kTileBytes);
        bulk_load(smem_u32(ring + (size_t)s * kTileElems), src, kTileBytes, bar);
      }
      if (++turn == kRingProducers) turn = 0;
      if (++s == R) { s = 0; ++lap; }
    };
    for (int tile = blockIdx.x; tile < h.total_tiles && ok; tile += gridDim.x) {
      tw.seek(tile);
      const long long e0 = tw.tile_start(tile);
      if (!tw.interior(e0)) continue;
      const long long snap_e0 = e0 + (tw.sp.snap_off - tw.sp.off);
      issue(A.theta_g + e0);
      if (kUpdates) issue(A.momentum + e0);
      for (int r = 0; r < n_recv; ++r) issue(A.delta_in[r] + e0);
      if (kLocalSum)
        for (int m = 0; m < M; ++m)
          issue(SAME ? A.w_now + m * A.now_stride + e0 : A.w_snap + m * A.snap_stride + snap_e0);
      if (kMerges && !(SAME && kLocalSum))      // fused zero delay: the current values are already in the ring
        for (int m = 0; m < M; ++m) {
          if (!kLocalSum && !SAME) issue(A.w_snap + m * A.snap_stride + snap_e0);
          issue(A.w_now + m * A.now_stride + e0);
        }
    }
    return;
  }

  // ------------------------------------------------------------------ consumers
  SlotAccumulator sa(kThreads / 32);
  TileWalker tw(A.plan, h.n_seg);
  unsigned cs = 0, cphase = 0;   // next slot to take and the phase of its "full" barrier (kept incrementally:
                                 // a division per slot and thread would cost more than the arithmetic)
  bool failed = false;
  // waits for the next slot; the verdict is the warp's
  auto landed = [&]() -> bool {
    const bool ok = mbar_wait_bounded(smem_u32(&full_bar[cs]), cphase);
    if (__all_sync(0xffffffffu, ok)) return true;
    record_status(A.status, A.err_timeout);
    s_fail = 1;
    failed = true;
    return false;
  };
  auto lane_of = [&](unsigned slot) -> float4 {
    return reinterpret_cast<const float4*>(ring + (size_t)slot * kTileElems)[tid];
  };
  // A slot is handed back once per warp, after every lane has read its part: with up to 2M + 2 slots per tile, one
  // arrival per thread would make the barrier updates the bottleneck.
  auto release = [&](unsigned slot) {
    __syncwarp();
    if ((tid & 31) == 0) mbar_arrive(smem_u32(&empty_bar[slot]));
  };
  auto advance = [&]() { if (++cs == R) { cs = 0; cphase ^= 1u; } };
  // next slot: wait, read this thread's lane, release
  auto take = [&](float4& v) -> bool {
    if (!landed()) return false;
    v = lane_of(cs);
    release(cs);
    advance();
    return true;
  };

  for (int tile = blockIdx.x; tile < h.total_tiles && !failed; tile += gridDim.x) {
    if (tw.seek(tile) && A.partial) sa.advance(tw.sp.slot, A.partial);
    const long long e0 = tw.tile_start(tile);
    if (!tw.interior(e0)) {
      ragged_lane<0, MODE, SAME>(A, tw.sp, e0 + 4LL * tid, sa.acc);
      continue;
    }
    const long long e = e0 + 4LL * tid;
    float4 thg, u, sum;
    if (!take(thg)) break;
    if (kUpdates && !take(u)) break;
    if (kRecv) {
      if (!take(sum)) break;
      for (int r = 1; r < n_recv && !failed; ++r) {
        float4 t;
        if (take(t)) sum = add4(sum, t);
      }
      if (failed) break;
    }
    unsigned held = cs;                // slot of worker 0's recorded values (modes that sum locally)
    if (kLocalSum) {
      for (int m = 0; m < M && !failed; ++m) {
        if (!landed()) break;
        const float4 b = lane_of(cs);
        if (!kMerges) release(cs);     // otherwise kept until worker m has been merged
        advance();
#pragma unroll
        for (int k = 0; k < 4; ++k) {
          const float d = __fsub_rn(comp(b, k), comp(thg, k));
          comp(sum, k) = (m == 0) ? d : __fadd_rn(comp(sum, k), d);
        }
      }
      if (failed) break;
    }
    if (MODE == MODE_PSEUDO_SUM) {
      st4(A.delta_out + e, sum);
      continue;
    }
    float4 G = thg;
    if (kUpdates) {
      float4 delta;
      float sq = 0.f;
#pragma unroll
      for (int k = 0; k < 4; ++k) {
        const float Delta = mean_of_sum<0>(comp(sum, k), A);
        float u_new, g;
        outer_update(Delta, comp(thg, k), comp(u, k), A, u_new, g);
        comp(delta, k) = Delta; comp(u, k) = u_new; comp(G, k) = g;
        sq = __fmaf_rn(Delta, Delta, sq);
      }
      sa.acc += (double)sq;
      st4(A.theta_g + e, G);
      st4(A.momentum + e, u);
      if (A.delta_out) st4(A.delta_out + e, delta);
    }
    if (kMerges) {
      for (int m = 0; m < M && !failed; ++m) {
        float4 a, b;
        if (kLocalSum) {
          b = lane_of(held);                    // landed above, still held
          if (SAME) {
            a = b;
          } else {
            if (!landed()) break;
            a = lane_of(cs);
            release(cs);
            advance();
          }
          release(held);
          if (++held == R) held = 0;
        } else {
          if (!SAME && !take(b)) break;
          if (!take(a)) break;
          if (SAME) b = a;
        }
        float4 out;
#pragma unroll
        for (int k = 0; k < 4; ++k) comp(out, k) = merged(comp(a, k), comp(b, k), comp(G, k), A);
        st4(A.w_now + m * A.now_stride + e, out);
      }
    }
  }
  if (failed) return;     // warp-uniform by construction
  if (A.partial) sa.finish(h.n_ids, A.partial);
}

}  // namespace cocodc

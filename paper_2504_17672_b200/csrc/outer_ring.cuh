// The outer-step kernel for worker counts that are not instantiated at compile time (M > 8, or more than
// four local workers in the received-sum mode): the same arithmetic and the same TMA staging as
// k_outer_tma, with the worker count a run-time value.
//
// Shared memory is a ring of 16 KB chunks.  A chunk holds one tile (4 KB) of up to four streams and has one
// "full" and one "empty" barrier.  Per tile the producers fill chunks in the order the arithmetic needs them:
//     head   : theta_g, momentum, received sums            (what the mode reads of them, four to a chunk)
//     sum    : recorded values of workers 0 .. M-1, four workers to a chunk   (modes that form the local sum)
//     merge  : current values, four workers to a chunk (fused mode), or recorded and current values of two
//              workers to a chunk (modes that merge without having summed)
// and the consumers take them in the same order, four (two) workers at a time.  Chunks are handed back as soon
// as their lanes are in registers, except the recorded values in the fused mode: they are needed twice (Eq. 1's
// sum, then Eq. 5-7 per worker), so those chunks stay in the ring until their workers have been merged, and the
// ring is that much larger.
//
// Why chunks: with one barrier pair per 4 KB stream-tile the kernel tops out near 6 million tiles per second and
// SM (5.4 TB/s at M = 16, and the same 20 % short at M = 4) whatever the number of producers, the ring size or
// the polling instruction; the cost sits in the per-barrier hand-shake, so four streams share one.
//
// Waits are bounded and verdicts are taken per warp, as in k_outer_tma.  Only this GPU's memory and mapped
// peer buffers of received sums are read, with plain one-CTA bulk copies.
#pragma once

#include "outer_tma.cuh"

namespace cocodc {

constexpr int kChunkStreams = 4;                                   // stream-tiles per chunk
constexpr unsigned kChunkBytes = kChunkStreams * kTileBytes;       // 16 KB
constexpr int kRingMaxChunks = 13;                                 // 208 KB of the 227 KB a CTA may use
constexpr int kRingFreeChunks = 6;                                 // chunks beyond the held ones: 96 KB in flight at most
constexpr int kRingProducers = 4;                                  // producer threads (one per warp), a chunk each in turn
constexpr int kRingThreads = kThreads + 32 * kRingProducers;

__host__ __device__ constexpr bool mode_sums_locally(int mode) {
  return mode == MODE_FUSED || mode == MODE_OUTER_ONLY || mode == MODE_PSEUDO_SUM;
}
// chunks of recorded values that stay in the ring from the sum to the merge
__host__ __device__ constexpr int ring_held_chunks(int mode, int M) {
  return (mode_sums_locally(mode) && mode_merges(mode)) ? (M + kChunkStreams - 1) / kChunkStreams : 0;
}
// 0: the worker count does not fit the ring (the caller falls back to the element loop)
__host__ __device__ constexpr int ring_chunks_for(int mode, int M) {
  const int held = ring_held_chunks(mode, M);
  const int want = held + kRingFreeChunks;
  const int chunks = want > kRingMaxChunks ? kRingMaxChunks : want;
  return chunks >= held + 3 ? chunks : 0;
}

template <int MODE, bool SAME>
__global__ void __launch_bounds__(kRingThreads, 1)
k_outer_ring(const __grid_constant__ OuterArgs A, const __grid_constant__ FragTable T) {
  static_assert(SAME ? (MODE == MODE_FUSED || MODE == MODE_MERGE_ONLY) : true, "zero delay needs the merge");
  constexpr bool kUpdates = mode_updates_global(MODE);
  constexpr bool kMerges = mode_merges(MODE);
  constexpr bool kLocalSum = mode_sums_locally(MODE);
  constexpr bool kRecv = (MODE == MODE_FUSED_RECV);
  constexpr bool kHeld = kLocalSum && kMerges;          // recorded values wait in the ring for the merge
  // merge phase: workers per chunk and streams per worker that are loaded then
  constexpr int kMergeStreams = !kMerges ? 0 : kHeld ? (SAME ? 0 : 1) : (SAME ? 1 : 2);
  constexpr int kMergeWorkers = (kMergeStreams == 2) ? 2 : 4;
  extern __shared__ __align__(128) unsigned char smem_raw[];
  float* const ring = reinterpret_cast<float*>(smem_raw);
  __shared__ __align__(8) unsigned long long full_bar[kRingMaxChunks];
  __shared__ __align__(8) unsigned long long empty_bar[kRingMaxChunks];
  __shared__ volatile int s_fail;
  __shared__ InlinePlan ip;
  const int tid = threadIdx.x;
  const int M = A.M;
  const unsigned R = (unsigned)A.ring_slots;            // chunks in the ring
  const int n_recv = kRecv ? A.n_recv : 0;
  const int n_head = 1 + (kUpdates ? 1 : 0) + n_recv;   // streams of the head
  const PlanView pv = acquire_plan(ip, T, A.rq, A.plan, A.hdr, A.status);
  const PlanHeader h = pv.hdr;
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
  // All walk the same chunk sequence; a producer fills the chunks whose turn is its own.  Every chunk has its own
  // barriers, hence the order in which the producers get to issue does not matter.
  if (tid >= kThreads) {
    if ((tid & 31) != 0) return;
    const unsigned me = (unsigned)(tid - kThreads) >> 5;
    TileWalker tw(pv.seg, h.n_seg);
    unsigned s = 0, lap = 0;   // next chunk of the ring, and how often the ring has been filled
    unsigned turn = 0;         // whose chunk the next one is
    bool ok = true;
    // opens the next chunk for n streams; true if it is this producer's to fill
    auto open = [&](int n, float*& dst, unsigned& bar) -> bool {
      const bool mine = ok && (turn == me);
      if (mine) {
        if (lap > 0 && (s_fail || !mbar_wait_bounded(smem_u32(&empty_bar[s]), (lap - 1) & 1))) {
          record_status(A.status, A.err_timeout);
          s_fail = 1;
          ok = false;
        } else {
          bar = smem_u32(&full_bar[s]);
          dst = ring + (size_t)s * (kChunkStreams * kTileElems);
          mbar_expect_tx(bar, (unsigned)n * kTileBytes);
        }
      }
      if (++turn == kRingProducers) turn = 0;
      if (++s == R) { s = 0; ++lap; }
      return mine && ok;
    };
    auto copy = [&](float* dst, int j, const float* src, unsigned bar) {
      bulk_load(smem_u32(dst + j * kTileElems), src, kTileBytes, bar);
    };
    for (int tile = blockIdx.x; tile < h.total_tiles && ok; tile += gridDim.x) {
      tw.seek(tile);
      const long long e0 = tw.tile_start(tile);
      if (!tw.interior(e0)) continue;
      const long long snap_e0 = e0 + (tw.sp.snap_off - tw.sp.off);
      float* dst = nullptr;
      unsigned bar = 0;
      // head: stream i of the head is theta_g, then momentum (if read), then the received sums
      for (int i0 = 0; i0 < n_head; i0 += kChunkStreams) {
        const int cnt = (n_head - i0 < kChunkStreams) ? n_head - i0 : kChunkStreams;
        if (!open(cnt, dst, bar)) continue;
        for (int j = 0; j < cnt; ++j) {
          const int i = i0 + j;
          const float* src = (i == 0) ? A.theta_g + e0
                           : (kUpdates && i == 1) ? A.momentum + e0
                           : A.delta_in[i - 1 - (kUpdates ? 1 : 0)] + e0;
          copy(dst, j, src, bar);
        }
      }
      if (kLocalSum)
        for (int m0 = 0; m0 < M; m0 += kChunkStreams) {
          const int cnt = (M - m0 < kChunkStreams) ? M - m0 : kChunkStreams;
          if (!open(cnt, dst, bar)) continue;
          for (int j = 0; j < cnt; ++j)
            copy(dst, j, SAME ? A.w_now + (m0 + j) * A.now_stride + e0
                              : A.w_snap + (m0 + j) * A.snap_stride + snap_e0, bar);
        }
      if (kMergeStreams > 0)
        for (int m0 = 0; m0 < M; m0 += kMergeWorkers) {
          const int cnt = (M - m0 < kMergeWorkers) ? M - m0 : kMergeWorkers;
          if (!open(cnt * kMergeStreams, dst, bar)) continue;
          for (int j = 0; j < cnt; ++j) {
            if (kMergeStreams == 2) {
              copy(dst, 2 * j, A.w_snap + (m0 + j) * A.snap_stride + snap_e0, bar);
              copy(dst, 2 * j + 1, A.w_now + (m0 + j) * A.now_stride + e0, bar);
            } else {
              copy(dst, j, A.w_now + (m0 + j) * A.now_stride + e0, bar);
            }
          }
        }
    }
    return;
  }

  // ------------------------------------------------------------------ consumers
  SlotAccumulator sa(kThreads / 32);
  TileWalker tw(pv.seg, h.n_seg);
  unsigned cs = 0, cphase = 0;   // next chunk to take and the phase of its "full" barrier
  bool failed = false;
  // waits for the next chunk; the verdict is the warp's
  auto landed = [&]() -> bool {
    const bool ok = mbar_wait_bounded(smem_u32(&full_bar[cs]), cphase);
    if (__all_sync(0xffffffffu, ok)) return true;
    record_status(A.status, A.err_timeout);
    s_fail = 1;
    failed = true;
    return false;
  };
  // this thread's lane of stream j of a chunk
  auto lane_of = [&](unsigned chunk, int j) -> float4 {
    return reinterpret_cast<const float4*>(ring + (size_t)chunk * (kChunkStreams * kTileElems) + j * kTileElems)[tid];
  };
  // a chunk is handed back once per warp, after every lane has read its part
  auto release = [&](unsigned chunk) {
    __syncwarp();
    if ((tid & 31) == 0) mbar_arrive(smem_u32(&empty_bar[chunk]));
  };
  auto advance = [&]() { if (++cs == R) { cs = 0; cphase ^= 1u; } };

  for (int tile = blockIdx.x; tile < h.total_tiles && !failed; tile += gridDim.x) {
    if (tw.seek(tile) && A.partial) sa.advance(tw.sp.slot, A.partial);
    const long long e0 = tw.tile_start(tile);
    if (!tw.interior(e0)) {
      ragged_lane<0, MODE, SAME>(A, tw.sp, e0 + 4LL * tid, sa.acc);
      continue;
    }
    const long long e = e0 + 4LL * tid;
    // ---- head
    float4 thg, u, sum;
    for (int i0 = 0; i0 < n_head && !failed; i0 += kChunkStreams) {
      const int cnt = (n_head - i0 < kChunkStreams) ? n_head - i0 : kChunkStreams;
      if (!landed()) break;
      float4 v[kChunkStreams];
#pragma unroll
      for (int j = 0; j < kChunkStreams; ++j)
        if (j < cnt) v[j] = lane_of(cs, j);
      release(cs);
      advance();
#pragma unroll
      for (int j = 0; j < kChunkStreams; ++j) {
        if (j >= cnt) continue;
        const int i = i0 + j;
        if (i == 0) thg = v[j];
        else if (kUpdates && i == 1) u = v[j];
        else if (i == 1 + (kUpdates ? 1 : 0)) sum = v[j];            // first received sum
        else sum = add4(sum, v[j]);                                  // the others, in the order listed
      }
    }
    if (failed) break;
    // ---- Eq. 1's sum over the local workers
    unsigned held = cs;                // chunk of workers 0-3's recorded values
    if (kLocalSum) {
      for (int m0 = 0; m0 < M && !failed; m0 += kChunkStreams) {
        const int cnt = (M - m0 < kChunkStreams) ? M - m0 : kChunkStreams;
        if (!landed()) break;
        float4 b[kChunkStreams];
#pragma unroll
        for (int j = 0; j < kChunkStreams; ++j)
          if (j < cnt) b[j] = lane_of(cs, j);
        if (!kHeld) release(cs);       // otherwise kept until these workers have been merged
        advance();
#pragma unroll
        for (int j = 0; j < kChunkStreams; ++j) {
          if (j >= cnt) continue;
#pragma unroll
          for (int k = 0; k < 4; ++k) {
            const float d = __fsub_rn(comp(b[j], k), comp(thg, k));
            comp(sum, k) = (m0 + j == 0) ? d : __fadd_rn(comp(sum, k), d);
          }
        }
      }
      if (failed) break;
    }
    if (MODE == MODE_PSEUDO_SUM) {
      st4(A.delta_out + e, sum);
      continue;
    }
    // ---- Eq. 2
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
    // ---- Eq. 3-7 per worker
    if (kMerges) {
      float* wp = A.w_now + e;         // worker m's lane of this tile
      for (int m0 = 0; m0 < M && !failed; m0 += kMergeWorkers) {
        const int cnt = (M - m0 < kMergeWorkers) ? M - m0 : kMergeWorkers;
        float4 a[kMergeWorkers], b[kMergeWorkers];
        if (kMergeStreams > 0 && !landed()) break;
#pragma unroll
        for (int j = 0; j < kMergeWorkers; ++j) {
          if (j >= cnt) continue;
          if (kHeld) {
            b[j] = lane_of(held, j);                     // landed during the sum, still in the ring
            a[j] = SAME ? b[j] : lane_of(cs, j);
          } else if (kMergeStreams == 2) {
            b[j] = lane_of(cs, 2 * j);
            a[j] = lane_of(cs, 2 * j + 1);
          } else {                                       // merge only, zero delay
            a[j] = lane_of(cs, j);
            b[j] = a[j];
          }
        }
        if (kMergeStreams > 0) { release(cs); advance(); }
        if (kHeld) { release(held); if (++held == R) held = 0; }
#pragma unroll
        for (int j = 0; j < kMergeWorkers; ++j) {
          if (j >= cnt) continue;
          float4 out;
#pragma unroll
          for (int k = 0; k < 4; ++k) comp(out, k) = merged(comp(a[j], k), comp(b[j], k), comp(G, k), A);
          st4(wp, out);
          wp += A.now_stride;
        }
      }
    }
  }
  if (failed) return;     // warp-uniform by construction
  if (A.partial) {
    sa.finish(h.n_ids, A.partial);
    finalize_epilogue(ip, A.fin, h, A.partial, kThreads / 32, A.status);
  }
}

}  // namespace cocodc

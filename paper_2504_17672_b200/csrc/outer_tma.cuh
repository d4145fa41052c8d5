// The fused outer-step kernel for the instantiated worker counts: the inputs of every tile are brought
// into shared memory by the TMA unit (1-D bulk asynchronous copies); the outputs leave from registers.
//
// One CTA per SM: warps 0-7 compute, warp 8 is the producer (lane l issues the copies of stream l).  A stage is
// one tile (1024 elements = 4 KB) of every stream the mode reads.  Per tile:
//   producer : waits until the stage is free ("empty" barrier, one arrival per consumer thread), arms the
//              stage's "full" barrier with the byte count, issues one bulk copy global->shared per stream;
//   consumers: wait on "full", read their 16-byte lane of every stream from shared memory into registers,
//              arrive on "empty" at once (the stage can be refilled while they compute), do the arithmetic
//              of outer.cuh, and write their outputs with streaming 16-byte stores.
// How far the producer runs ahead is the tuning knob: measured on B200, bandwidth peaks at 16-20
// outstanding 4 KB copies per SM (64-80 KB in flight) and falls by 5-8 % at twice that, so the ring has
// only as many stages as that takes (2 at M = 4), not as many as shared memory would hold.
// Tiles that are ragged or whose snapshot placement is not 16-byte compatible never enter the
// pipeline: the consumers process them straight from global memory (ragged_lane); producer and
// consumers agree on which tiles those are from the plan alone.
//
// Every wait is bounded.  When one runs out the thread records COCODC_ERR_TIMEOUT, raises a flag the
// others poll, and leaves; no thread waits on a barrier another thread could have abandoned.
// Every copy is a plain one-CTA bulk copy (no cluster-wide form); only this GPU's memory is read, apart from
// buffers of received sums that the caller may have mapped from a peer.
//
// Every kernel here is the whole of its C-ABI call: it expands the device-resident id list in its prologue
// (acquire_plan) and, where scores are asked for, its last warp forms them (finalize_epilogue); the snapshot
// kernel can also run Algorithm 2 first (select_in_cta).  The streaming loops between prologue and epilogue are
// separate out-of-line functions: inlined next to that code they ran up to 1 % slower, by amounts that moved
// with unrelated edits.
#pragma once

#include "outer.cuh"
#include "select.cuh"

namespace cocodc {

// k_outer_tma runs eight consumer warps and one producer warp, whose lanes each issue one stream's copies.
__host__ __device__ constexpr int tma_threads(int /*M*/) { return kThreads + 32; }
constexpr unsigned kTileBytes = kTileElems * sizeof(float);   // one stream's share of a stage
constexpr int kWaitLimit = 1 << 22;                           // polls of a barrier before giving up
constexpr int kMaxStages = 10;

// ---- PTX wrappers ------------------------------------------------------------------------------
__device__ __forceinline__ unsigned smem_u32(const void* p) { return (unsigned)__cvta_generic_to_shared(p); }
__device__ __forceinline__ void mbar_init(unsigned bar, int count) {
  asm volatile("mbarrier.init.shared::cta.b64 [%0], %1;" ::"r"(bar), "r"(count));
}
__device__ __forceinline__ void mbar_expect_tx(unsigned bar, unsigned bytes) {
  asm volatile("mbarrier.arrive.expect_tx.shared::cta.b64 _, [%0], %1;" ::"r"(bar), "r"(bytes) : "memory");
}
__device__ __forceinline__ void mbar_arrive(unsigned bar) {
  asm volatile("mbarrier.arrive.shared::cta.b64 _, [%0];" ::"r"(bar) : "memory");
}
__device__ __forceinline__ bool mbar_try_wait(unsigned bar, unsigned parity) {
  unsigned ok;
  asm volatile(
      "{\n .reg .pred p;\n mbarrier.try_wait.parity.shared::cta.b64 p, [%1], %2;\n selp.u32 %0, 1, 0, p;\n}"
      : "=r"(ok) : "r"(bar), "r"(parity) : "memory");
  return ok != 0;
}
// false if the phase did not complete within the poll limit
__device__ __forceinline__ bool mbar_wait_bounded(unsigned bar, unsigned parity) {
  for (int i = 0; i < kWaitLimit; ++i)
    if (mbar_try_wait(bar, parity)) return true;
  return false;
}
// the same with a caller-chosen limit
__device__ __forceinline__ bool mbar_wait_limit(unsigned bar, unsigned parity, int limit) {
  for (int i = 0; i < limit; ++i)
    if (mbar_try_wait(bar, parity)) return true;
  return false;
}
__device__ __forceinline__ void bulk_load(unsigned dst_smem, const void* src, unsigned bytes, unsigned bar) {
  asm volatile("cp.async.bulk.shared::cluster.global.mbarrier::complete_tx::bytes [%0], [%1], %2, [%3];"
               ::"r"(dst_smem), "l"(src), "r"(bytes), "r"(bar) : "memory");
}
// Bulk stores (the snapshot copy): the lines written are not read again soon, so they are marked
// evict-first in L2 and drain to DRAM early instead of displacing the loads that follow.
__device__ __forceinline__ unsigned long long l2_evict_first_policy() {
  unsigned long long pol;
  asm volatile("createpolicy.fractional.L2::evict_first.b64 %0, 1.0;" : "=l"(pol));
  return pol;
}
__device__ __forceinline__ void bulk_store(void* dst, unsigned src_smem, unsigned bytes, unsigned long long policy) {
  asm volatile("cp.async.bulk.global.shared::cta.bulk_group.L2::cache_hint [%0], [%1], %2, %3;"
               ::"l"(dst), "r"(src_smem), "r"(bytes), "l"(policy) : "memory");
}
__device__ __forceinline__ void bulk_commit() { asm volatile("cp.async.bulk.commit_group;" ::: "memory"); }
__device__ __forceinline__ void bulk_wait_all() { asm volatile("cp.async.bulk.wait_group 0;" ::: "memory"); }

// Ring depth of the received-sum mode, whose stage size is known only at run time: about 72 KB of
// copies in flight, at least two stages (host and device use the same function).
__host__ __device__ constexpr int stages_for(int loaded_streams) {
  const int stage = loaded_streams * (int)kTileBytes;
  const int raw = (72 * 1024 + stage / 2) / stage;
  return raw < 2 ? 2 : (raw > kMaxStages ? kMaxStages : raw);
}

// ---- stage layout ----------------------------------------------------------------------------
// Slots of kTileElems floats each: [recorded x nS][current x nN][global][momentum x nU], then, in
// MODE_FUSED_RECV, one slot per buffer of received sums (a run-time count, so that mode sizes its ring at
// run time: stages_for()).
// U: tiles of kTileElems elements that one stage holds per stream (one bulk copy of U * 4 KB per stream; every
// consumer thread then owns U lanes).  One producer thread starts a copy every few hundred cycles whatever its
// size, so a mode that reads only two or three streams cannot be fed 4 KB at a time (the pseudo-gradient sum of
// a single worker ran at 4.9 TB/s that way); such modes take wider tiles.  Measured on B200 (GB/s through the C
// ABI, 100 M parameters per worker, tile widths 1 / 2 / 4 / 8 where tried):
//   pseudo-gradient sum  M = 1 (2 streams): 4941 / - / 6190 / 6038     M = 2 (3): 5977 / 6740 / 6759 / -
//                        M = 3 (4 streams): 6696 / 6832 / 6869 / -     M = 4 (5): 6736 / 6682 / - / -
//   merge only           M = 1 (3 streams): 5760 / 6600 / 6766 / -     M = 2 (5): 6498 / 6792 / - / -
//   outer update only    M = 1 (3 streams): 6237 / 6161 / 6304 / -     M = 2 (4): 6194 / 6373 / 6195 / -
//   fused                M = 1 (4 streams): 6392 / 6404 / 6154 / -     M = 2 (6): 6495 / 6433 / - / -
__host__ __device__ constexpr int tile_width(int loaded_streams) {
  return loaded_streams <= 3 ? 4 : loaded_streams <= 5 ? 2 : 1;
}

template <int M, int MODE, bool SAME, int U = 1>
struct StageLayout {
  static constexpr int nS = SAME ? 0 : M;
  static constexpr int nN = mode_merges(MODE) ? M : 0;
  static constexpr int nU = mode_updates_global(MODE) ? 1 : 0;
  static constexpr int kSnap = 0;
  static constexpr int kNow = nS;
  static constexpr int kGlobal = nS + nN;
  static constexpr int kMomentum = kGlobal + 1;
  static constexpr int kDeltaIn = kMomentum + nU;
  static constexpr int kLoaded = nS + nN + 1 + nU;       // streams brought in by the producer (plus the received sums)
  static constexpr unsigned kSlotElems = U * kTileElems;  // one stream's share of a stage
  static constexpr unsigned kStageBytes = kLoaded * U * kTileBytes;
  // about 72 KB of copies in flight (see the note at the top), never fewer than two stages; the
  // read-heavy modes measure best with more: OUTER_ONLY (3 reads per write) one stage deeper,
  // PSEUDO_SUM (M + 1 reads per write) at 100-110 KB
  static constexpr int kInFlightBytes =
      (MODE == MODE_PSEUDO_SUM ? 110 : MODE == MODE_OUTER_ONLY ? 96 : 72) * 1024;
  static constexpr int kStagesRaw = (kInFlightBytes + (int)kStageBytes / 2) / (int)kStageBytes;   // nearest
  static constexpr int kStages = kStagesRaw < 2 ? 2 : (kStagesRaw > kMaxStages ? kMaxStages : kStagesRaw);
  static constexpr unsigned kSmemBytes = kStages * kStageBytes;
  static_assert(kSmemBytes <= 227 * 1024, "stages do not fit in shared memory");
  static_assert(SAME ? (MODE == MODE_FUSED || MODE == MODE_MERGE_ONLY) : true,
                "zero-delay mode needs the merge and local pseudo-gradients");
  static_assert(U == 1 || MODE != MODE_FUSED_RECV, "the received-sum mode sizes its stages at run time for U = 1");
  static_assert(kLoaded + (MODE == MODE_FUSED_RECV ? kMaxRecv : 0) <= 32, "one lane of the producer warp per stream");
};

// The two roles of k_outer_tma are compiled as functions of their own (out of line): what the compiler makes
// of the streaming loops then does not depend on the prologue and epilogue code around them (measured: the
// same loops inlined next to that code ran up to 1 % slower, depending on what exactly stood beside them).
struct TmaShared {
  float* stages;
  unsigned long long* full_bar;
  unsigned long long* empty_bar;
  volatile int* s_fail;
  double* warp_part;     // where the warps' sums of squares go (shared memory for short id lists), or nullptr
};

// Lane l of the producer warp owns stream l of the stage (slot order: recorded values, current values, global
// state, momentum, received sums): it keeps that stream's base pointer in registers and issues the stream's
// one bulk copy per tile.  The lanes' copies leave with one warp instruction instead of one instruction
// sequence per stream (a single issuing thread needed a few hundred cycles per copy, and with only two or
// three stages the time from "stage free" to "last copy issued" sits on the pipeline's critical path).  Lane 0
// arms the barrier with the whole byte count; a copy that completes before the arming arrival only runs the
// transaction count negative for a moment, the phase cannot end before that arrival.
template <int M, int MODE, bool SAME, int U>
__device__ __noinline__ void tma_producer_warp(const OuterArgs& A, const SegPlan* plan, const PlanHeader h,
                                               const TmaShared sh) {
  using L = StageLayout<M, MODE, SAME, U>;
  constexpr int kSlot = U * kTileElems;
  constexpr unsigned kSlotBytes = U * kTileBytes;
  constexpr bool kRecv = (MODE == MODE_FUSED_RECV);
  const int n_recv = kRecv ? A.n_recv : 0;
  const int loaded = L::kLoaded + n_recv;
  const int S = kRecv ? stages_for(loaded) : L::kStages;
  const int lane = threadIdx.x & 31;
  const bool has_stream = lane < loaded;
  const bool from_snap = lane < L::nS;
  const float* base = nullptr;
  if (has_stream) {
    if (lane < L::nS) base = A.w_snap + (long long)lane * A.snap_stride;
    else if (lane < L::nS + L::nN) base = A.w_now + (long long)(lane - L::nS) * A.now_stride;
    else if (lane == L::kGlobal) base = A.theta_g;
    else if (L::nU && lane == L::kMomentum) base = A.momentum;
    else base = A.delta_in[lane - L::kDeltaIn];
  }
  TileWalker tw(plan, h.n_seg, kSlot);
  int k = 0;   // staged tiles issued so far
  // Leaving early (a wait ran out here or in a consumer): the copies already issued may still be landing in
  // this CTA's shared memory, which must not be handed to another CTA before they have; wait for the stages
  // armed last, again with a limit.
  auto drain = [&]() {
    for (int i = (k > S ? k - S : 0); i < k; ++i) mbar_wait_bounded(smem_u32(&sh.full_bar[i % S]), (i / S) & 1);
  };
  for (int tile = blockIdx.x; tile < h.total_tiles; tile += gridDim.x) {
    tw.seek(tile);
    const long long e0 = tw.tile_start(tile);
    if (!tw.interior(e0)) continue;
    const int s = k % S;
    const bool free_now = (k < S) || mbar_wait_bounded(smem_u32(&sh.empty_bar[s]), ((k / S) - 1) & 1);
    if (!__all_sync(0xffffffffu, free_now && !*sh.s_fail)) {      // one verdict for the warp
      if (!free_now) record_status(A.status, A.err_timeout);
      *sh.s_fail = 1;
      drain();
      return;
    }
    const unsigned bar = smem_u32(&sh.full_bar[s]);
    if (lane == 0) mbar_expect_tx(bar, loaded * kSlotBytes);
    if (has_stream) {
      const long long e_src = from_snap ? e0 + (tw.sp.snap_off - tw.sp.off) : e0;
      bulk_load(smem_u32(sh.stages + ((size_t)s * loaded + lane) * kSlot), base + e_src, kSlotBytes, bar);
    }
    ++k;
  }
}

// The eight consumer warps: returns false if a wait ran out (warp-uniform), after writing this warp's partial
// sums otherwise.
template <int M, int MODE, bool SAME, int U>
__device__ __noinline__ bool tma_consumer_warps(const OuterArgs& A, const SegPlan* plan, const PlanHeader h,
                                                const TmaShared sh) {
  using L = StageLayout<M, MODE, SAME, U>;
  constexpr int kSlot = U * kTileElems;
  constexpr bool kRecv = (MODE == MODE_FUSED_RECV);
  const int n_recv = kRecv ? A.n_recv : 0;
  const int loaded = L::kLoaded + n_recv;
  const int S = kRecv ? stages_for(loaded) : L::kStages;
  const int tid = threadIdx.x;
  SlotAccumulator sa(kThreads / 32);
  sa.cta_part = sh.warp_part;
  TileWalker tw(plan, h.n_seg, kSlot);
  int k = 0;           // staged tiles consumed so far
  for (int tile = blockIdx.x; tile < h.total_tiles; tile += gridDim.x) {
    if (tw.seek(tile) && A.partial) sa.advance(tw.sp.slot, A.partial);
    const long long e0 = tw.tile_start(tile);
    if (!tw.interior(e0)) {
      sa.acc += ragged_tile<M, MODE, SAME, U>(A, tw.sp, e0 + 4LL * tid);
      continue;
    }
    const int s = k % S;
    // the verdict is taken per warp, so that a warp never splits around the full-warp shuffles of the
    // score accumulation
    const bool landed = !*sh.s_fail && mbar_wait_bounded(smem_u32(&sh.full_bar[s]), (k / S) & 1);
    if (!__all_sync(0xffffffffu, landed)) {
      record_status(A.status, A.err_timeout);
      *sh.s_fail = 1;
      return false;
    }
    const float* st = sh.stages + (size_t)s * loaded * kSlot;
    Lane<M, MODE, SAME> ln[U];
#pragma unroll
    for (int v = 0; v < U; ++v) {
      auto slot = [&](int idx) -> const float4& {
        return reinterpret_cast<const float4*>(st + idx * kSlot)[v * kThreads + tid];
      };
      ln[v].thg = slot(L::kGlobal);
      if (L::nU) ln[v].u = slot(L::kMomentum);
      if (kRecv) {
        ln[v].delta = slot(L::kDeltaIn);
        for (int r = 1; r < n_recv; ++r) ln[v].delta = add4(ln[v].delta, slot(L::kDeltaIn + r));
      }
      if (SAME) {
#pragma unroll
        for (int m = 0; m < M; ++m) ln[v].b[m] = slot(L::kNow + m);
      } else {
#pragma unroll
        for (int m = 0; m < M; ++m) ln[v].b[m] = slot(L::kSnap + m);
        if (L::nN) {
#pragma unroll
          for (int m = 0; m < M; ++m) ln[v].a[m] = slot(L::kNow + m);
        }
      }
    }
    mbar_arrive(smem_u32(&sh.empty_bar[s]));   // this thread's lanes are in registers: its share of the stage is free
#pragma unroll
    for (int v = 0; v < U; ++v) {
      ln[v].compute(A, sa.acc);
      ln[v].store(A, e0 + 4LL * (v * kThreads + tid));
    }
    ++k;
  }
  if (A.partial) sa.finish(h.n_ids, A.partial);
  return true;
}

template <int M, int MODE, bool SAME, int U = 1>
__global__ void __launch_bounds__(tma_threads(M), 1)
k_outer_tma(const __grid_constant__ OuterArgs A, const __grid_constant__ FragTable T) {
  using L = StageLayout<M, MODE, SAME, U>;
  constexpr bool kRecv = (MODE == MODE_FUSED_RECV);
  const int S = kRecv ? stages_for(L::kLoaded + A.n_recv) : L::kStages;   // a compile-time constant unless kRecv
  extern __shared__ __align__(128) unsigned char smem_raw[];
  __shared__ __align__(8) unsigned long long full_bar[kMaxStages];
  __shared__ __align__(8) unsigned long long empty_bar[kMaxStages];
  __shared__ volatile int s_fail;
  __shared__ InlinePlan ip;

  const int tid = threadIdx.x;
  const PlanView pv = acquire_plan(ip, T, A.rq, A.plan, A.hdr, A.status);
  if (tid == 0) {
    for (int s = 0; s < S; ++s) {
      mbar_init(smem_u32(&full_bar[s]), 1);
      mbar_init(smem_u32(&empty_bar[s]), kThreads);   // every consumer thread releases its own lane
    }
    s_fail = 0;
    asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory");
  }
  __syncthreads();
  TmaShared sh;
  sh.stages = reinterpret_cast<float*>(smem_raw);
  sh.full_bar = full_bar;
  sh.empty_bar = empty_bar;
  sh.s_fail = &s_fail;
  // short id lists: the warps' sums meet in shared memory and the CTA writes one entry per slot
  const bool in_shared = A.fin.ticket != nullptr && pv.hdr.n_ids <= kFastSlots;
  sh.warp_part = in_shared ? ip.warp_part : nullptr;
  if (tid >= kThreads) {
    tma_producer_warp<M, MODE, SAME, U>(A, pv.seg, pv.hdr, sh);
    return;
  }
  if (!tma_consumer_warps<M, MODE, SAME, U>(A, pv.seg, pv.hdr, sh)) return;     // warp-uniform by construction
  if (A.partial) finalize_epilogue(ip, A.fin, pv.hdr, A.partial, kThreads / 32, A.status, in_shared);
}

}  // namespace cocodc

namespace cocodc {

// ---------------------------------------------------------------------------------------------
// S0 as a pure DMA job: copy the listed fragments of every worker from w_now into w_snap.
//
// One thread per CTA drives the TMA unit: bulk load of a 32 KB chunk (one tile of one worker) into
// a shared-memory stage, and, once it has landed, a bulk store of the same stage to its place in
// w_snap.  kSnapStages stages with up to kSnapDepth loads in flight keep 64 KB of reads and as much of
// writes outstanding per SM (measured optimum: 48-64 KB; 80 KB and more lose 5 %).  Warps 1-7 meanwhile copy the ragged tiles (segment
// edges, snapshot placements that are not 16-byte compatible) with ordinary loads and stores.
// ---------------------------------------------------------------------------------------------
constexpr int kSnapU = 8;                                      // lanes per thread and tile
constexpr int kSnapTileElems = kTileElems * kSnapU;            // 8192 elements = 32 KB per worker
constexpr unsigned kSnapChunkBytes = kSnapTileElems * sizeof(float);
constexpr int kSnapStages = 4;
constexpr int kSnapDepth = 2;                                  // loads in flight before the oldest is stored
constexpr unsigned kSnapSmemBytes = kSnapStages * kSnapChunkBytes;

template <int N> __device__ __forceinline__ void bulk_wait_read_n() {
  asm volatile("cp.async.bulk.wait_group.read %0;" ::"n"(N) : "memory");
}

struct SnapshotJob {
  const float* w_now;
  float* w_snap;
  long long now_stride, snap_stride;
  int M;
  int* status;
  int err_timeout;
};

// The copy loops of k_snapshot_tma, out of line for the same reason as the roles of k_outer_tma.
static __device__ __noinline__ void snapshot_copy(const SnapshotJob J, const SegPlan* plan, const PlanHeader h,
                                                  float* stages, unsigned long long* full_bar, float** dst_of_stage) {
  const float* __restrict__ w_now = J.w_now;
  float* __restrict__ w_snap = J.w_snap;
  const long long now_stride = J.now_stride, snap_stride = J.snap_stride;
  const int M = J.M;
  int* status = J.status;
  const int err_timeout = J.err_timeout;
  const int tid = threadIdx.x;
  auto tile_geometry = [&](int tile, int& seg, SegPlan& sp, int& loaded, long long& e0, bool& interior) {
    while (seg + 1 < h.n_seg && tile >= plan[seg + 1].first_tile) ++seg;
    if (seg != loaded) { sp = plan[seg]; loaded = seg; }
    e0 = sp.abase + (long long)(tile - sp.first_tile) * kSnapTileElems;
    interior = sp.vec_ok && e0 >= sp.off && e0 + kSnapTileElems <= sp.off + sp.len;
  };

  if (tid == 0) {
    // ---- DMA driver
    int seg = 0, loaded = -1;
    SegPlan sp;
    int issued = 0, stored = 0;
    bool ok = true;
    const unsigned long long store_policy = l2_evict_first_policy();
    auto drain_one = [&]() {
      const int s = stored % kSnapStages;
      if (!mbar_wait_bounded(smem_u32(&full_bar[s]), (stored / kSnapStages) & 1)) {
        record_status(status, err_timeout);
        ok = false;
        return;
      }
      bulk_store(dst_of_stage[s], smem_u32(stages + (size_t)s * kSnapTileElems), kSnapChunkBytes, store_policy);
      bulk_commit();
      ++stored;
    };
    for (int tile = blockIdx.x; tile < h.total_tiles && ok; tile += gridDim.x) {
      long long e0; bool interior;
      tile_geometry(tile, seg, sp, loaded, e0, interior);
      if (!interior) continue;
      const long long shift = sp.snap_off - sp.off;
      for (int m = 0; m < M && ok; ++m) {
        if (issued - stored == kSnapDepth) drain_one();
        if (!ok) break;
        const int s = issued % kSnapStages;
        // the stage's previous store (chunk issued - kSnapStages) is older than the newest
        // kSnapStages - kSnapDepth - 1 committed groups: waiting until at most that many are
        // still reading guarantees it has finished with the stage
        if (issued >= kSnapStages) bulk_wait_read_n<kSnapStages - kSnapDepth - 1>();
        const unsigned bar = smem_u32(&full_bar[s]);
        mbar_expect_tx(bar, kSnapChunkBytes);
        bulk_load(smem_u32(stages + (size_t)s * kSnapTileElems), w_now + m * now_stride + e0, kSnapChunkBytes, bar);
        dst_of_stage[s] = w_snap + m * snap_stride + shift + e0;
        ++issued;
      }
    }
    while (ok && stored < issued) drain_one();
    bulk_wait_all();
    return;
  }
  if (tid < 32) return;

  // ---- ragged tiles, warps 1-7
  const int wtid = tid - 32;
  constexpr int kWorkers = kThreads - 32;
  int seg = 0, loaded = -1;
  SegPlan sp;
  for (int tile = blockIdx.x; tile < h.total_tiles; tile += gridDim.x) {
    long long e0; bool interior;
    tile_geometry(tile, seg, sp, loaded, e0, interior);
    if (interior) continue;
    const long long seg_end = sp.off + sp.len;
    const long long shift = sp.snap_off - sp.off;
    // one lane: false once the tile has run past the end of the segment
    auto copy_lane = [&](int l) -> bool {
      const long long e = e0 + 4LL * l;
      if (e >= seg_end) return false;
      if (sp.vec_ok && e >= sp.off && e + 4 <= seg_end) {
        for (int m = 0; m < M; ++m) st4(w_snap + m * snap_stride + shift + e, ld4(w_now + m * now_stride + e));
      } else if (e >= sp.off && e + 4 <= seg_end) {   // a place that is not 16-byte compatible: vector in, elements out
        for (int m = 0; m < M; ++m) {
          const float4 v = ld4(w_now + m * now_stride + e);
          float* d = w_snap + m * snap_stride + shift + e;
          st1(d, v.x); st1(d + 1, v.y); st1(d + 2, v.z); st1(d + 3, v.w);
        }
      } else {
        for (int k = 0; k < 4; ++k) {
          const long long ee = e + k;
          if (ee >= sp.off && ee < seg_end)
            for (int m = 0; m < M; ++m) st1(w_snap + m * snap_stride + shift + ee, ld1(w_now + m * now_stride + ee));
        }
      }
      return true;
    };
    // A segment whose place is not 16-byte compatible has no interior tiles: all of it comes through here, so
    // full lanes go kBatch at a time per thread, loads first (enough of them in flight to matter), stores after.
    constexpr int kBatch = 8;
    for (int l0 = wtid; l0 < kSnapTileElems / 4; l0 += kWorkers * kBatch) {
      const int l_last = l0 + (kBatch - 1) * kWorkers;
      const bool batch = !sp.vec_ok && l_last < kSnapTileElems / 4 && e0 + 4LL * l0 >= sp.off &&
                         e0 + 4LL * l_last + 4 <= seg_end;
      if (batch) {
        for (int m = 0; m < M; ++m) {
          float4 v[kBatch];
#pragma unroll
          for (int j = 0; j < kBatch; ++j) v[j] = ld4(w_now + m * now_stride + e0 + 4LL * (l0 + j * kWorkers));
#pragma unroll
          for (int j = 0; j < kBatch; ++j) {
            float* d = w_snap + m * snap_stride + shift + e0 + 4LL * (l0 + j * kWorkers);
            st1(d, v[j].x); st1(d + 1, v[j].y); st1(d + 2, v[j].z); st1(d + 3, v[j].w);
          }
        }
      } else {
        for (int j = 0; j < kBatch; ++j) {
          const int l = l0 + j * kWorkers;
          if (l >= kSnapTileElems / 4 || !copy_lane(l)) break;
        }
      }
    }
  }
}

__global__ void __launch_bounds__(kThreads, 1)
k_snapshot_tma(const float* __restrict__ w_now, float* __restrict__ w_snap, long long now_stride,
               long long snap_stride, int M, const SegPlan* __restrict__ gplan,
               const PlanHeader* __restrict__ ghdr, const __grid_constant__ PlanRequest rq,
               int* __restrict__ status, int err_timeout, const __grid_constant__ FragTable T,
               const __grid_constant__ SelectRequest sel) {
  extern __shared__ __align__(128) unsigned char smem_raw[];
  __shared__ __align__(8) unsigned long long full_bar[kSnapStages];
  __shared__ float* dst_of_stage[kSnapStages];
  __shared__ InlinePlan ip;
  __shared__ InlineSelect is;
  PlanView pv;
  if (sel.scores != nullptr) {
    // initiation in one launch: Algorithm 2 first, then the snapshot of what it picked
    select_in_cta(is, sel, T, status);
    PlanRequest mine = rq;
    mine.ids = is.ids;
    mine.n_ids = &is.n;
    mine.snap_offset = sel.pool_offset ? is.pool : nullptr;
    pv = acquire_plan(ip, T, mine, nullptr, nullptr, status);
  } else {
    pv = acquire_plan(ip, T, rq, gplan, ghdr, status);
  }
  if (threadIdx.x == 0) {
    for (int s = 0; s < kSnapStages; ++s) mbar_init(smem_u32(&full_bar[s]), 1);
    asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory");
  }
  __syncthreads();
  SnapshotJob J;
  J.w_now = w_now; J.w_snap = w_snap; J.now_stride = now_stride; J.snap_stride = snap_stride; J.M = M;
  J.status = status; J.err_timeout = err_timeout;
  snapshot_copy(J, pv.seg, pv.hdr, reinterpret_cast<float*>(smem_raw), full_bar, dst_of_stage);
  // the selection's writes to the schedule state, from a copy warp that is done (the DMA thread still has the
  // whole copy ahead of it, so the counter's round trip costs nothing)
  if (sel.scores != nullptr && threadIdx.x == 32) select_commit(is, sel, status);
}

// ---------------------------------------------------------------------------------------------
// Zero delay (w_snap == w_now, the blocking synchronisation of DiLoCo): every stream that is read is
// also written, one byte out per byte in.  At that mix stores from registers fall short (6.3 TB/s); what
// measures best is the snapshot kernel's shape with the arithmetic in the middle: the TMA unit moves
// the tiles in both directions and the consumers update the stage in place in shared memory.
//   loader   : waits until the stage's previous store has read it ("empty"), bulk loads of the tile ("full");
//   consumers: wait on "full", lane into registers, arithmetic, results back into the same lane of the
//              stage, proxy fence, arrive on "done" (one arrival per consumer thread);
//   storer   : waits on "done", bulk stores of the stage to theta_g, momentum and w_now, waits until they
//              have read shared memory, arrives on "empty".
// Loader and storer are single threads of two further warps (one thread doing both jobs: 6.57 against 6.62 TB/s
// at M = 4).  The ring depth per worker count is measured: inplace_stages().
// ---------------------------------------------------------------------------------------------
constexpr int kInplaceThreads = kThreads + 64;

// Stages of the in-place ring per worker count (a stage is M + 2 tiles of 4 KB), measured on B200 with 2 to 6
// stages each (GB/s of the zero-delay step, 100 M parameters per worker; the chosen depth first):
//   M = 1: 6 stages 6453 (5: 6351, 4: 5943)      M = 5: 3 stages 6369 (4: 6011, 2: 5725)
//   M = 2: 4 stages 6413 (5: 6168, 3: 5829)      M = 6: 3 stages 6224 (4: 5967, 2: 5915)
//   M = 3: 4 stages 6282 (3: 6216, 5: 5962)      M = 7: 3 stages 6187 (2: 6080, 4: 5961)
//   M = 4: 3 stages 6501 (4: 6120, 2: 5521)      M = 8: 2 stages 6292 (3: 6165, 4: 6023)
// Loading, updating and storing each hold a stage, so fewer than three serialise the pipeline unless a stage is
// large; beyond about 80 KB the loads in flight crowd out the stores.
__host__ __device__ constexpr int inplace_stages(int M) {
  return M == 1 ? 6 : M <= 3 ? 4 : M <= 7 ? 3 : 2;
}

template <int M>
struct InplaceLayout {
  using L = StageLayout<M, MODE_FUSED, true>;
  static constexpr int kStages = inplace_stages(M);
  static constexpr unsigned kSmemBytes = kStages * L::kStageBytes;
  static_assert(kSmemBytes <= 227 * 1024, "stages do not fit in shared memory");
};

template <int M>
__global__ void __launch_bounds__(kInplaceThreads, 1)
k_outer_inplace(const __grid_constant__ OuterArgs A, const __grid_constant__ FragTable T) {
  using IL = InplaceLayout<M>;
  using L = typename IL::L;
  constexpr int S = IL::kStages;
  extern __shared__ __align__(128) unsigned char smem_raw[];
  float* const stages = reinterpret_cast<float*>(smem_raw);
  __shared__ __align__(8) unsigned long long full_bar[S];
  __shared__ __align__(8) unsigned long long done_bar[S];
  __shared__ __align__(8) unsigned long long empty_bar[S];
  __shared__ volatile int s_fail;
  __shared__ InlinePlan ip;
  const int tid = threadIdx.x;
  const PlanView pv = acquire_plan(ip, T, A.rq, A.plan, A.hdr, A.status);
  const PlanHeader h = pv.hdr;
  if (tid == 0) {
    for (int s = 0; s < S; ++s) {
      mbar_init(smem_u32(&full_bar[s]), 1);
      mbar_init(smem_u32(&done_bar[s]), kThreads);
      mbar_init(smem_u32(&empty_bar[s]), 1);
    }
    s_fail = 0;
    asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory");
  }
  __syncthreads();

  // ------------------------------------------------------------------ loader
  if (tid == kThreads) {
    TileWalker tw(pv.seg, h.n_seg);
    int k = 0;   // staged tiles issued so far
    for (int tile = blockIdx.x; tile < h.total_tiles; tile += gridDim.x) {
      tw.seek(tile);
      const long long e0 = tw.tile_start(tile);
      if (!tw.interior(e0)) continue;
      const int s = k % S;
      if (k >= S && (s_fail || !mbar_wait_bounded(smem_u32(&empty_bar[s]), ((k / S) - 1) & 1))) {
        record_status(A.status, A.err_timeout);
        s_fail = 1;
        // the loads already issued must land before this CTA's shared memory can go to another one
        for (int i = (k > S ? k - S : 0); i < k; ++i) mbar_wait_bounded(smem_u32(&full_bar[i % S]), (i / S) & 1);
        return;
      }
      const unsigned bar = smem_u32(&full_bar[s]);
      float* st = stages + (size_t)s * L::kLoaded * kTileElems;
      mbar_expect_tx(bar, L::kLoaded * kTileBytes);
#pragma unroll
      for (int m = 0; m < M; ++m)
        bulk_load(smem_u32(st + (L::kNow + m) * kTileElems), A.w_now + m * A.now_stride + e0, kTileBytes, bar);
      bulk_load(smem_u32(st + L::kGlobal * kTileElems), A.theta_g + e0, kTileBytes, bar);
      bulk_load(smem_u32(st + L::kMomentum * kTileElems), A.momentum + e0, kTileBytes, bar);
      ++k;
    }
    return;
  }
  // ------------------------------------------------------------------ storer
  if (tid == kThreads + 32) {
    TileWalker tw(pv.seg, h.n_seg);
    const unsigned long long policy = l2_evict_first_policy();
    int k = 0;   // staged tiles stored so far
    for (int tile = blockIdx.x; tile < h.total_tiles; tile += gridDim.x) {
      tw.seek(tile);
      const long long e0 = tw.tile_start(tile);
      if (!tw.interior(e0)) continue;
      const int s = k % S;
      if (s_fail || !mbar_wait_bounded(smem_u32(&done_bar[s]), (k / S) & 1)) {
        record_status(A.status, A.err_timeout);
        s_fail = 1;
        break;
      }
      const float* st = stages + (size_t)s * L::kLoaded * kTileElems;
      bulk_store(A.theta_g + e0, smem_u32(st + L::kGlobal * kTileElems), kTileBytes, policy);
      bulk_store(A.momentum + e0, smem_u32(st + L::kMomentum * kTileElems), kTileBytes, policy);
#pragma unroll
      for (int m = 0; m < M; ++m)
        bulk_store(A.w_now + m * A.now_stride + e0, smem_u32(st + (L::kNow + m) * kTileElems), kTileBytes, policy);
      bulk_commit();
      bulk_wait_read_n<0>();                    // the stores have read the stage: it may be loaded again
      mbar_arrive(smem_u32(&empty_bar[s]));
      ++k;
    }
    bulk_wait_all();    // shared memory must outlive the last stores (also after a failed wait)
    return;
  }
  if (tid >= kThreads) return;

  // ------------------------------------------------------------------ consumers
  SlotAccumulator sa(kThreads / 32);
  TileWalker tw(pv.seg, h.n_seg);
  int k = 0;
  bool failed = false;
  for (int tile = blockIdx.x; tile < h.total_tiles; tile += gridDim.x) {
    if (tw.seek(tile) && A.partial) sa.advance(tw.sp.slot, A.partial);
    const long long e0 = tw.tile_start(tile);
    if (!tw.interior(e0)) {
      sa.acc += ragged_tile<M, MODE_FUSED, true, 1>(A, tw.sp, e0 + 4LL * tid);
      continue;
    }
    const int s = k % S;
    const bool landed = !s_fail && mbar_wait_bounded(smem_u32(&full_bar[s]), (k / S) & 1);
    if (!__all_sync(0xffffffffu, landed)) {   // per-warp verdict, as in k_outer_tma
      record_status(A.status, A.err_timeout);
      s_fail = 1;
      failed = true;
      break;
    }
    float* st = stages + (size_t)s * L::kLoaded * kTileElems;
    auto slot = [&](int idx) -> float4& { return reinterpret_cast<float4*>(st + idx * kTileElems)[tid]; };
    Lane<M, MODE_FUSED, true> ln;
    ln.thg = slot(L::kGlobal);
    ln.u = slot(L::kMomentum);
#pragma unroll
    for (int m = 0; m < M; ++m) ln.b[m] = slot(L::kNow + m);
    ln.compute(A, sa.acc);
    slot(L::kGlobal) = ln.thg;
    slot(L::kMomentum) = ln.u;
#pragma unroll
    for (int m = 0; m < M; ++m) slot(L::kNow + m) = ln.out(m);
    if (A.delta_out) st4(A.delta_out + e0 + 4LL * tid, ln.delta);
    asm volatile("fence.proxy.async.shared::cta;" ::: "memory");   // make the lane visible to the bulk store
    mbar_arrive(smem_u32(&done_bar[s]));
    ++k;
  }
  if (failed) return;     // warp-uniform by construction
  if (A.partial) {
    sa.finish(h.n_ids, A.partial);
    finalize_epilogue(ip, A.fin, h, A.partial, kThreads / 32, A.status);
  }
}

// ---------------------------------------------------------------------------------------------
// Self-test of the bounded wait: one thread waits on a barrier that nothing will ever complete.
// The loop ends after `polls` polls, the kernel records the timeout code and returns, and the
// context stays usable - this is the path a stalled copy would take in the kernels above.
// ---------------------------------------------------------------------------------------------
static __global__ void k_selftest_bounded_wait(int polls, int* __restrict__ status, int err_timeout) {
  __shared__ __align__(8) unsigned long long bar;
  if (threadIdx.x != 0) return;
  mbar_init(smem_u32(&bar), 1);
  asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory");
  if (!mbar_wait_limit(smem_u32(&bar), 0, polls)) record_status(status, err_timeout);
}

}  // namespace cocodc

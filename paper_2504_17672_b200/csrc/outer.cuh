// Arithmetic of the outer synchronisation step and the kernels that do not stage through
// shared memory: the generic-M fallback and the stand-alone sum of squares.
//
// Per element the step reads every worker's recorded and current value, the global state and the
// momentum once, keeps pseudo-gradient, mean, Nesterov update, delay compensation and merge in
// registers, and writes each output once (Eq. 1-7, Eq. 3).  The sum of squares of the mean
// pseudo-gradient (Eq. 10) is collected on the way.  Nothing here is a contraction: every kernel
// is bound by HBM bandwidth.
//
// The main kernel for the instantiated worker counts lives in outer_tma.cuh and uses the
// per-lane code (struct Lane, ragged_lane) defined here.
#pragma once

#include "plan.cuh"

namespace cocodc {

constexpr int kThreads = 256;        // consumer threads per CTA; a tile is kThreads lanes of 16 bytes
constexpr int kTileElems = 4 * kThreads;

// MODE_FUSED_RECV: as MODE_FUSED, but Eq. 1's sum over ALL workers arrives ready-made (delta_in, the result
// of the all-reduce when every device holds only some of the workers) and is divided by the total count.
// MODE_PSEUDO_SUM: only S1 and the local part of S2 -- the sum over this device's workers of
// theta^m_{p,t_p} - theta^g goes to delta_out (what the all-reduce of Section 2.1 then sums); nothing else is touched.
enum : int { MODE_FUSED = 0, MODE_OUTER_ONLY = 1, MODE_MERGE_ONLY = 2, MODE_FUSED_RECV = 3, MODE_PSEUDO_SUM = 4 };
__host__ __device__ constexpr bool mode_updates_global(int mode) { return mode == MODE_FUSED || mode == MODE_OUTER_ONLY || mode == MODE_FUSED_RECV; }
__host__ __device__ constexpr bool mode_merges(int mode) { return mode == MODE_FUSED || mode == MODE_MERGE_ONLY || mode == MODE_FUSED_RECV; }

constexpr int kMaxRecv = 8;          // buffers of partial sums a received-sum step can add up

struct OuterArgs {
  float* w_now;             // [M][now_stride]
  const float* w_snap;      // [M][snap_stride]
  long long now_stride;
  long long snap_stride;
  float* theta_g;           // in/out (MODE_MERGE_ONLY: read only, the new global state)
  float* momentum;          // in/out
  float* delta_out;         // optional
  const float* delta_in[kMaxRecv];   // MODE_FUSED_RECV: sums of pseudo-gradients, one buffer per contributing device
  int n_recv;               // how many of them (added in this order, so every device that lists them alike gets the same bits)
  const SegPlan* plan;      // plan in global memory (written by k_plan / k_plan_chunk), or nullptr: every CTA
  const PlanHeader* hdr;    //   expands `rq` itself in its prologue
  PlanRequest rq;
  Finalize fin;             // what the last warp does with the sums of squares (fin.ticket == nullptr: nothing)
  double* partial;          // nullptr: no score accumulation
  int* status;              // device status word
  int err_timeout;          // code recorded when a bounded wait runs out
  int M;                    // runtime worker count (used by the generic kernel and scalar paths)
  float eta, mu;            // outer learning rate, Nesterov momentum
  float c1, c2;             // target = G + c1*d + c2*d*d*D
  float alpha, one_minus_alpha;
  float Mf;                 // divisor of Eq. 1 as float: M, or the total worker count in MODE_FUSED_RECV
  float inv_M;              // its reciprocal, correctly rounded (exact when the divisor is a power of two)
  int M_pow2;               // 1 if the divisor is a power of two
  int ring_slots;           // k_outer_ring: chunks in its shared-memory ring
};

// ---- memory access helpers -------------------------------------------------
// Every byte is used exactly once per launch. Direct loads are marked streaming (evict-first in L2). Register
// stores are ordinary write-back stores: marked streaming they made the fused step about 1 % slower at every
// worker count (the dirty lines then leave L2 in the order the hint imposes rather than the order the memory
// controller would batch them in); .cg and .wt stores time like the ordinary ones.
__device__ __forceinline__ float4 ld4(const float* p) { return __ldcs(reinterpret_cast<const float4*>(p)); }
__device__ __forceinline__ void st4(float* p, float4 v) { *reinterpret_cast<float4*>(p) = v; }
__device__ __forceinline__ float ld1(const float* p) { return __ldcs(p); }
__device__ __forceinline__ void st1(float* p, float v) { *p = v; }

// The received sum of Eq. 1: the listed buffers added in order (a single buffer when a collective has already
// summed them; one buffer per device when they are read straight from the peers' memory).
__device__ __forceinline__ float received_sum1(const OuterArgs& A, long long e) {
  float s = ld1(A.delta_in[0] + e);
  for (int r = 1; r < A.n_recv; ++r) s = __fadd_rn(s, ld1(A.delta_in[r] + e));
  return s;
}
__device__ __forceinline__ float4 add4(float4 a, const float4& b) {
  a.x = __fadd_rn(a.x, b.x); a.y = __fadd_rn(a.y, b.y); a.z = __fadd_rn(a.z, b.z); a.w = __fadd_rn(a.w, b.w);
  return a;
}
__device__ __forceinline__ float4 received_sum4(const OuterArgs& A, long long e) {
  float4 s = ld4(A.delta_in[0] + e);
  for (int r = 1; r < A.n_recv; ++r) s = add4(s, ld4(A.delta_in[r] + e));
  return s;
}

// ---- the arithmetic of one element -----------------------------------------
// S2.  The sum of the workers' pseudo-gradients divided by M (Eq. 1).  The IEEE division routine branches
// on zero or tiny numerators, and that data-dependent slow path costs bandwidth as soon as many elements
// have converged (every pseudo-gradient is zero right after a blocking synchronisation), so no instruction
// here divides.  For a power of two the product with 1/M is the correctly rounded quotient, bit for bit.
// For any other M: q0 = RN(sum * RN(1/M)) is within an ulp of the quotient, the residual sum - q0*M comes
// exactly out of one fused multiply-add, and q0 + residual * RN(1/M) rounds to the correctly rounded
// quotient (the usual correction step of division by iteration; it holds while the residual does not
// underflow, i.e. for |sum| above about 2^-100, below which the result may differ by one unit of its last
// place).  Non-finite sums keep q0, which is what the division would give.
__device__ __forceinline__ float quotient_by_count(float sum, float count, float inv_count) {
  const float q0 = __fmul_rn(sum, inv_count);
  const float r = __fmaf_rn(-q0, count, sum);
  const float q = __fmaf_rn(r, inv_count, q0);
  return (r != 0.0f && fabsf(q0) <= 3.402823466e+38f) ? q : q0;   // r == 0: q0 is exact (keeps the sign of a zero)
}
template <int M>
__device__ __forceinline__ float mean_of_sum(float sum, const OuterArgs& A) {
  if constexpr (M > 0 && (M & (M - 1)) == 0) return __fmul_rn(sum, 1.0f / (float)M);
  else if constexpr (M > 0) return quotient_by_count(sum, (float)M, 1.0f / (float)M);
  else return A.M_pow2 ? __fmul_rn(sum, A.inv_M) : quotient_by_count(sum, A.Mf, A.inv_M);
}

// S3.  u' = mu*u + Delta, G = thg + eta*(Delta + mu*u') (Eq. 2, Nesterov).
__device__ __forceinline__ void outer_update(float Delta, float thg, float u, const OuterArgs& A,
                                             float& u_new, float& G) {
  u_new = __fmaf_rn(A.mu, u, Delta);
  const float t = __fmaf_rn(A.mu, u_new, Delta);
  G = __fmaf_rn(A.eta, t, thg);
}

// S4-S5.  d = a - b is the local change over the overlap (tau times Eq. 4's rate), D = G - b the
// divergence of Eq. 5; Eq. 6-7 collapse to target = G + c1*d + c2*d*d*D with c2 = +-lambda/(tau*H);
// then Eq. 3's blend.
__device__ __forceinline__ float merged(float a, float b, float G, const OuterArgs& A) {
  const float d = __fsub_rn(a, b);
  const float D = __fsub_rn(G, b);
  const float lin = __fmaf_rn(A.c1, d, G);
  const float target = __fmaf_rn(__fmul_rn(__fmul_rn(A.c2, d), d), D, lin);
  return __fmaf_rn(A.alpha, target, __fmul_rn(A.one_minus_alpha, a));
}

__device__ __forceinline__ float& comp(float4& v, int k) { return reinterpret_cast<float*>(&v)[k]; }
__device__ __forceinline__ float comp(const float4& v, int k) { return reinterpret_cast<const float*>(&v)[k]; }

// One scalar element, any M (ragged edges, unaligned snapshot layouts, worker counts not instantiated).
template <int MODE, bool SAME>
__device__ __forceinline__ void scalar_element(const OuterArgs& A, long long e, long long snap_e, float& sq) {
  const int M = A.M;
  const float thg = ld1(A.theta_g + e);
  if (MODE == MODE_PSEUDO_SUM) {
    float sum = 0.f;
    for (int m = 0; m < M; ++m) sum = __fadd_rn(sum, __fsub_rn(ld1(A.w_snap + m * A.snap_stride + snap_e), thg));
    st1(A.delta_out + e, sum);
    return;
  }
  float G;
  if (MODE == MODE_MERGE_ONLY) {
    G = thg;
  } else {
    float sum = 0.f;
    if (MODE == MODE_FUSED_RECV) {
      sum = received_sum1(A, e);
    } else {
      for (int m = 0; m < M; ++m) sum = __fadd_rn(sum, __fsub_rn(ld1(A.w_snap + m * A.snap_stride + snap_e), thg));
    }
    const float Delta = mean_of_sum<0>(sum, A);
    float u_new;
    outer_update(Delta, thg, ld1(A.momentum + e), A, u_new, G);
    sq = __fmaf_rn(Delta, Delta, sq);   // the lane's squares add up in fp32, element order, as in Lane::compute
    st1(A.theta_g + e, G);
    st1(A.momentum + e, u_new);
    if (A.delta_out) st1(A.delta_out + e, Delta);
  }
  if (mode_merges(MODE)) {
    for (int m = 0; m < M; ++m) {
      const float b = ld1(A.w_snap + m * A.snap_stride + snap_e);
      const float a = SAME ? b : ld1(A.w_now + m * A.now_stride + e);
      st1(A.w_now + m * A.now_stride + e, merged(a, b, G, A));
    }
  }
}

// Registers of one 16-byte lane (four consecutive elements) of every stream.
// compute() works in place: afterwards thg holds G, u holds u', delta holds Delta (on entry, in
// MODE_FUSED_RECV, the received sum) and the merged
// local parameters sit in out(m) (= a[m], or b[m] when the snapshot is the current state).
template <int M, int MODE, bool SAME>
struct Lane {
  static constexpr bool kHasNow = mode_merges(MODE) && !SAME;
  float4 b[M];
  float4 a[kHasNow ? M : 1];
  float4 thg;
  float4 u;
  float4 delta;

  __device__ __forceinline__ float4& out(int m) {
    if constexpr (kHasNow) return a[m];
    else return b[m];
  }

  __device__ __forceinline__ void load(const OuterArgs& A, long long e, long long snap_e) {
    thg = ld4(A.theta_g + e);
    if (mode_updates_global(MODE)) u = ld4(A.momentum + e);
    if (MODE == MODE_FUSED_RECV) delta = received_sum4(A, e);
#pragma unroll
    for (int m = 0; m < M; ++m) b[m] = ld4(A.w_snap + m * A.snap_stride + snap_e);
    if (kHasNow) {
#pragma unroll
      for (int m = 0; m < M; ++m) a[m] = ld4(A.w_now + m * A.now_stride + e);
    }
  }

  // The same lane when the recorded values sit at a place that is not 16-byte compatible with the native one
  // (snap_e is any element index): they come in as four 4-byte loads per worker, everything else as vectors.
  __device__ __forceinline__ void load_shifted(const OuterArgs& A, long long e, long long snap_e) {
    thg = ld4(A.theta_g + e);
    if (mode_updates_global(MODE)) u = ld4(A.momentum + e);
    if (MODE == MODE_FUSED_RECV) delta = received_sum4(A, e);
#pragma unroll
    for (int m = 0; m < M; ++m) {
      const float* p = A.w_snap + m * A.snap_stride + snap_e;
      b[m] = make_float4(ld1(p), ld1(p + 1), ld1(p + 2), ld1(p + 3));
    }
    if (kHasNow) {
#pragma unroll
      for (int m = 0; m < M; ++m) a[m] = ld4(A.w_now + m * A.now_stride + e);
    }
  }

  __device__ __forceinline__ void compute(const OuterArgs& A, double& acc) {
    if (MODE == MODE_PSEUDO_SUM) {
#pragma unroll
      for (int k = 0; k < 4; ++k) {
        const float t = comp(thg, k);
        float sum = __fsub_rn(comp(b[0], k), t);
#pragma unroll
        for (int m = 1; m < M; ++m) sum = __fadd_rn(sum, __fsub_rn(comp(b[m], k), t));
        comp(delta, k) = sum;
      }
    }
    if (mode_updates_global(MODE)) {
      float sq = 0.f;
#pragma unroll
      for (int k = 0; k < 4; ++k) {
        const float t = comp(thg, k);
        float Delta;
        if (MODE == MODE_FUSED_RECV) {
          Delta = mean_of_sum<0>(comp(delta, k), A);      // delta holds the received sum on entry
        } else {
          float sum = __fsub_rn(comp(b[0], k), t);
#pragma unroll
          for (int m = 1; m < M; ++m) sum = __fadd_rn(sum, __fsub_rn(comp(b[m], k), t));
          Delta = mean_of_sum<M>(sum, A);
        }
        float u_new, G;
        outer_update(Delta, t, comp(u, k), A, u_new, G);
        comp(delta, k) = Delta; comp(u, k) = u_new; comp(thg, k) = G;
        sq = __fmaf_rn(Delta, Delta, sq);
      }
      acc += (double)sq;
    }
    if (mode_merges(MODE)) {
#pragma unroll
      for (int m = 0; m < M; ++m) {
#pragma unroll
        for (int k = 0; k < 4; ++k) {
          const float bb = comp(b[m], k);
          const float aa = kHasNow ? comp(a[m], k) : bb;
          comp(out(m), k) = merged(aa, bb, comp(thg, k), A);
        }
      }
    }
  }

  __device__ __forceinline__ void store(const OuterArgs& A, long long e) {
    if (MODE == MODE_PSEUDO_SUM) st4(A.delta_out + e, delta);
    if (mode_updates_global(MODE)) {
      st4(A.theta_g + e, thg);
      st4(A.momentum + e, u);
      if (A.delta_out) st4(A.delta_out + e, delta);
    }
    if (mode_merges(MODE)) {
#pragma unroll
      for (int m = 0; m < M; ++m) st4(A.w_now + m * A.now_stride + e, out(m));
    }
  }
};

// A full lane whose recorded values sit at a place that is not 16-byte compatible.  Kept out of line: inlined
// into the staged kernels it cost their main loop 1.5 % of bandwidth (6.71 -> 6.61 TB/s on the 1B shape).
template <int M, int MODE, bool SAME>
__device__ __noinline__ double shifted_lane(const OuterArgs& A, long long e, long long snap_e) {
  Lane<M, MODE, SAME> L;
  double sumsq = 0.0;       // this lane's contribution to the sum of squares
  L.load_shifted(A, e, snap_e);
  L.compute(A, sumsq);
  L.store(A, e);
  return sumsq;
}

// One lane at element e of a segment, straight from global memory: a full lane goes through registers as a
// vector (its recorded values by element when their place is not 16-byte compatible), a partial lane element
// by element.  M = 0: always by element.
template <int M, int MODE, bool SAME>
__device__ __forceinline__ void ragged_lane(const OuterArgs& A, const SegPlan& sp, long long e, double& acc) {
  const long long seg_end = sp.off + sp.len;
  const long long snap_shift = sp.snap_off - sp.off;   // snapshot index = native index + shift
  if (e >= seg_end) return;
  if constexpr (M > 0) {
    if (sp.vec_ok && e >= sp.off && e + 4 <= seg_end) {
      Lane<M, MODE, SAME> L;
      L.load(A, e, e + snap_shift);
      L.compute(A, acc);
      L.store(A, e);
      return;
    }
    if (!SAME && e >= sp.off && e + 4 <= seg_end) {
      acc += shifted_lane<M, MODE, SAME>(A, e, e + snap_shift);
      return;
    }
  }
  // Element by element, with the lane's sum of squares formed exactly as the vector path forms it (fp32 over
  // the lane's elements in order, then one conversion): every kernel that walks the same tiles then arrives at
  // the same fragment norms bit for bit, whichever path its lanes took.
  float sq = 0.f;
  for (int k = 0; k < 4; ++k) {
    const long long ee = e + k;
    if (ee >= sp.off && ee < seg_end) scalar_element<MODE, SAME>(A, ee, ee + snap_shift, sq);
  }
  if (mode_updates_global(MODE)) acc += (double)sq;
}

// A whole ragged tile of one thread (U lanes, kThreads lanes apart), out of line: these tiles are the exception
// (segment edges, pool places that are not 16-byte compatible), and kept inline their code sat in the middle of
// the staged kernels' main loop.  The segment entry travels by value so that the caller's copy stays in
// registers.  Returns the thread's contribution to the sum of squares.
template <int M, int MODE, bool SAME, int U>
__device__ __noinline__ double ragged_tile(const OuterArgs& A, const SegPlan sp, long long e_first) {
  double acc = 0.0;
#pragma unroll
  for (int v = 0; v < U; ++v) ragged_lane<M, MODE, SAME>(A, sp, e_first + 4LL * (v * kThreads), acc);
  return acc;
}

// Walks the tiles of one CTA (tile = blockIdx.x + i*gridDim.x) and keeps the segment they fall in.
struct TileWalker {
  const SegPlan* plan;
  int n_seg;
  int seg = 0;
  int loaded = -1;
  int tile_elems;      // elements per tile of this launch (the plan was built with tile_elems / 4 lanes per tile)
  SegPlan sp;

  __device__ __forceinline__ TileWalker(const SegPlan* p, int n, int tile_elems_ = kTileElems)
      : plan(p), n_seg(n), tile_elems(tile_elems_) {}
  // returns true if the segment changed
  __device__ __forceinline__ bool seek(int tile) {
    while (seg + 1 < n_seg && tile >= plan[seg + 1].first_tile) ++seg;
    if (seg == loaded) return false;
    sp = plan[seg];
    loaded = seg;
    return true;
  }
  __device__ __forceinline__ long long tile_start(int tile) const {   // first element (16-byte aligned)
    return sp.abase + (long long)(tile - sp.first_tile) * tile_elems;
  }
  // the whole tile lies inside the segment and every stream is 16-byte aligned there
  __device__ __forceinline__ bool interior(long long e_tile) const {
    return sp.vec_ok && e_tile >= sp.off && e_tile + tile_elems <= sp.off + sp.len;
  }
};

// Generic kernel: any worker count, every lane through ragged_lane<0> (element loop with runtime M;
// the second pass over the recorded values hits in cache).
template <int MODE, bool SAME>
__global__ void __launch_bounds__(kThreads)
k_outer_generic(const __grid_constant__ OuterArgs A, const __grid_constant__ FragTable T) {
  __shared__ InlinePlan ip;
  const PlanView pv = acquire_plan(ip, T, A.rq, A.plan, A.hdr, A.status);
  const PlanHeader h = pv.hdr;
  SlotAccumulator sa(kThreads / 32);
  TileWalker tw(pv.seg, h.n_seg);
  for (int tile = blockIdx.x; tile < h.total_tiles; tile += gridDim.x) {
    if (tw.seek(tile) && A.partial) sa.advance(tw.sp.slot, A.partial);
    ragged_lane<0, MODE, SAME>(A, tw.sp, tw.tile_start(tile) + 4LL * threadIdx.x, sa.acc);
  }
  if (A.partial) {
    sa.finish(h.n_ids, A.partial);
    finalize_epilogue_cta(ip, A.fin, h, A.partial, kThreads / 32, A.status);
  }
}

// ---------------------------------------------------------------------------
// S6 stand-alone: sums of squares of an N-sized vector over the planned tiles.
// ---------------------------------------------------------------------------
// The accumulation loop, out of line (its registers then do not depend on the prologue and epilogue around it).
template <int U>
static __device__ __noinline__ void sumsq_tiles(const float* __restrict__ x, const SegPlan* plan, const PlanHeader h,
                                                double* __restrict__ partial) {
  constexpr int LPT = kThreads * U;
  SlotAccumulator sa(kThreads / 32);
  int seg = 0, seg_loaded = -1;
  SegPlan sp;
  for (int tile = blockIdx.x; tile < h.total_tiles; tile += gridDim.x) {
    while (seg + 1 < h.n_seg && tile >= plan[seg + 1].first_tile) ++seg;
    if (seg != seg_loaded) { sp = plan[seg]; seg_loaded = seg; sa.advance(sp.slot, partial); }
    const long long e_tile = sp.abase + 4LL * (long long)(tile - sp.first_tile) * LPT;
    const long long seg_end = sp.off + sp.len;
    if (e_tile >= sp.off && e_tile + 4LL * LPT <= seg_end) {
      float4 v[U];
#pragma unroll
      for (int j = 0; j < U; ++j) v[j] = ld4(x + e_tile + 4LL * (j * kThreads + threadIdx.x));
#pragma unroll
      for (int j = 0; j < U; ++j) {
        float sq = __fmul_rn(v[j].x, v[j].x);
        sq = __fmaf_rn(v[j].y, v[j].y, sq);
        sq = __fmaf_rn(v[j].z, v[j].z, sq);
        sq = __fmaf_rn(v[j].w, v[j].w, sq);
        sa.acc += (double)sq;
      }
    } else {
      for (int j = 0; j < U; ++j) {
        const long long e = e_tile + 4LL * (j * kThreads + threadIdx.x);
        if (e >= seg_end) break;
        for (int k = 0; k < 4; ++k) {
          const long long ee = e + k;
          if (ee >= sp.off && ee < seg_end) { const float t = ld1(x + ee); sa.acc += (double)__fmul_rn(t, t); }
        }
      }
    }
  }
  sa.finish(h.n_ids, partial);
}

template <int U>
__global__ void __launch_bounds__(kThreads)
k_sumsq(const float* __restrict__ x, const SegPlan* __restrict__ gplan, const PlanHeader* __restrict__ ghdr,
        const __grid_constant__ PlanRequest rq, const __grid_constant__ Finalize fin,
        double* __restrict__ partial, int* __restrict__ status, const __grid_constant__ FragTable T) {
  __shared__ InlinePlan ip;
  const PlanView pv = acquire_plan(ip, T, rq, gplan, ghdr, status);
  sumsq_tiles<U>(x, pv.seg, pv.hdr, partial);
  finalize_epilogue_cta(ip, fin, pv.hdr, partial, kThreads / 32, status);
}

}  // namespace cocodc

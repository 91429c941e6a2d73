// dmx_kernels.cuh — device code of the fused gradient step (sm_100a).
//
// One pass over the K gradient streams and the three fp32 state streams does, per parameter j:
//   g_j  = sum_k w_k x_kj                       (batch-size-weighted aggregate, w_k = b_k/B)
//   d_j  = sum_k b_k (x_kj - g_j)^2             (spread of the workers around it)
//   q_k += x_kj^2,  N_s += g_j^2,  V_s += d_j,  c += g_j a_j,  pp += a_j^2
//   m_j  = beta m_j + g_j,  theta_j -= lr m_j,  a_j = g_j            (SGD with momentum), or
//   m_j  = b1 m_j + (1-b1) g_j,  v_j = b2 v_j + (1-b2) g_j^2,
//   theta_j -= lr mhat_j / (sqrt(vhat_j) + eps),  a_j = g_j            (Adam, bias-corrected)
// The sums over k use the shifted one-pass form around a pivot worker (the one with the
// largest batch): with e_k = x_k - x_pivot,  g = x_pivot + sum w_k e_k  and
// d = sum b_k e_k^2 - B (sum w_k e_k)^2. Identical workers give d = 0 exactly, and the
// cancellation is between noise-sized terms only. The arithmetic runs on pairs of fp32
// values with the packed f32x2 instructions of sm_100 (each lane IEEE fp32, round to nearest).
//
// With fp32 gradients the per-parameter recurrence itself (aggregate -> momentum -> parameter) is
// carried in fp64 and rounded once at each store, as its definition says:
//   g = (sum_k b_k x_k) / B,  m' = beta m + g,  theta' = theta - lr m'.
// The stored fp32 values are then the correctly rounded ones in all but about one case in 2^29,
// so a long run stays on the trajectory of the definition bit for bit; with an fp32 aggregate
// every step left a last-bit difference in g that the momentum's and the parameters' own
// roundings turned into whole-ulp differences, amplified by 1/(1 - beta) and accumulated over
// the steps (1e-4 of a parameter's forward-error scale after 100 steps). The statistics keep
// the fp32 shifted sums. With bf16 gradients (tolerance 4e-3) the aggregate stays fp32.
//
// Work layout. The parameter range is cut into tiles of T elements, taken in groups of R
// consecutive tiles. The unit of work is a chunk: a few groups, interleaved with the other
// chunks of its wave (chunk l of a wave of n chunks holds groups first+l, first+l+n, ...), so
// that the CTAs working on one wave sweep a compact window of every stream (DRAM sees a few
// dozen linear sweeps instead of thousands of scattered 4 KB reads). The chunk list is fixed by
// the host; waves shrink towards the end of the range. The pipelined kernel hands chunks to its
// CTAs dynamically (an atomic counter): SMs do not all stream at the same rate, and a static
// split left the fast ones idle for 3-12 % of the kernel.
//
// Reductions are deterministic: per-thread fp32 partials over a chunk, warp shuffles, a
// fixed-order sum over the warps, one scratch row per chunk and one scratch slot per
// (chunk, run of tiles in one segment), then an fp64 fixed-order second level in the
// finalize kernel. A chunk's sums do not depend on which CTA computes it, so results are
// bitwise reproducible under the dynamic schedule. There are no floating-point atomics and no
// waits between CTAs.
#pragma once
#include <cuda_runtime.h>
#include <stdint.h>

namespace dmx {

constexpr int kMaxK = 64;
constexpr int kSegBuf = 32;                 // segment partials a CTA buffers in shared memory between drains
constexpr int kTileBoundaryBit = 1 << 30;   // flag in the per-tile segment table

// Error word of a handle: bit 0 = a bounded wait ran out, bit 1 = an index was out of range.
constexpr unsigned kErrWait = 1u, kErrBounds = 2u;

// Checked build (-DDMX_DEBUG): every index into the tables and the scratch is tested against its
// range; a violation sets kErrBounds in the handle's error word (reported as DMX_FLAG_BOUNDS in
// the state vector) and the access is skipped. Nothing traps. In the normal build the test
// folds to `true`.
#ifdef DMX_DEBUG
__device__ __forceinline__ bool in_range(unsigned* err, long long i, long long n) {
  if (i >= 0 && i < n) return true;
  atomicOr(err, kErrBounds);
  return false;
}
#define DMX_IN_RANGE(err, i, n) (::dmx::in_range((err), (long long)(i), (long long)(n)))
#else
#define DMX_IN_RANGE(err, i, n) (true)
#endif

// Arguments of one step; passed by value as a __grid_constant__ kernel parameter, so a step
// needs no host-to-device copy. Worker arrays are in processing order (pivot first).
struct StepArgs {
  const void* grad[kMaxK];
  float w[kMaxK];        // b_k / B
  float bf[kMaxK];       // b_k
  double bd[kMaxK];      // b_k (fp32 gradients: the fp64 aggregate)
  double rB, lr64, beta64;   // 1/B, and lr and beta widened exactly
  float* params;
  float* momentum;
  float* prev;
  float* second;         // Adam's second-moment estimate v (Adam kernels only)
  float lr, beta, Bf;    // beta is the momentum coefficient, or Adam's beta1
  float beta2, eps, omb1, omb2, c1, c2;   // Adam: beta2, eps, 1-beta1, 1-beta2, 1/(1-beta1^t), 1/(1-beta2^t)
  int K, S;
  int64_t P;
  int tile_group;              // R: consecutive tiles per group
  int nchunks;
  unsigned* next_chunk;        // dynamic schedule: the draw counter (zero at launch; the finalize kernel zeroes it again)
  const int64_t* seg_off;      // S+1
  const int32_t* tile_seg;     // ntiles: segment of the tile's first element; kTileBoundaryBit set
                               //         when a segment boundary lies strictly inside the tile
  const int32_t* chunk_tile0;  // nchunks: first tile of the chunk
  const int32_t* chunk_ntiles; // nchunks: tiles in the chunk
  const int32_t* chunk_stride; // nchunks: tiles between the starts of the chunk's successive groups
  const int32_t* chunk_slot0;  // nchunks: index of the chunk's first (V,N) entry in slot_dest
  const int32_t* slot_dest;    // nslots: where entry e of the step goes in `slots` (entries in the order the chunks emit them)
  float* rows;                 // (K+4) x nchunks, one column after the other: q_k..., c, pp, and (Adam) su, su2
  float2* slots;               // nslots: (V partial, N partial), grouped by segment, each group in entry order
  unsigned* err;               // bit 0: a bounded wait gave up; bit 1 (checked build): an index was out of range
  int ntiles, nslots;          // table sizes (range checks of the checked build)
};

struct FinalArgs {
  int K, S, nchunks, nunits;
  int adam;                    // 1: also emit the optimizer-normalised statistics (columns K+2, K+3)
  double P;
  int orig[kMaxK];             // processing slot -> caller's worker index
  double b[kMaxK];             // batch sizes, processing order
  double B;
  const float* rows;
  const float2* slots;
  const int32_t* seg_ptr;      // S+1: the partials of segment s are slots[seg_ptr[s] .. seg_ptr[s+1])
  const int32_t* unit_lo;      // nunits: a unit is a run slots[unit_lo .. unit_hi) of one segment,
  const int32_t* unit_hi;      //         at most kFinalPart slots long
  int nslots;
  const int32_t* seg_unit_ptr; // S+1: units of segment s are [seg_unit_ptr[s], seg_unit_ptr[s+1])
  double2* segpart;            // nunits: (V, N) of each unit
  double* colsum;              // K+4
  unsigned* ticket;
  unsigned* err;
  unsigned* next_chunk;        // the fused pass's draw counter, zeroed here for the next step
  float* out_state;
  double* partials;            // not null: emit the raw fp64 sums of this parameter shard instead of out_state
};

// Raw sums of a step over a parameter range, as dmx_step_partial emits them (K + 5 + 2 S doubles):
// q_k in the caller's worker order [K], <g,a>, |a|^2, Adam's sum and sum of squares of ghat (0
// otherwise), Vraw_s [S], N_s [S], and a word that is non-zero if a bounded wait ran out.
// Shards of one problem add up entry by entry.
struct DeriveArgs {
  int K, S, adam;
  double P, B;
  double b[kMaxK];             // batch sizes, caller's order
  const double* partials;
  float* out_state;
};

typedef unsigned long long u64;

// ---- packed fp32 pairs ---------------------------------------------------------------------
__device__ __forceinline__ u64 pk(uint32_t lo, uint32_t hi) {
  u64 r; asm("mov.b64 %0, {%1,%2};" : "=l"(r) : "r"(lo), "r"(hi)); return r;
}
__device__ __forceinline__ u64 pkf(float lo, float hi) { return pk(__float_as_uint(lo), __float_as_uint(hi)); }
__device__ __forceinline__ void upk(u64 v, float& lo, float& hi) {
  uint32_t a, b; asm("mov.b64 {%0,%1}, %2;" : "=r"(a), "=r"(b) : "l"(v));
  lo = __uint_as_float(a); hi = __uint_as_float(b);
}
__device__ __forceinline__ u64 fma2(u64 a, u64 b, u64 c) {
  u64 d; asm("fma.rn.f32x2 %0, %1, %2, %3;" : "=l"(d) : "l"(a), "l"(b), "l"(c)); return d;
}
__device__ __forceinline__ u64 add2(u64 a, u64 b) {
  u64 d; asm("add.rn.f32x2 %0, %1, %2;" : "=l"(d) : "l"(a), "l"(b)); return d;
}
__device__ __forceinline__ u64 mul2(u64 a, u64 b) {
  u64 d; asm("mul.rn.f32x2 %0, %1, %2;" : "=l"(d) : "l"(a), "l"(b)); return d;
}

// i-th tile of a chunk whose first tile is t0 and whose groups start `stride` tiles apart
__device__ __forceinline__ int tile_of(const StepArgs& A, int t0, int stride, int i) {
  const int g = i / A.tile_group;
  return t0 + g * stride + (i - g * A.tile_group);
}

// Processing order of a chunk's tiles: position i -> index of the tile within the chunk. A chunk
// that ends with the ragged last tile of the problem takes that tile first: it is read with plain
// loads (several dependent round trips to memory), and taken first that latency overlaps with
// the bulk copies of the chunk's other tiles instead of following them. The host enumerates a
// chunk's segment entries in the same order.
__host__ __device__ __forceinline__ int chunk_order(int i, int nt, bool ragged_last) {
  return ragged_last ? (i == 0 ? nt - 1 : i - 1) : i;
}

__device__ __forceinline__ float sqrt_approx(float x) { float r; asm("sqrt.approx.f32 %0, %1;" : "=f"(r) : "f"(x)); return r; }
__device__ __forceinline__ float rcp_approx(float x) { float r; asm("rcp.approx.f32 %0, %1;" : "=f"(r) : "f"(x)); return r; }

template <bool BF16> struct Elem;
template <> struct Elem<false> { static constexpr int VEC = 4; typedef float T; };
template <> struct Elem<true>  { static constexpr int VEC = 8; typedef uint16_t T; };

// 16 bytes of gradient -> VEC/2 fp32 pairs (bf16 widens exactly: its 16 bits are the top half)
template <bool BF16>
__device__ __forceinline__ void unpack2(const uint4& r, u64* x) {
  if constexpr (BF16) {
    x[0] = pk(r.x << 16, r.x & 0xffff0000u); x[1] = pk(r.y << 16, r.y & 0xffff0000u);
    x[2] = pk(r.z << 16, r.z & 0xffff0000u); x[3] = pk(r.w << 16, r.w & 0xffff0000u);
  } else {
    x[0] = pk(r.x, r.y); x[1] = pk(r.z, r.w);
  }
}
__device__ __forceinline__ void unpack4f(const uint4& r, float* x) {
  x[0] = __uint_as_float(r.x); x[1] = __uint_as_float(r.y); x[2] = __uint_as_float(r.z); x[3] = __uint_as_float(r.w);
}

__device__ __forceinline__ uint4 ld_stream(const void* p) {
  uint4 r;
  asm volatile("ld.global.cs.v4.u32 {%0,%1,%2,%3}, [%4];"
               : "=r"(r.x), "=r"(r.y), "=r"(r.z), "=r"(r.w) : "l"(p));
  return r;
}
__device__ __forceinline__ void st_stream(float* p, float a, float b, float c, float d) {
  asm volatile("st.global.cs.v4.f32 [%0], {%1,%2,%3,%4};" :: "l"(p), "f"(a), "f"(b), "f"(c), "f"(d) : "memory");
}

// Per-thread running state of one tile (VEC consecutive parameters) and of the chunk.
template <int KT, int VEC>
struct Acc {
  static constexpr int NP2 = VEC / 2;
  static constexpr bool WIDE = VEC == 4;   // fp32 gradients (4 per 16 bytes): aggregate and update in fp64
  u64 np[NP2], s1[NP2], s2[NP2];    // -pivot, sum w e, sum b e^2 (pairs)
  double S[WIDE ? VEC : 1];         // sum_k b_k x_k (exact products, fp64 sums)
  float q[KT];                      // per-worker sum of squares (chunk)
  float c, pp, vs, ns;              // <g,a>, |a|^2, current segment's V and N partials
  float su, su2;                    // Adam only: sums of g/(sqrt(vhat)+eps) and of its square (chunk)

  __device__ __forceinline__ void reset_chunk() {
#pragma unroll
    for (int k = 0; k < KT; ++k) q[k] = 0.f;
    c = pp = vs = ns = 0.f;
    su = su2 = 0.f;
  }
  // k is a compile-time constant after unrolling at every call site, so q[k] is a register.
  __device__ __forceinline__ void add(int k, const u64* x, float w, float bf, double bd) {
    u64 sq = mul2(x[0], x[0]);
#pragma unroll
    for (int i = 1; i < NP2; ++i) sq = fma2(x[i], x[i], sq);
    if constexpr (WIDE) {
#pragma unroll
      for (int i = 0; i < NP2; ++i) {
        float lo, hi;
        upk(x[i], lo, hi);
        S[2 * i] = k == 0 ? bd * (double)lo : fma(bd, (double)lo, S[2 * i]);
        S[2 * i + 1] = k == 0 ? bd * (double)hi : fma(bd, (double)hi, S[2 * i + 1]);
      }
    }
    if (k == 0) {
#pragma unroll
      for (int i = 0; i < NP2; ++i) { np[i] = x[i] ^ 0x8000000080000000ull; s1[i] = 0ull; s2[i] = 0ull; }
    } else {
      const u64 w2 = pkf(w, w), b2 = pkf(bf, bf);
#pragma unroll
      for (int i = 0; i < NP2; ++i) {
        const u64 d = add2(x[i], np[i]);
        s1[i] = fma2(w2, d, s1[i]);
        s2[i] = fma2(mul2(b2, d), d, s2[i]);
      }
    }
    float lo, hi;
    upk(sq, lo, hi);
    q[k] += lo + hi;
  }
};

template <int NW>
__device__ __forceinline__ void named_sync(int bar_id) {
  asm volatile("bar.sync %0, %1;" :: "r"(bar_id), "r"(NW * 32) : "memory");
}

// Barrier among the NW warps that take part in the reductions (hardware named barrier 1).
template <int NW>
struct BarSync {
  __device__ __forceinline__ void sync() { named_sync<NW>(1); }
};

__device__ __forceinline__ float warp_sum(float v) {
#pragma unroll
  for (int o = 16; o > 0; o >>= 1) v += __shfl_xor_sync(0xffffffffu, v, o);
  return v;
}

// Shared-memory work area of the reductions (used by the NW participating warps only). Two
// copies, used by alternate chunks: a chunk ends with ONE barrier (after the warps have written
// their partials), and the warps that leave it first may fill the other copy for the next chunk
// while the slower ones still read this one. A copy is reused two chunks later, i.e. after the
// next chunk's barrier, which every thread reaches only after it has finished reading.
template <int KT, int NW>
struct RedArea {
  float rows[2][NW][KT + 4];
  float2 seg[2][kSegBuf][NW];
};

// Segment bookkeeping; identical in every participating thread.
struct SegState {
  int cur;      // segment the running (vs, ns) belong to; -1 before the chunk's first tile
  int nent;     // entries emitted so far in this chunk
  int nbuf;     // of which still buffered in shared memory
  int par;      // which copy of the work area the current chunk uses
  __device__ __forceinline__ void begin_chunk() { cur = -1; nent = 0; nbuf = 0; }
};

// Sum the buffered segment partials over the warps (fixed order) into their slots.
template <int KT, int NW>
__device__ __forceinline__ void seg_write(RedArea<KT, NW>* R, const SegState& st, const StepArgs& A, int slot0) {
  for (int e = threadIdx.x; e < st.nbuf; e += NW * 32) {
    float v = 0.f, n = 0.f;
#pragma unroll
    for (int w = 0; w < NW; ++w) { const float2 t = R->seg[st.par][e][w]; v += t.x; n += t.y; }
    const int entry = slot0 + st.nent - st.nbuf + e;
    if (DMX_IN_RANGE(A.err, entry, A.nslots)) {
      const int dest = A.slot_dest[entry];
      if (DMX_IN_RANGE(A.err, dest, A.nslots)) A.slots[dest] = make_float2(v, n);
    }
  }
}

// The buffer is full in the middle of a chunk (more than kSegBuf segment boundaries in it):
// empty it between two barriers.
template <int KT, int NW, class SY>
__device__ __forceinline__ void seg_drain(RedArea<KT, NW>* R, SegState& st, const StepArgs& A, int slot0, SY& sy) {
  sy.sync();
  seg_write<KT, NW>(R, st, A, slot0);
  sy.sync();
  st.nbuf = 0;
}

// Close the running (vs, ns) as the next entry of the chunk: a warp reduction and one
// shared-memory store per warp; no block barrier unless the shared buffer is full.
template <int KT, int VEC, int NW, class SY>
__device__ __forceinline__ void seg_entry(Acc<KT, VEC>& a, RedArea<KT, NW>* R, SegState& st, const StepArgs& A, int slot0,
                                          SY& sy, int wid, int lane) {
  const float v = warp_sum(a.vs), n = warp_sum(a.ns);
  if (lane == 0) R->seg[st.par][st.nbuf][wid] = make_float2(v, n);
  a.vs = 0.f; a.ns = 0.f;
  ++st.nbuf; ++st.nent;
  if (st.nbuf == kSegBuf) seg_drain<KT, NW>(R, st, A, slot0, sy);
}

// Attribute the tile's per-element (d, g^2) to segments. `tseg` is the tile's table entry.
// The host enumerates the entries of a chunk with the same rules (see build_tables).
template <int KT, int VEC, int NW, class SY>
__device__ __forceinline__ void segment_accumulate(Acc<KT, VEC>& a, const StepArgs& A, const float* dv,
                                                   const float* nv, int64_t jt, int64_t tile_begin,
                                                   int64_t tile_end, int tseg, RedArea<KT, NW>* R, SegState& st,
                                                   int slot0, SY& sy, int wid, int lane) {
  const int s0 = tseg & (kTileBoundaryBit - 1);
  if (s0 != st.cur) {
    if (st.cur >= 0) seg_entry<KT, VEC, NW>(a, R, st, A, slot0, sy, wid, lane);
    st.cur = s0;
  }
  if (!(tseg & kTileBoundaryBit)) {
#pragma unroll
    for (int e = 0; e < VEC; ++e) { a.vs += dv[e]; a.ns += nv[e]; }
    return;
  }
  int64_t lo = tile_begin;                       // nothing below it is pending
  int64_t next_bound = A.seg_off[st.cur + 1];
  while (st.cur < A.S - 1 && next_bound < tile_end) {
#pragma unroll
    for (int e = 0; e < VEC; ++e) {
      const int64_t j = jt + e;
      if (j >= lo && j < next_bound) { a.vs += dv[e]; a.ns += nv[e]; }
    }
    seg_entry<KT, VEC, NW>(a, R, st, A, slot0, sy, wid, lane);
    lo = next_bound;
    ++st.cur;
    next_bound = A.seg_off[st.cur + 1];
  }
#pragma unroll
  for (int e = 0; e < VEC; ++e) {
    if (jt + e >= lo) { a.vs += dv[e]; a.ns += nv[e]; }
  }
}

// End of a chunk: last segment entry, then the segment partials -> their slots and q_k, c, pp ->
// the chunk's scratch row.
template <int KT, int VEC, int NW, bool ADAM, class SY>
__device__ __forceinline__ void flush_chunk(Acc<KT, VEC>& a, const StepArgs& A, RedArea<KT, NW>* R, SegState& st,
                                            int chunk, int slot0, SY& sy, int wid, int lane) {
  if (st.cur >= 0) seg_entry<KT, VEC, NW>(a, R, st, A, slot0, sy, wid, lane);
  constexpr int NV = KT + 2 + (ADAM ? 2 : 0);
  float v[NV];
#pragma unroll
  for (int k = 0; k < KT; ++k) v[k] = warp_sum(a.q[k]);
  v[KT] = warp_sum(a.c); v[KT + 1] = warp_sum(a.pp);
  if constexpr (ADAM) { v[KT + 2] = warp_sum(a.su); v[KT + 3] = warp_sum(a.su2); }
  if (lane == 0) {
#pragma unroll
    for (int i = 0; i < NV; ++i) R->rows[st.par][wid][i] = v[i];
  }
  sy.sync();                                       // the chunk's only barrier: every warp's partials are in place
  seg_write<KT, NW>(R, st, A, slot0);
  const int t = wid * 32 + lane;
  if (t < NV) {
    float s = 0.f;
#pragma unroll
    for (int w = 0; w < NW; ++w) s += R->rows[st.par][w][t];
    if (DMX_IN_RANGE(A.err, chunk, A.nchunks)) {
      if (t < KT) { if (t < A.K) A.rows[(int64_t)t * A.nchunks + chunk] = s; }
      else A.rows[(int64_t)(A.K + t - KT) * A.nchunks + chunk] = s;
    }
  }
  st.par ^= 1;                                     // the next chunk fills the other copy
  a.reset_chunk();
}

// Tile epilogue for one thread: aggregate, spread, update, statistics. State values
// th/m/pv are inputs and are overwritten with the outputs (theta', m', g).
// Four consecutive elements (pairs E0/2 and E0/2+1 of the thread) at a time, so that the
// state values of only four elements are live at once.
template <int KT, int VEC, bool ADAM, int E0>
__device__ __forceinline__ void finish4(Acc<KT, VEC>& a, const StepArgs& A, float* th, float* m, float* pv,
                                        float* dv, float* nv, float* vv) {
  float p[4], s1[4], s2[4];
#pragma unroll
  for (int i = 0; i < 2; ++i) {
    upk(a.np[E0 / 2 + i], p[2 * i], p[2 * i + 1]);
    upk(a.s1[E0 / 2 + i], s1[2 * i], s1[2 * i + 1]);
    upk(a.s2[E0 / 2 + i], s2[2 * i], s2[2 * i + 1]);
  }
#pragma unroll
  for (int e = 0; e < 4; ++e) {
    double g64 = 0.0;
    float g;
    if constexpr (Acc<KT, VEC>::WIDE) {
      g64 = a.S[E0 + e] * A.rB;
      g = (float)g64;
    } else {
      g = s1[e] - p[e];                          // p holds the negated pivot
    }
    dv[E0 + e] = fmaf(-A.Bf * s1[e], s1[e], s2[e]);
    nv[E0 + e] = g * g;
    a.c = fmaf(g, pv[e], a.c);
    a.pp = fmaf(pv[e], pv[e], a.pp);
    if constexpr (ADAM) {
      const float mn = fmaf(A.beta, m[e], A.omb1 * g);
      const float vn = fmaf(A.beta2, vv[e], A.omb2 * (g * g));
      // one approximate square root and one approximate reciprocal per element (each within
      // 2^-22 relative, subnormals kept): IEEE sqrt and two divisions made the bf16 consumer
      // compute-bound
      const float rden = rcp_approx(sqrt_approx(vn * A.c2) + A.eps);
      th[e] = fmaf(-A.lr, (mn * A.c1) * rden, th[e]);
      const float gh = g * rden;                   // the gradient in units of Adam's running scale
      a.su += gh;
      a.su2 = fmaf(gh, gh, a.su2);
      m[e] = mn;
      vv[e] = vn;
    } else if constexpr (Acc<KT, VEC>::WIDE) {
      const double mn = fma(A.beta64, (double)m[e], g64);
      th[e] = (float)fma(-A.lr64, mn, (double)th[e]);
      m[e] = (float)mn;
    } else {
      const float mn = fmaf(A.beta, m[e], g);
      th[e] = fmaf(-A.lr, mn, th[e]);
      m[e] = mn;
    }
    pv[e] = g;
  }
}

template <int KT, int VEC, bool ADAM = false>
__device__ __forceinline__ void finish_elements(Acc<KT, VEC>& a, const StepArgs& A, float* th, float* m,
                                                float* pv, float* dv, float* nv, float* vv = nullptr) {
  finish4<KT, VEC, ADAM, 0>(a, A, th, m, pv, dv, nv, vv);
  if constexpr (VEC == 8) finish4<KT, VEC, ADAM, 4>(a, A, th + 4, m + 4, pv + 4, dv, nv, ADAM ? vv + 4 : vv);
}

// ------------------------------------------------------------------------------------------
// Direct tile: every thread streams its own 16-byte pieces with plain vector loads, U worker
// loads in flight at a time. With GUARD it is the code path of the ragged last tile.

template <int KT, bool BF16, bool GUARD, int U, bool ADAM = false>
__device__ __forceinline__ void direct_tile(Acc<KT, Elem<BF16>::VEC>& a, const StepArgs& A, int64_t jt,
                                            float* dv, float* nv) {
  constexpr int VEC = Elem<BF16>::VEC;
  typedef typename Elem<BF16>::T GT;
#pragma unroll
  for (int k0 = 0; k0 < KT; k0 += U) {
    if (k0 < A.K) {
      u64 x[U][VEC / 2];
#pragma unroll
      for (int u = 0; u < U; ++u) {
        if (k0 + u < KT && k0 + u < A.K) {
          const GT* src = static_cast<const GT*>(A.grad[k0 + u]) + jt;
          if constexpr (GUARD) {
            if (jt + VEC <= A.P) {              // the whole 16-byte piece is inside: one vector load
              const uint4 r = ld_stream(src);
              unpack2<BF16>(r, x[u]);
            } else {                            // the piece that straddles P (and those beyond it): element by element
              uint32_t bits[VEC];
#pragma unroll
              for (int e = 0; e < VEC; ++e) {
                bits[e] = 0u;
                if (jt + e < A.P) {
                  if constexpr (BF16) bits[e] = (uint32_t)src[e] << 16; else bits[e] = __float_as_uint(src[e]);
                }
              }
#pragma unroll
              for (int i = 0; i < VEC / 2; ++i) x[u][i] = pk(bits[2 * i], bits[2 * i + 1]);
            }
          } else {
            const uint4 r = ld_stream(src);
            unpack2<BF16>(r, x[u]);
          }
        }
      }
#pragma unroll
      for (int u = 0; u < U; ++u) {
        if (k0 + u < KT && k0 + u < A.K) a.add(k0 + u, x[u], A.w[k0 + u], A.bf[k0 + u], A.bd[k0 + u]);
      }
    }
  }
  // state streams
  float th[VEC], m[VEC], pv[VEC], vv[ADAM ? VEC : 1];
  if constexpr (GUARD) {
#pragma unroll
    for (int e = 0; e < VEC; ++e) {
      const bool ok = jt + e < A.P;
      th[e] = ok ? A.params[jt + e] : 0.f; m[e] = ok ? A.momentum[jt + e] : 0.f; pv[e] = ok ? A.prev[jt + e] : 0.f;
      if constexpr (ADAM) vv[e] = ok ? A.second[jt + e] : 1.f;   // 1: keeps the unused lanes' divisions finite
    }
  } else {
#pragma unroll
    for (int h = 0; h < VEC / 4; ++h) {
      uint4 r = ld_stream(A.params + jt + 4 * h);   unpack4f(r, th + 4 * h);
      r = ld_stream(A.momentum + jt + 4 * h);       unpack4f(r, m + 4 * h);
      r = ld_stream(A.prev + jt + 4 * h);           unpack4f(r, pv + 4 * h);
      if constexpr (ADAM) { r = ld_stream(A.second + jt + 4 * h); unpack4f(r, vv + 4 * h); }
    }
  }
  // (lanes beyond P carry g = 0 and v = 1: they add exact zeros to every sum)
  finish_elements<KT, VEC, ADAM>(a, A, th, m, pv, dv, nv, vv);
  if constexpr (GUARD) {
#pragma unroll
    for (int e = 0; e < VEC; ++e) {
      if (jt + e < A.P) {
        A.params[jt + e] = th[e]; A.momentum[jt + e] = m[e]; A.prev[jt + e] = pv[e];
        if constexpr (ADAM) A.second[jt + e] = vv[e];
      } else { dv[e] = 0.f; nv[e] = 0.f; }
    }
  } else {
#pragma unroll
    for (int h = 0; h < VEC / 4; ++h) {
      st_stream(A.params + jt + 4 * h, th[4 * h], th[4 * h + 1], th[4 * h + 2], th[4 * h + 3]);
      st_stream(A.momentum + jt + 4 * h, m[4 * h], m[4 * h + 1], m[4 * h + 2], m[4 * h + 3]);
      st_stream(A.prev + jt + 4 * h, pv[4 * h], pv[4 * h + 1], pv[4 * h + 2], pv[4 * h + 3]);
      if constexpr (ADAM) st_stream(A.second + jt + 4 * h, vv[4 * h], vv[4 * h + 1], vv[4 * h + 2], vv[4 * h + 3]);
    }
  }
}

// The ragged last tile of the pipelined kernel: plain loads, every element tested against P.
// All of the tile's lines are requested from memory at once (prefetch to L2) before the loads,
// which are issued four workers at a time. Two forms, chosen by the kernel's worker capacity:
//  - in the loop's own registers (few workers). Out of line, the running sums live in local
//    memory, which the large shared-memory carve-out leaves almost no L1 for: the one tile then
//    took 10-80 us, a large part of a step of a few million parameters.
//  - out of line, on copies (many workers). Inlined, this second unrolled body changed the code
//    the compiler produced for the full tiles: with 32 workers the fused pass lost 1 % at full
//    clock and 3-10 % when the power limit lowers the SM clock and the consumers' instruction
//    stream starts to matter. The copies (not the loop's registers) have their address taken.
template <int KT, bool BF16, bool ADAM>
__device__ __forceinline__ void ragged_tile_body(Acc<KT, Elem<BF16>::VEC>& a, const StepArgs& A, int64_t jt, float* dv, float* nv) {
  typedef typename Elem<BF16>::T GT;
  if (jt < A.P) {
#pragma unroll 4
    for (int k = 0; k < A.K; ++k)
      asm volatile("prefetch.global.L2 [%0];" :: "l"(static_cast<const GT*>(A.grad[k]) + jt));
    asm volatile("prefetch.global.L2 [%0];" :: "l"(A.params + jt));
    asm volatile("prefetch.global.L2 [%0];" :: "l"(A.momentum + jt));
    asm volatile("prefetch.global.L2 [%0];" :: "l"(A.prev + jt));
    if constexpr (ADAM) asm volatile("prefetch.global.L2 [%0];" :: "l"(A.second + jt));
  }
  direct_tile<KT, BF16, true, 4, ADAM>(a, A, jt, dv, nv);
}

template <int KT, bool BF16, bool ADAM>
__device__ __noinline__ void ragged_tile_call(Acc<KT, Elem<BF16>::VEC>& a, const StepArgs& A, int64_t jt, float* dv, float* nv) {
  ragged_tile_body<KT, BF16, ADAM>(a, A, jt, dv, nv);
}

constexpr int kRaggedInlineMaxK = 8;   // kernels for up to this many workers take the ragged tile inline

template <int KT, bool BF16, bool ADAM>
__device__ __forceinline__ void ragged_tile(Acc<KT, Elem<BF16>::VEC>& a, const StepArgs& A, int64_t jt, float* dv, float* nv) {
  if constexpr (KT <= kRaggedInlineMaxK) {
    ragged_tile_body<KT, BF16, ADAM>(a, A, jt, dv, nv);
  } else {
    constexpr int VEC = Elem<BF16>::VEC;
    Acc<KT, VEC> a2 = a;
    float dv2[VEC], nv2[VEC];
    ragged_tile_call<KT, BF16, ADAM>(a2, A, jt, dv2, nv2);
    a = a2;
#pragma unroll
    for (int e = 0; e < VEC; ++e) { dv[e] = dv2[e]; nv[e] = nv2[e]; }
  }
}

template <int KT, bool BF16, int NW, int U, bool ADAM>
__global__ void __launch_bounds__(NW * 32)
direct_kernel(const __grid_constant__ StepArgs A) {
  constexpr int VEC = Elem<BF16>::VEC;
  constexpr int T = NW * 32 * VEC;
  __shared__ RedArea<KT, NW> R;
  const int wid = threadIdx.x >> 5, lane = threadIdx.x & 31;
  Acc<KT, VEC> a;
  a.reset_chunk();
  BarSync<NW> sy;
  SegState st; st.par = 0;
  // chunks are dealt statically here: chunk c belongs to CTA c mod grid
  for (int c = blockIdx.x; c < A.nchunks; c += gridDim.x) {
    const int t0 = A.chunk_tile0[c], nt = A.chunk_ntiles[c], cstride = A.chunk_stride[c];
    const int slot0 = A.chunk_slot0[c];
    const bool rl = A.P % T != 0 && tile_of(A, t0, cstride, nt - 1) == A.ntiles - 1;
    st.begin_chunk();
    for (int i = 0; i < nt; ++i) {
      const int t = tile_of(A, t0, cstride, chunk_order(i, nt, rl));
      if (!DMX_IN_RANGE(A.err, t, A.ntiles)) continue;
      const int tseg = A.tile_seg[t];
      const int64_t tile_begin = (int64_t)t * T;
      const int64_t jt = tile_begin + (int64_t)threadIdx.x * VEC;
      int64_t tile_end = tile_begin + T;
      float dv[VEC], nv[VEC];
      if (tile_end <= A.P) {
        direct_tile<KT, BF16, false, U, ADAM>(a, A, jt, dv, nv);
      } else {
        tile_end = A.P;
        direct_tile<KT, BF16, true, U, ADAM>(a, A, jt, dv, nv);
      }
      segment_accumulate<KT, VEC, NW>(a, A, dv, nv, jt, tile_begin, tile_end, tseg, &R, st, slot0, sy, wid, lane);
    }
    flush_chunk<KT, VEC, NW, ADAM>(a, A, &R, st, c, slot0, sy, wid, lane);
  }
}

// ------------------------------------------------------------------------------------------
// Finalize: fp64 second level in a fixed order, then the derived scalars.

__device__ __forceinline__ double warp_sum_d(double v) {
#pragma unroll
  for (int o = 16; o > 0; o >>= 1) v += __shfl_xor_sync(0xffffffffu, v, o);
  return v;
}

constexpr int kFinalWarps = 8;

// The scalar part of the state vector from the step's reduced sums (the definitions of the state
// layout): D = sum_s Vraw_s, A = sum_s N_s, Qw = sum_k b_k q_k, c = <g,a>, pp = |a|^2.
// (Out of line on purpose: the finalize kernel runs it once on zeros while it waits for the fused
// pass, so that the one real call finds this code in the instruction caches.)
static __device__ __noinline__ void emit_header(float* out, int K, double B, double D, double A, double Qw, double c, double pp,
                                            bool nonfinite_q, unsigned errbits, int adam, double su, double su2, double P) {
  int flags = 0;
  double trS = 0.0;
  if (K >= 2) trS = D / (double)(K - 1); else flags |= 8;
  const double G2 = A - trS / B;
  double gns = 0.0;
  if (G2 > 0.0) gns = trS / G2; else flags |= 2;
  double cosv = 0.0;
  if (A > 0.0 && pp > 0.0) cosv = c / sqrt(A * pp); else flags |= 4;
  const double sig2 = A > 0.0 ? trS / (B * A) : 0.0;
  const double sig = sqrt(sig2 > 0.0 ? sig2 : 0.0);
  if (nonfinite_q || !isfinite((float)A) || !isfinite((float)pp)) flags |= 1;
  if (errbits & kErrWait) flags |= 16;
  if (errbits & kErrBounds) flags |= 32;
  out[0] = (float)B; out[1] = (float)A; out[2] = (float)trS; out[3] = (float)G2; out[4] = (float)gns;
  out[5] = (float)cosv; out[6] = (float)c; out[7] = (float)pp; out[8] = (float)sig2; out[9] = (float)sig;
  out[10] = (float)(Qw / B); out[11] = (float)flags;
  out[12] = out[13] = out[14] = out[15] = 0.f;
  if (adam) {
    // the gradient in units of Adam's running scale, ghat_j = g_j / (sqrt(vhat_j) + eps):
    // its mean, variance and standard deviation across the parameters
    const double mean = su / P;
    const double var = su2 / P - mean * mean;
    out[12] = (float)mean; out[13] = (float)var; out[14] = (float)sqrt(var > 0.0 ? var : 0.0);
  }
}

constexpr int kFinalPart = 256;  // slots per segment unit

// First level. Blocks 0..ncol-1 each sum one column (q_k, c, pp, and Adam's two) of the chunk
// rows: warp w takes the w-th eighth of the column, lanes stride through it with eight loads in
// flight, and the eight warp sums are added in warp order. The other blocks take segment units
// (runs of at most kFinalPart slots of one segment), one warp each. Second level, in the last
// block to finish: the units of each segment in order, then the derived scalars.
static __global__ void __launch_bounds__(kFinalWarps * 32) finalize_kernel(const __grid_constant__ FinalArgs F) {
  const int wid = threadIdx.x >> 5, lane = threadIdx.x & 31;
  const int K = F.K, S = F.S;
  const int ncol = K + 2 + 2 * F.adam;
  __shared__ double s_col[kFinalWarps];
  __shared__ float s_warm[16];
  // Launched as a programmatic dependent, this kernel's blocks are usually resident long before
  // the fused pass ends. What does not depend on that pass is done while they wait: the table
  // entries each thread will need are fetched (after a step's worth of streaming they come from
  // DRAM, a microsecond per dependent load), and thread 0 runs the header arithmetic once on
  // zeros into shared memory, which brings its code (a few KB, cold as well) into the
  // instruction caches. After the wait only loads of the fused pass's own output remain.
  const int u_mine = ((int)blockIdx.x - ncol) * kFinalWarps + wid;
  int pre_lo = 0, pre_hi = 0, pre_u0 = 0, pre_u1 = 0;
  if ((int)blockIdx.x >= ncol && u_mine < F.nunits) { pre_lo = F.unit_lo[u_mine]; pre_hi = F.unit_hi[u_mine]; }
  if ((int)threadIdx.x < S) { pre_u0 = F.seg_unit_ptr[threadIdx.x]; pre_u1 = F.seg_unit_ptr[threadIdx.x + 1]; }
  if (threadIdx.x == 0) emit_header(s_warm, K, F.B, 0.0, 0.0, 0.0, 0.0, 0.0, false, 0u, F.adam, 0.0, 0.0, F.P);
  // everything read from here on was written by the step's fused pass: with a programmatic
  // dependent launch this is where its completion (and the visibility of its writes) is awaited
  asm volatile("griddepcontrol.wait;" ::: "memory");
  if ((int)blockIdx.x < ncol) {
    const float* col = F.rows + (int64_t)blockIdx.x * F.nchunks;
    const int per = (F.nchunks + kFinalWarps - 1) / kFinalWarps;
    const int lo = wid * per, hi = lo + per < F.nchunks ? lo + per : F.nchunks;
    double a[8];
#pragma unroll
    for (int i = 0; i < 8; ++i) a[i] = 0.0;
    int c = lo + lane;
    for (; c + 224 < hi; c += 256) {
#pragma unroll
      for (int i = 0; i < 8; ++i) a[i] += (double)col[c + 32 * i];
    }
    for (; c < hi; c += 32) a[0] += (double)col[c];
    const double acc = warp_sum_d(((a[0] + a[1]) + (a[2] + a[3])) + ((a[4] + a[5]) + (a[6] + a[7])));
    if (lane == 0) s_col[wid] = acc;
    __syncthreads();
    if (threadIdx.x == 0) {
      double t = 0.0;
      for (int w = 0; w < kFinalWarps; ++w) t += s_col[w];
      F.colsum[blockIdx.x] = t;
    }
  } else {
    const int u = u_mine;
    if (u < F.nunits) {
      int lo = pre_lo, hi = pre_hi;
      if (!DMX_IN_RANGE(F.err, lo, F.nslots + 1) || !DMX_IN_RANGE(F.err, hi, F.nslots + 1)) hi = lo = 0;
      double v = 0.0, n = 0.0, v1 = 0.0, n1 = 0.0, v2 = 0.0, n2 = 0.0, v3 = 0.0, n3 = 0.0;
      int i = lo + lane;
      for (; i + 96 < hi; i += 128) {          // four loads in flight per lane; fixed summation order
        const float2 t0 = F.slots[i], t1 = F.slots[i + 32], t2 = F.slots[i + 64], t3 = F.slots[i + 96];
        v += (double)t0.x; n += (double)t0.y; v1 += (double)t1.x; n1 += (double)t1.y;
        v2 += (double)t2.x; n2 += (double)t2.y; v3 += (double)t3.x; n3 += (double)t3.y;
      }
      for (; i < hi; i += 32) {
        const float2 t = F.slots[i];
        v += (double)t.x; n += (double)t.y;
      }
      v = warp_sum_d((v + v1) + (v2 + v3)); n = warp_sum_d((n + n1) + (n2 + n3));
      if (lane == 0) F.segpart[u] = make_double2(v, n);
    }
  }
  __shared__ unsigned s_last;
  __shared__ double s_red[2][kFinalWarps];
  __threadfence();
  __syncthreads();
  if (threadIdx.x == 0) s_last = (atomicAdd(F.ticket, 1u) == gridDim.x - 1) ? 1u : 0u;
  __syncthreads();
  if (!s_last) return;
  __threadfence();
  // last block: everything below reads what all blocks wrote. The K+2 column sums go through
  // shared memory so that the serial part at the end does not pay a global load per term.
  __shared__ double cs[kMaxK + 4];
  {
    const volatile double* gcs = F.colsum;
    if (threadIdx.x < ncol) cs[threadIdx.x] = gcs[threadIdx.x];
  }
  const volatile double2* sp = F.segpart;
  if (F.partials) {
    // a parameter shard of a larger problem: hand out the raw sums, to be added over the shards
    double* pt = F.partials;
    for (int s = threadIdx.x; s < S; s += blockDim.x) {
      double v = 0.0, n = 0.0;
      const int u0 = s == (int)threadIdx.x ? pre_u0 : F.seg_unit_ptr[s], u1 = s == (int)threadIdx.x ? pre_u1 : F.seg_unit_ptr[s + 1];
      for (int u = u0; u < u1; ++u) { v += sp[u].x; n += sp[u].y; }
      pt[K + 4 + s] = v;
      pt[K + 4 + S + s] = n;
    }
    __syncthreads();                                   // cs[] is in place
    for (int k = threadIdx.x; k < K; k += blockDim.x) pt[F.orig[k]] = cs[k];
    if (threadIdx.x == 0) {
      pt[K] = cs[K]; pt[K + 1] = cs[K + 1];
      pt[K + 2] = F.adam ? cs[K + 2] : 0.0; pt[K + 3] = F.adam ? cs[K + 3] : 0.0;
      const unsigned errbits = *reinterpret_cast<volatile unsigned*>(F.err);
      // summed over the shards: waits that ran out count 1 each, range violations 65536 each
      pt[K + 4 + 2 * S] = (double)(errbits & kErrWait) + 65536.0 * (double)((errbits & kErrBounds) != 0u);
      if (errbits) *F.err = 0u;
      *F.next_chunk = 0u;
      *F.ticket = 0u;
    }
    return;
  }
  float* out = F.out_state;
  double aV = 0.0, aN = 0.0;
  // (thread 0 asks for the error word now; it is used at the very end)
  unsigned errbits = 0u;
  if (threadIdx.x == 0) errbits = *reinterpret_cast<volatile unsigned*>(F.err);
  for (int s = threadIdx.x; s < S; s += blockDim.x) {
    double v = 0.0, n = 0.0;
    const int u0 = s == (int)threadIdx.x ? pre_u0 : F.seg_unit_ptr[s], u1 = s == (int)threadIdx.x ? pre_u1 : F.seg_unit_ptr[s + 1];
    for (int u = u0; u < u1; ++u) { v += sp[u].x; n += sp[u].y; }
    out[16 + K + s] = K >= 2 ? (float)(v / (double)(K - 1)) : 0.f;
    out[16 + K + S + s] = (float)n;
    aV += v; aN += n;
  }
  aV = warp_sum_d(aV); aN = warp_sum_d(aN);
  if (lane == 0) { s_red[0][wid] = aV; s_red[1][wid] = aN; }
  __syncthreads();
  for (int k = threadIdx.x; k < K; k += blockDim.x) out[16 + F.orig[k]] = (float)cs[k];
  if (wid == 0) {
    // sum_k b_k q_k: lane l takes workers l and l + 32, then the shuffle tree (a fixed order)
    double Qw = 0.0;
    bool bad = false;
    for (int k = lane; k < K; k += 32) { const double qk = cs[k]; Qw += F.b[k] * qk; bad = bad | !isfinite((float)qk); }
    Qw = warp_sum_d(Qw);
    bad = __any_sync(0xffffffffu, bad);
    if (lane != 0) return;
    double D = 0.0, A = 0.0;
    for (int w = 0; w < kFinalWarps; ++w) { D += s_red[0][w]; A += s_red[1][w]; }
    if (errbits) *F.err = 0u;
    emit_header(out, K, F.B, D, A, Qw, cs[K], cs[K + 1], bad, errbits, F.adam, F.adam ? cs[K + 2] : 0.0,
                F.adam ? cs[K + 3] : 0.0, F.P);
    *F.next_chunk = 0u;                      // the fused pass has completed: ready for the next step (or a graph replay)
    *F.ticket = 0u;
  }
}

// The state vector from raw sums added over the parameter shards of one problem (one block).
static __global__ void __launch_bounds__(kFinalWarps * 32) derive_kernel(const __grid_constant__ DeriveArgs G) {
  const int wid = threadIdx.x >> 5, lane = threadIdx.x & 31;
  const int K = G.K, S = G.S;
  const double* pt = G.partials;
  float* out = G.out_state;
  __shared__ double s_red[2][kFinalWarps];
  double aV = 0.0, aN = 0.0;
  for (int s = threadIdx.x; s < S; s += blockDim.x) {
    const double v = pt[K + 4 + s], n = pt[K + 4 + S + s];
    out[16 + K + s] = K >= 2 ? (float)(v / (double)(K - 1)) : 0.f;
    out[16 + K + S + s] = (float)n;
    aV += v; aN += n;
  }
  aV = warp_sum_d(aV); aN = warp_sum_d(aN);
  if (lane == 0) { s_red[0][wid] = aV; s_red[1][wid] = aN; }
  __syncthreads();
  for (int k = threadIdx.x; k < K; k += blockDim.x) out[16 + k] = (float)pt[k];
  if (wid == 0) {
    // sum_k b_k q_k in the order the single-GPU finalize takes it. There the workers are in
    // processing order (largest batch first); a sum over lanes and a shuffle tree of a permuted
    // list differs in the last bits of the fp64 value only, below what the fp32 output keeps.
    double Qw = 0.0;
    bool bad = false;
    for (int k = lane; k < K; k += 32) { const double qk = pt[k]; Qw += G.b[k] * qk; bad = bad | !isfinite((float)qk); }
    Qw = warp_sum_d(Qw);
    bad = __any_sync(0xffffffffu, bad);
    if (lane != 0) return;
    double D = 0.0, A = 0.0;
    for (int w = 0; w < kFinalWarps; ++w) { D += s_red[0][w]; A += s_red[1][w]; }
    // the error words of the shards were added up: any wait that ran out, any index out of range
    const double ew = pt[K + 4 + 2 * S];
    const unsigned errbits = (fmod(ew, 65536.0) != 0.0 ? kErrWait : 0u) | (ew >= 65536.0 ? kErrBounds : 0u);
    emit_header(out, K, G.B, D, A, Qw, pt[K], pt[K + 1], bad, errbits, G.adam, pt[K + 2], pt[K + 3], G.P);
  }
}

// ------------------------------------------------------------------------------------------
// Pipelined kernel: a producer warp streams whole tiles into a shared-memory ring with bulk
// asynchronous copies (the TMA engine; non-tensor 1-D form, no multicast) completing on
// mbarriers; CW consumer warps read 16 bytes per thread per stream from the ring and do the
// arithmetic. Every wait is bounded; a wait that runs out raises the handle's error word and
// the CTA drains without waiting any more.

__device__ __forceinline__ uint32_t smem_u32(const void* p) { return (uint32_t)__cvta_generic_to_shared(p); }

__device__ __forceinline__ void mbar_init(uint32_t bar, uint32_t count) {
  asm volatile("mbarrier.init.shared::cta.b64 [%0], %1;" :: "r"(bar), "r"(count) : "memory");
}
__device__ __forceinline__ void mbar_expect_tx(uint32_t bar, uint32_t bytes) {
  asm volatile("mbarrier.arrive.expect_tx.shared::cta.b64 _, [%0], %1;" :: "r"(bar), "r"(bytes) : "memory");
}
__device__ __forceinline__ void mbar_arrive(uint32_t bar) {
  asm volatile("mbarrier.arrive.shared::cta.b64 _, [%0];" :: "r"(bar) : "memory");
}
__device__ __forceinline__ bool mbar_try_wait(uint32_t bar, uint32_t parity) {
  uint32_t ok;
  asm volatile(
      "{\n\t.reg .pred p;\n\t"
      "mbarrier.try_wait.parity.shared::cta.b64 p, [%1], %2;\n\t"
      "selp.u32 %0, 1, 0, p;\n\t}"
      : "=r"(ok) : "r"(bar), "r"(parity) : "memory");
  return ok != 0;
}

// Polling budget of a wait. A poll (mbarrier.try_wait) that finds the barrier incomplete suspends the thread for
// about 4 us on B200 (measured with dmx_selftest_wait: 1043 ms for 2^18 polls), so this is about one second:
// a thousand times the longest wait of a healthy step, and short enough for a caller to notice a failure at once.
constexpr uint32_t kWaitLimit = 1u << 18;

// Bounded wait. Returns false (at once) when the CTA has given up, and raises the give-up
// flag itself when its own polling budget runs out.
__device__ __forceinline__ bool mbar_wait(uint32_t bar, uint32_t parity, volatile uint32_t* give_up, unsigned* err,
                                          uint32_t limit = kWaitLimit) {
  if (mbar_try_wait(bar, parity)) return true;
  if (*give_up) return false;
  for (uint32_t i = 0; i < limit; ++i) {
    if (mbar_try_wait(bar, parity)) return true;
    if ((i & 1023u) == 1023u && *give_up) return false;
  }
  *give_up = 1u;
  atomicOr(err, 1u);
  return false;
}

__device__ __forceinline__ uint64_t policy_evict_first() {
  uint64_t p;
  asm volatile("createpolicy.fractional.L2::evict_first.b64 %0, 1.0;" : "=l"(p));
  return p;
}

// global -> shared bulk copy; src and dst 16-byte aligned, bytes a multiple of 16
__device__ __forceinline__ void bulk_load(uint32_t dst, const void* src, uint32_t bytes, uint32_t bar, uint64_t pol) {
  asm volatile(
      "cp.async.bulk.shared::cluster.global.mbarrier::complete_tx::bytes.L2::cache_hint [%0], [%1], %2, [%3], %4;"
      :: "r"(dst), "l"(src), "r"(bytes), "r"(bar), "l"(pol) : "memory");
}

__device__ __forceinline__ uint4 lds128(uint32_t addr) {
  uint4 r;
  asm volatile("ld.shared.v4.u32 {%0,%1,%2,%3}, [%4];" : "=r"(r.x), "=r"(r.y), "=r"(r.z), "=r"(r.w) : "r"(addr));
  return r;
}

// Barrier among the consumer warps built on an mbarrier (one arrival per warp), so that its
// wait is bounded like every other wait of this kernel: if a warp has left after a failed wait,
// the others time out, raise the error word and go on instead of hanging in a hardware barrier.
struct MbarSync {
  uint32_t bar, phase;
  volatile uint32_t* give_up;
  unsigned* err;
  int lane;
  __device__ __forceinline__ void sync() {
    __syncwarp();
    if (lane == 0) mbar_arrive(bar);
    (void)mbar_wait(bar, phase, give_up, err);
    phase ^= 1u;
  }
};

template <int KT_, bool BF16_, int CW_, int G_, int NSTAGE_, int NSS_, bool ADAM_ = false, int LB_ = G_>
struct PipeCfg {
  static constexpr int KT = KT_, CW = CW_, G = G_, NSTAGE = NSTAGE_, NSS = NSS_;
  static constexpr int LB = LB_;                     // streams of a stage a consumer thread loads before it accumulates them
  static constexpr bool BF16 = BF16_, ADAM = ADAM_;
  static constexpr int NST = ADAM ? 4 : 3;           // state streams: prev_agg, momentum, params (, second moment)
  static constexpr int VEC = Elem<BF16>::VEC;
  static constexpr int CT = CW * 32;                 // consumer threads
  static constexpr int THREADS = CT + 32;            // + the producer warp
  static constexpr int T = CT * VEC;                 // elements per tile
  static constexpr int SLOT = CT * 16;               // one gradient stream's tile, bytes
  static constexpr int STAGE = G * SLOT;
  static constexpr int SSLOT = T * 4;                // one state stream's tile, bytes
  static constexpr int SSTAGE = NST * SSLOT;
  static constexpr int RING = NSTAGE * STAGE;
  static constexpr int SRING = NSS * SSTAGE;
  static constexpr int RED = (int)((sizeof(RedArea<KT, CW>) + 15) / 16 * 16);
  static constexpr int QN = 4;                       // chunk descriptors in flight from the producer to the consumers
  static constexpr int NBAR = 2 * NSTAGE + 2 * NSS + 2 * QN + 1;
  static constexpr int TAIL = 16 + QN * 32;          // give-up word, chunk queue (8 ints per entry)
  static constexpr size_t SMEM = (size_t)RING + SRING + RED + NBAR * 8 + TAIL;
  static_assert(G >= 1 && G <= 32, "one producer lane per stream of a stage");
  static_assert(LB >= 1 && LB <= G, "load batch");
  static_assert(NSTAGE <= 32 && NSS <= 32, "stage masks are 32 bits wide");
  static_assert(SMEM <= 227 * 1024, "ring does not fit in shared memory");
};

template <class C>
__global__ void __launch_bounds__(C::THREADS, 1) pipe_kernel(const __grid_constant__ StepArgs A) {
  constexpr int KT = C::KT, VEC = C::VEC, CW = C::CW, G = C::G, NSTAGE = C::NSTAGE, NSS = C::NSS, T = C::T, QN = C::QN;
  constexpr int LB = C::LB;
  constexpr bool BF16 = C::BF16, ADAM = C::ADAM;
  extern __shared__ __align__(128) unsigned char smem[];
  const uint32_t ring = smem_u32(smem);
  const uint32_t sring = ring + C::RING;
  RedArea<KT, CW>* R = reinterpret_cast<RedArea<KT, CW>*>(smem + C::RING + C::SRING);
  const uint32_t bars = sring + C::SRING + C::RED;
  unsigned char* tail = smem + C::RING + C::SRING + C::RED + C::NBAR * 8;
  volatile uint32_t* give_up = reinterpret_cast<volatile uint32_t*>(tail);
  volatile int* queue = reinterpret_cast<volatile int*>(tail + 16);   // entry: chunk (-1: none left), first tile,
                                                                       // tiles, group stride, first slot
  // barriers, 8 bytes each: full_g[NSTAGE], empty_g[NSTAGE], full_s[NSS], empty_s[NSS],
  // full_q[QN], empty_q[QN], and the consumers' own barrier
  const uint32_t full_g = bars, empty_g = bars + 8 * NSTAGE, full_s = bars + 16 * NSTAGE, empty_s = full_s + 8 * NSS;
  const uint32_t full_q = empty_s + 8 * NSS, empty_q = full_q + 8 * QN, csync = empty_q + 8 * QN;
  const int wid = threadIdx.x >> 5, lane = threadIdx.x & 31;
  // one thread per barrier (a single thread initialising all of them in turn costs the CTA half a
  // microsecond before its first copy): "full" barriers take one arrival, the others one per consumer warp
  static_assert(C::NBAR <= C::THREADS, "one thread per barrier");
  if ((int)threadIdx.x < C::NBAR) {
    const int i = threadIdx.x;
    const bool full = i < NSTAGE || (i >= 2 * NSTAGE && i < 2 * NSTAGE + NSS) ||
                      (i >= 2 * NSTAGE + 2 * NSS && i < 2 * NSTAGE + 2 * NSS + QN);
    mbar_init(bars + 8 * i, full ? 1 : CW);
    if (i == 0) *give_up = 0u;
    asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory");
    asm volatile("fence.proxy.async.shared::cta;" ::: "memory");
  }
  __syncthreads();
  // the step's second kernel may be made resident from now on; it waits for this grid to complete
  asm volatile("griddepcontrol.launch_dependents;" ::: "memory");
  constexpr int ESZ = BF16 ? 2 : 4;

  if (wid == CW) {
    // ---------------- producer ----------------
    // The whole warp takes part: every lane waits for the stage to be free, lane 0 arms the
    // barrier with the byte count, then lane u issues the copy of stream u of the stage (one
    // thread issuing every copy in turn is itself the bottleneck: each issue is a dependent
    // chain of about a hundred cycles). Lane 0 also draws the CTA's next chunk from the step's
    // counter and passes it to the consumers through a small queue in shared memory.
    const uint64_t pol = policy_evict_first();
    uint32_t stage = 0, phase = 0, ss = 0, sphase = 0, qi = 0, qphase = 0;
    uint32_t armed_g = 0, par_g = 0, armed_s = 0, par_s = 0;   // stages armed, and the parity of the last arming
    bool ok = true;
    // Lane 0 draws the next chunk a few tiles before the current chunk's copies have all been
    // issued, and fetches its descriptor when they have (the ring then holds several
    // microseconds of work, which covers that load). Drawing earlier would reserve chunks that a
    // slow SM cannot start for a long time, which is what the dynamic schedule is there to avoid. The first chunk of CTA b is chunk b; draws
    // hand out the chunks from `gridDim.x` on.
    int cur = -1, c_t0 = 0, c_nt = 0, c_stride = 0, c_slot0 = 0;
    if (lane == 0 && (int)blockIdx.x < A.nchunks) {
      cur = (int)blockIdx.x;
      c_t0 = A.chunk_tile0[cur]; c_nt = A.chunk_ntiles[cur]; c_stride = A.chunk_stride[cur]; c_slot0 = A.chunk_slot0[cur];
    }
    while (ok) {
      ok = __all_sync(0xffffffffu, mbar_wait(empty_q + 8 * qi, qphase ^ 1u, give_up, A.err));
      if (!ok) break;
      unsigned drawn = 0xffffffffu;                              // no draw made: nothing more for this CTA
      if (lane == 0) {
        volatile int* e = queue + 8 * qi;
        e[0] = cur; e[1] = c_t0; e[2] = c_nt; e[3] = c_stride; e[4] = c_slot0;
        mbar_arrive(full_q + 8 * qi);                            // (release: the consumers' wait sees the entry)
      }
      const int c = __shfl_sync(0xffffffffu, cur, 0);
      if (++qi == QN) { qi = 0; qphase ^= 1u; }
      if (c < 0) break;                                          // the list is exhausted: the consumers leave too
      const int t0 = __shfl_sync(0xffffffffu, c_t0, 0), nt = __shfl_sync(0xffffffffu, c_nt, 0);
      const int cstride = __shfl_sync(0xffffffffu, c_stride, 0);
      const int draw_at = nt > 3 ? nt - 3 : 0;
      const bool rl = A.P % T != 0 && tile_of(A, t0, cstride, nt - 1) == A.ntiles - 1;
      for (int i = 0; i < nt && ok; ++i) {
        if (lane == 0 && i == draw_at) drawn = atomicAdd(A.next_chunk, 1u) + gridDim.x;
        const int t = tile_of(A, t0, cstride, chunk_order(i, nt, rl));
        if (!DMX_IN_RANGE(A.err, t, A.ntiles)) continue;
        const int64_t tile_begin = (int64_t)t * T;
        if (tile_begin + T > A.P) continue;  // the ragged last tile is read by the consumers with plain loads
        for (int k0 = 0; k0 < A.K; k0 += G) {
          ok = __all_sync(0xffffffffu, mbar_wait(empty_g + 8 * stage, phase ^ 1u, give_up, A.err));
          if (!ok) break;
          const int n = A.K - k0 < G ? A.K - k0 : G;
          if (lane == 0) mbar_expect_tx(full_g + 8 * stage, (uint32_t)n * C::SLOT);
          armed_g |= 1u << stage;
          par_g = (par_g & ~(1u << stage)) | (phase << stage);
          __syncwarp();
          if (lane < n)
            bulk_load(ring + stage * C::STAGE + lane * C::SLOT,
                      static_cast<const unsigned char*>(A.grad[k0 + lane]) + tile_begin * ESZ, C::SLOT, full_g + 8 * stage, pol);
          if (++stage == NSTAGE) { stage = 0; phase ^= 1u; }
        }
        if (!ok) break;
        ok = __all_sync(0xffffffffu, mbar_wait(empty_s + 8 * ss, sphase ^ 1u, give_up, A.err));
        if (!ok) break;
        if (lane == 0) mbar_expect_tx(full_s + 8 * ss, C::SSTAGE);
        armed_s |= 1u << ss;
        par_s = (par_s & ~(1u << ss)) | (sphase << ss);
        __syncwarp();
        if (lane < C::NST) {
          const float* src = lane == 0 ? A.prev : (lane == 1 ? A.momentum : (lane == 2 ? A.params : A.second));
          bulk_load(sring + ss * C::SSTAGE + lane * C::SSLOT, src + tile_begin, C::SSLOT, full_s + 8 * ss, pol);
        }
        if (++ss == NSS) { ss = 0; sphase ^= 1u; }
      }
      if (lane == 0) {
        cur = -1;
        if (drawn < (unsigned)A.nchunks) {
          cur = (int)drawn;
          c_t0 = A.chunk_tile0[cur]; c_nt = A.chunk_ntiles[cur]; c_stride = A.chunk_stride[cur]; c_slot0 = A.chunk_slot0[cur];
        }
      }
    }
    if (!ok && lane == 0) {
      // gave up: let the copies already issued land before the CTA's shared memory is released
      for (uint32_t i = 0; i < (uint32_t)NSTAGE; ++i) {
        if (!((armed_g >> i) & 1u)) continue;
        for (uint32_t n = 0; n < kWaitLimit && !mbar_try_wait(full_g + 8 * i, (par_g >> i) & 1u); ++n) {}
      }
      for (uint32_t i = 0; i < (uint32_t)NSS; ++i) {
        if (!((armed_s >> i) & 1u)) continue;
        for (uint32_t n = 0; n < kWaitLimit && !mbar_try_wait(full_s + 8 * i, (par_s >> i) & 1u); ++n) {}
      }
    }
    return;
  }

  // ---------------- consumers ----------------
  const int tid = threadIdx.x;  // 0 .. CT-1
  Acc<KT, VEC> a;
  a.reset_chunk();
  MbarSync sy;
  sy.bar = csync; sy.phase = 0u; sy.give_up = give_up; sy.err = A.err; sy.lane = lane;
  uint32_t stage = 0, phase = 0, ss = 0, sphase = 0, qi = 0, qphase = 0;
  bool ok = true;
  SegState st; st.par = 0;
  for (;;) {
    // next chunk of this CTA, as drawn by the producer; a failed wait ends the CTA's work
    ok = mbar_wait(full_q + 8 * qi, qphase, give_up, A.err) && ok;
    volatile int* qe = queue + 8 * qi;
    const int c = ok ? qe[0] : -1;
    const int t0 = qe[1], nt = qe[2], cstride = qe[3], slot0 = qe[4];
    __syncwarp();
    if (lane == 0) mbar_arrive(empty_q + 8 * qi);
    if (++qi == QN) { qi = 0; qphase ^= 1u; }
    if (c < 0) break;
    const bool rl = A.P % T != 0 && tile_of(A, t0, cstride, nt - 1) == A.ntiles - 1;
    st.begin_chunk();
    for (int i = 0; i < nt; ++i) {
      const int t = tile_of(A, t0, cstride, chunk_order(i, nt, rl));
      if (!DMX_IN_RANGE(A.err, t, A.ntiles)) continue;
      const int tseg = A.tile_seg[t];          // needed only at the end of the tile: latency hidden
      const int64_t tile_begin = (int64_t)t * T;
      const int64_t jt = tile_begin + (int64_t)tid * VEC;
      int64_t tile_end = tile_begin + T;
      float dv[VEC], nv[VEC];
      if (tile_end <= A.P) {
#pragma unroll
        for (int s = 0; s < (KT + G - 1) / G; ++s) {
          if (s * G < A.K) {
            ok = mbar_wait(full_g + 8 * stage, phase, give_up, A.err) && ok;
            const uint32_t src = ring + stage * C::STAGE + tid * 16;
            // the stage's streams LB at a time: load, (after the last load: release the stage,) accumulate
#pragma unroll
            for (int u0 = 0; u0 < G; u0 += LB) {
              uint4 r[LB];
#pragma unroll
              for (int u = 0; u < LB; ++u)
                if (u0 + u < G && s * G + u0 + u < KT && s * G + u0 + u < A.K) r[u] = lds128(src + (u0 + u) * C::SLOT);
              if (u0 + LB >= G) {
                __syncwarp();
                if (lane == 0) mbar_arrive(empty_g + 8 * stage);
                if (++stage == NSTAGE) { stage = 0; phase ^= 1u; }
              }
#pragma unroll
              for (int u = 0; u < LB; ++u) {
                if (u0 + u < G && s * G + u0 + u < KT && s * G + u0 + u < A.K) {
                  u64 x[VEC / 2];
                  unpack2<BF16>(r[u], x);
                  a.add(s * G + u0 + u, x, A.w[s * G + u0 + u], A.bf[s * G + u0 + u], A.bd[s * G + u0 + u]);
                }
              }
            }
          }
        }
        ok = mbar_wait(full_s + 8 * ss, sphase, give_up, A.err) && ok;
        // the tile's state in halves of four elements: load, update, store (only one half's
        // values are live at a time; the stage is released after the last load)
        const uint32_t ssrc = sring + ss * C::SSTAGE + tid * (VEC * 4);
#pragma unroll
        for (int h = 0; h < VEC / 4; ++h) {
          float th[4], m[4], pv[4], vv[4];
          uint4 r = lds128(ssrc + 16 * h);                  unpack4f(r, pv);
          r = lds128(ssrc + C::SSLOT + 16 * h);             unpack4f(r, m);
          r = lds128(ssrc + 2 * C::SSLOT + 16 * h);         unpack4f(r, th);
          if constexpr (ADAM) { r = lds128(ssrc + 3 * C::SSLOT + 16 * h); unpack4f(r, vv); }
          if (h == VEC / 4 - 1) {
            __syncwarp();
            if (lane == 0) mbar_arrive(empty_s + 8 * ss);
            if (++ss == NSS) { ss = 0; sphase ^= 1u; }
          }
          if (h == 0) finish4<KT, VEC, ADAM, 0>(a, A, th, m, pv, dv, nv, vv);
          else finish4<KT, VEC, ADAM, (VEC == 8 ? 4 : 0)>(a, A, th, m, pv, dv, nv, vv);
          if (ok) {
            st_stream(A.params + jt + 4 * h, th[0], th[1], th[2], th[3]);
            st_stream(A.momentum + jt + 4 * h, m[0], m[1], m[2], m[3]);
            st_stream(A.prev + jt + 4 * h, pv[0], pv[1], pv[2], pv[3]);
            if constexpr (ADAM) st_stream(A.second + jt + 4 * h, vv[0], vv[1], vv[2], vv[3]);
          }
        }
      } else {
        tile_end = A.P;
        ragged_tile<KT, BF16, ADAM>(a, A, jt, dv, nv);
      }
      segment_accumulate<KT, VEC, CW>(a, A, dv, nv, jt, tile_begin, tile_end, tseg, R, st, slot0, sy, wid, lane);
    }
    flush_chunk<KT, VEC, CW, ADAM>(a, A, R, st, c, slot0, sy, wid, lane);
  }
}

// Self-test of the bounded wait: one warp waits, with a polling budget of `limit`, on an
// mbarrier that nothing will ever complete (no copy is in flight, nobody else arrives), so the
// wait must run out: it raises the give-up word and the handle's error word exactly as a wait
// of the fused pass would. out[0] = 1 if the wait reported failure, out[1] = the give-up word,
// out[2..3] = nanoseconds spent in the wait (%globaltimer).
static __global__ void __launch_bounds__(32) wait_selftest_kernel(unsigned* err, uint32_t limit, unsigned long long* out) {
  __shared__ __align__(8) unsigned long long bar_storage;
  __shared__ uint32_t give_up_word;
  const uint32_t bar = smem_u32(&bar_storage);
  if (threadIdx.x == 0) {
    mbar_init(bar, 1);
    give_up_word = 0u;
    asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory");
  }
  __syncwarp();
  unsigned long long t0, t1;
  asm volatile("mov.u64 %0, %globaltimer;" : "=l"(t0));
  const bool ok = mbar_wait(bar, 0u, &give_up_word, err, limit);
  asm volatile("mov.u64 %0, %globaltimer;" : "=l"(t1));
  __syncwarp();
  if (threadIdx.x == 0) {
    out[0] = ok ? 0ull : 1ull;
    out[1] = (unsigned long long)give_up_word;
    out[2] = t1 - t0;
  }
}

}  // namespace dmx

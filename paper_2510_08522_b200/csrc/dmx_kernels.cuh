// dmx_kernels.cuh — device code of the fused gradient step (sm_100a).
//
// One pass over the K gradient streams and the three fp32 state streams does, per parameter j:
//   g_j  = sum_k w_k x_kj                       (batch-size-weighted aggregate, w_k = b_k/B)
//   d_j  = sum_k b_k (x_kj - g_j)^2             (spread of the workers around it)
//   q_k += x_kj^2,  N_s += g_j^2,  V_s += d_j,  c += g_j a_j,  pp += a_j^2
//   m_j  = beta m_j + g_j,  theta_j -= lr m_j,  a_j = g_j
// The sums over k use the shifted one-pass form around a pivot worker (the one with the
// largest batch): with e_k = x_k - x_pivot,  g = x_pivot + sum w_k e_k  and
// d = sum b_k e_k^2 - B (sum w_k e_k)^2. Identical workers give d = 0 exactly, and the
// cancellation is between noise-sized terms only.
//
// Reductions are deterministic: per-thread fp32 partials over a "chunk" of tiles, warp
// shuffles, a fixed-order sum over the warps, one scratch row per chunk (and one scratch slot
// per (chunk, segment) pair), then an fp64 fixed-order second level in the finalize kernel.
// There are no floating-point atomics and no waits between CTAs.
#pragma once
#include <cuda_runtime.h>
#include <stdint.h>

namespace dmx {

constexpr int kMaxK = 64;

// Arguments of one step; passed by value as a __grid_constant__ kernel parameter, so a step
// needs no host-to-device copy. Worker arrays are in processing order (pivot first).
struct StepArgs {
  const void* grad[kMaxK];
  float w[kMaxK];        // b_k / B
  float bf[kMaxK];       // b_k
  float* params;
  float* momentum;
  float* prev;
  float lr, beta, Bf;
  int K, S;
  int64_t P;
  const int64_t* seg_off;      // S+1
  const int32_t* cta_chunk0;   // grid+1: chunks [cta_chunk0[b], cta_chunk0[b+1]) belong to CTA b
  const int32_t* chunk_tile0;  // nchunks+1: tiles [chunk_tile0[c], chunk_tile0[c+1])
  const int32_t* chunk_seg0;   // nchunks: segment holding the chunk's first element
  const int32_t* chunk_slot0;  // nchunks: first (V,N) slot of the chunk
  float* rows;                 // nchunks x (K+2): q_k..., c, pp
  float* slots;                // nslots x 2: V partial, N partial
  unsigned* err;               // set non-zero when a bounded wait gives up
};

struct FinalArgs {
  int K, S, nchunks;
  int orig[kMaxK];             // processing slot -> caller's worker index
  double b[kMaxK];             // batch sizes, processing order
  double B;
  const float* rows;
  const float* slots;
  const int32_t* chunk_seg0;
  const int32_t* chunk_slot0;
  const int32_t* seg_chunk_lo; // S: first chunk touching segment s (lo > hi: empty segment)
  const int32_t* seg_chunk_hi; // S
  double* colsum;              // K+2+2S
  unsigned* ticket;
  unsigned* err;
  float* out_state;
};

__device__ __forceinline__ float bits2f(uint32_t u) { return __uint_as_float(u); }

template <bool BF16> struct Elem;
template <> struct Elem<false> { static constexpr int VEC = 4; typedef float T; };
template <> struct Elem<true>  { static constexpr int VEC = 8; typedef uint16_t T; };

// 16 bytes of gradient -> VEC fp32 values
template <bool BF16>
__device__ __forceinline__ void unpack(const uint4& r, float* x) {
  if constexpr (BF16) {
    x[0] = bits2f(r.x << 16); x[1] = bits2f(r.x & 0xffff0000u);
    x[2] = bits2f(r.y << 16); x[3] = bits2f(r.y & 0xffff0000u);
    x[4] = bits2f(r.z << 16); x[5] = bits2f(r.z & 0xffff0000u);
    x[6] = bits2f(r.w << 16); x[7] = bits2f(r.w & 0xffff0000u);
  } else {
    x[0] = bits2f(r.x); x[1] = bits2f(r.y); x[2] = bits2f(r.z); x[3] = bits2f(r.w);
  }
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
  float p[VEC], s1[VEC], s2[VEC];   // pivot value, sum w e, sum b e^2
  float q[KT];                      // per-worker sum of squares (chunk)
  float c, pp, vs, ns;              // <g,a>, |a|^2, current segment's V and N partials (chunk)

  __device__ __forceinline__ void reset_chunk() {
#pragma unroll
    for (int k = 0; k < KT; ++k) q[k] = 0.f;
    c = pp = vs = ns = 0.f;
  }
  // k is a compile-time constant after unrolling at every call site, so q[k] is a register.
  __device__ __forceinline__ void add(int k, const float* x, float w, float bf) {
    float sq = 0.f;
    if (k == 0) {
#pragma unroll
      for (int e = 0; e < VEC; ++e) { p[e] = x[e]; s1[e] = 0.f; s2[e] = 0.f; sq = fmaf(x[e], x[e], sq); }
    } else {
#pragma unroll
      for (int e = 0; e < VEC; ++e) {
        const float d = x[e] - p[e];
        s1[e] = fmaf(w, d, s1[e]);
        s2[e] = fmaf(bf * d, d, s2[e]);
        sq = fmaf(x[e], x[e], sq);
      }
    }
    q[k] += sq;
  }
};

// Block-level pieces shared by both kernels. NW = number of participating warps; `bar_id`
// and `nthreads` name the barrier the participating threads meet on.
template <int NW>
__device__ __forceinline__ void named_sync(int bar_id) {
  asm volatile("bar.sync %0, %1;" :: "r"(bar_id), "r"(NW * 32) : "memory");
}

__device__ __forceinline__ float warp_sum(float v) {
#pragma unroll
  for (int o = 16; o > 0; o >>= 1) v += __shfl_xor_sync(0xffffffffu, v, o);
  return v;
}

// Sum (vs, ns) over the participating warps in warp order and store the pair to `dst`.
template <int NW>
__device__ __forceinline__ void flush_pair(float vs, float ns, float* red, float* dst, int bar_id,
                                           int wid, int lane) {
  vs = warp_sum(vs); ns = warp_sum(ns);
  named_sync<NW>(bar_id);                 // red[] free
  if (lane == 0) { red[2 * wid] = vs; red[2 * wid + 1] = ns; }
  named_sync<NW>(bar_id);
  if (wid == 0 && lane < 2) {
    float t = 0.f;
#pragma unroll
    for (int w = 0; w < NW; ++w) t += red[2 * w + lane];
    dst[lane] = t;
  }
}

// End of a chunk: q_k, c, pp -> its scratch row; (vs, ns) -> the slot of the current segment.
template <int KT, int VEC, int NW>
__device__ __forceinline__ void flush_chunk(Acc<KT, VEC>& a, int K, float* red, float* row,
                                            float* slot, int bar_id, int wid, int lane) {
  constexpr int NV = KT + 4;
  float v[NV];
#pragma unroll
  for (int k = 0; k < KT; ++k) v[k] = warp_sum(a.q[k]);
  v[KT] = warp_sum(a.c); v[KT + 1] = warp_sum(a.pp); v[KT + 2] = warp_sum(a.vs); v[KT + 3] = warp_sum(a.ns);
  named_sync<NW>(bar_id);
  if (lane == 0) {
#pragma unroll
    for (int i = 0; i < NV; ++i) red[wid * NV + i] = v[i];
  }
  named_sync<NW>(bar_id);
  const int t = wid * 32 + lane;
  if (t < NV) {
    float s = 0.f;
#pragma unroll
    for (int w = 0; w < NW; ++w) s += red[w * NV + t];
    if (t < KT) { if (t < K) row[t] = s; }
    else if (t < KT + 2) row[K + (t - KT)] = s;
    else slot[t - KT - 2] = s;
  }
  a.reset_chunk();
}

// Tile epilogue for one thread: aggregate, spread, update, statistics. `valid` = number of
// this thread's elements below P (VEC for full tiles). State values th/m/pv are inputs and
// are overwritten with the outputs (theta', m', g).
template <int KT, int VEC>
__device__ __forceinline__ void finish_elements(Acc<KT, VEC>& a, const StepArgs& A, float* th, float* m,
                                                float* pv, float* dv, float* nv) {
#pragma unroll
  for (int e = 0; e < VEC; ++e) {
    const float g = a.p[e] + a.s1[e];
    dv[e] = fmaf(-A.Bf * a.s1[e], a.s1[e], a.s2[e]);
    nv[e] = g * g;
    a.c = fmaf(g, pv[e], a.c);
    a.pp = fmaf(pv[e], pv[e], a.pp);
    const float mn = fmaf(A.beta, m[e], g);
    th[e] = fmaf(-A.lr, mn, th[e]);
    m[e] = mn;
    pv[e] = g;
  }
}

// Attribute the tile's per-element (d, g^2) to segments. Uniform control flow across the
// participating threads: cur_seg / next_bound are the same in all of them.
template <int KT, int VEC, int NW>
__device__ __forceinline__ void segment_accumulate(Acc<KT, VEC>& a, const StepArgs& A, const float* dv,
                                                   const float* nv, int64_t jt, int64_t tile_begin,
                                                   int64_t tile_end,
                                                   int& cur_seg, int64_t& next_bound, float* red,
                                                   int chunk_seg0, int chunk_slot0, int bar_id, int wid,
                                                   int lane) {
  if (next_bound >= tile_end || cur_seg >= A.S - 1) {
#pragma unroll
    for (int e = 0; e < VEC; ++e) { a.vs += dv[e]; a.ns += nv[e]; }
    return;
  }
  int64_t lo = tile_begin;  // nothing below it is pending
  while (cur_seg < A.S - 1 && next_bound < tile_end) {
#pragma unroll
    for (int e = 0; e < VEC; ++e) {
      const int64_t j = jt + e;
      if (j >= lo && j < next_bound) { a.vs += dv[e]; a.ns += nv[e]; }
    }
    flush_pair<NW>(a.vs, a.ns, red, A.slots + 2 * (int64_t)(chunk_slot0 + cur_seg - chunk_seg0), bar_id, wid, lane);
    a.vs = 0.f; a.ns = 0.f;
    lo = next_bound;
    ++cur_seg;
    next_bound = A.seg_off[cur_seg + 1];
  }
#pragma unroll
  for (int e = 0; e < VEC; ++e) {
    if (jt + e >= lo) { a.vs += dv[e]; a.ns += nv[e]; }
  }
}

// ------------------------------------------------------------------------------------------
// Direct kernel: every thread streams its own 16-byte pieces with plain vector loads, U
// worker loads in flight at a time. Also the code path of the ragged last tile.

template <int KT, bool BF16, bool GUARD, int U>
__device__ __forceinline__ void direct_tile(Acc<KT, Elem<BF16>::VEC>& a, const StepArgs& A, int64_t jt,
                                            float* dv, float* nv) {
  constexpr int VEC = Elem<BF16>::VEC;
  typedef typename Elem<BF16>::T GT;
#pragma unroll
  for (int k0 = 0; k0 < KT; k0 += U) {
    if (k0 < A.K) {
      float x[U][VEC];
#pragma unroll
      for (int u = 0; u < U; ++u) {
        if (k0 + u < KT && k0 + u < A.K) {
          const GT* src = static_cast<const GT*>(A.grad[k0 + u]) + jt;
          if constexpr (GUARD) {
#pragma unroll
            for (int e = 0; e < VEC; ++e) {
              if (jt + e < A.P) {
                if constexpr (BF16) x[u][e] = bits2f((uint32_t)src[e] << 16); else x[u][e] = src[e];
              } else x[u][e] = 0.f;
            }
          } else {
            const uint4 r = ld_stream(src);
            unpack<BF16>(r, x[u]);
          }
        }
      }
#pragma unroll
      for (int u = 0; u < U; ++u) {
        if (k0 + u < KT && k0 + u < A.K) a.add(k0 + u, x[u], A.w[k0 + u], A.bf[k0 + u]);
      }
    }
  }
  // state streams
  float th[VEC], m[VEC], pv[VEC];
  if constexpr (GUARD) {
#pragma unroll
    for (int e = 0; e < VEC; ++e) {
      const bool ok = jt + e < A.P;
      th[e] = ok ? A.params[jt + e] : 0.f; m[e] = ok ? A.momentum[jt + e] : 0.f; pv[e] = ok ? A.prev[jt + e] : 0.f;
    }
  } else {
#pragma unroll
    for (int h = 0; h < VEC / 4; ++h) {
      uint4 r = ld_stream(A.params + jt + 4 * h);   unpack<false>(r, th + 4 * h);
      r = ld_stream(A.momentum + jt + 4 * h);       unpack<false>(r, m + 4 * h);
      r = ld_stream(A.prev + jt + 4 * h);           unpack<false>(r, pv + 4 * h);
    }
  }
  finish_elements<KT, VEC>(a, A, th, m, pv, dv, nv);
  if constexpr (GUARD) {
#pragma unroll
    for (int e = 0; e < VEC; ++e) {
      if (jt + e < A.P) { A.params[jt + e] = th[e]; A.momentum[jt + e] = m[e]; A.prev[jt + e] = pv[e]; }
      else { dv[e] = 0.f; nv[e] = 0.f; }
    }
  } else {
#pragma unroll
    for (int h = 0; h < VEC / 4; ++h) {
      st_stream(A.params + jt + 4 * h, th[4 * h], th[4 * h + 1], th[4 * h + 2], th[4 * h + 3]);
      st_stream(A.momentum + jt + 4 * h, m[4 * h], m[4 * h + 1], m[4 * h + 2], m[4 * h + 3]);
      st_stream(A.prev + jt + 4 * h, pv[4 * h], pv[4 * h + 1], pv[4 * h + 2], pv[4 * h + 3]);
    }
  }
}

template <int KT, bool BF16, int NW, int U>
__global__ void __launch_bounds__(NW * 32)
direct_kernel(const __grid_constant__ StepArgs A) {
  constexpr int VEC = Elem<BF16>::VEC;
  constexpr int T = NW * 32 * VEC;
  __shared__ float red[NW * (KT + 4)];
  const int wid = threadIdx.x >> 5, lane = threadIdx.x & 31;
  Acc<KT, VEC> a;
  a.reset_chunk();
  const int c_begin = A.cta_chunk0[blockIdx.x], c_end = A.cta_chunk0[blockIdx.x + 1];
  for (int c = c_begin; c < c_end; ++c) {
    const int t0 = A.chunk_tile0[c], t1 = A.chunk_tile0[c + 1];
    const int seg0 = A.chunk_seg0[c], slot0 = A.chunk_slot0[c];
    int cur_seg = seg0;
    int64_t next_bound = A.seg_off[cur_seg + 1];
    for (int t = t0; t < t1; ++t) {
      const int64_t tile_begin = (int64_t)t * T;
      const int64_t jt = tile_begin + (int64_t)threadIdx.x * VEC;
      int64_t tile_end = tile_begin + T;
      float dv[VEC], nv[VEC];
      if (tile_end <= A.P) {
        direct_tile<KT, BF16, false, U>(a, A, jt, dv, nv);
      } else {
        tile_end = A.P;
        direct_tile<KT, BF16, true, U>(a, A, jt, dv, nv);
      }
      segment_accumulate<KT, VEC, NW>(a, A, dv, nv, jt, tile_begin, tile_end, cur_seg, next_bound, red, seg0, slot0, 1, wid, lane);
    }
    flush_chunk<KT, VEC, NW>(a, A.K, red, A.rows + (int64_t)c * (A.K + 2),
                             A.slots + 2 * (int64_t)(slot0 + cur_seg - seg0), 1, wid, lane);
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

__global__ void __launch_bounds__(kFinalWarps * 32) finalize_kernel(const __grid_constant__ FinalArgs F) {
  const int wid = threadIdx.x >> 5, lane = threadIdx.x & 31;
  const int K = F.K, S = F.S;
  const int ncols = K + 2 + 2 * S;
  const int col = blockIdx.x * kFinalWarps + wid;
  if (col < ncols) {
    double acc = 0.0;
    if (col < K + 2) {
      for (int c = lane; c < F.nchunks; c += 32) acc += (double)F.rows[(int64_t)c * (K + 2) + col];
    } else {
      const int which = (col - K - 2) >= S ? 1 : 0;
      const int s = (col - K - 2) - which * S;
      const int lo = F.seg_chunk_lo[s], hi = F.seg_chunk_hi[s];
      for (int c = lo + lane; c <= hi; c += 32)
        acc += (double)F.slots[2 * (int64_t)(F.chunk_slot0[c] + s - F.chunk_seg0[c]) + which];
    }
    acc = warp_sum_d(acc);
    if (lane == 0) F.colsum[col] = acc;
  }
  __shared__ unsigned s_last;
  __shared__ double s_red[2][kFinalWarps];
  __threadfence();
  __syncthreads();
  if (threadIdx.x == 0) s_last = (atomicAdd(F.ticket, 1u) == gridDim.x - 1) ? 1u : 0u;
  __syncthreads();
  if (!s_last) return;
  __threadfence();
  // last block: everything below reads colsum written by all blocks
  const volatile double* cs = F.colsum;
  double aV = 0.0, aN = 0.0;
  for (int s = threadIdx.x; s < S; s += blockDim.x) { aV += cs[K + 2 + s]; aN += cs[K + 2 + S + s]; }
  aV = warp_sum_d(aV); aN = warp_sum_d(aN);
  if (lane == 0) { s_red[0][wid] = aV; s_red[1][wid] = aN; }
  __syncthreads();
  const double inv = K >= 2 ? 1.0 / (double)(K - 1) : 0.0;
  float* out = F.out_state;
  for (int k = threadIdx.x; k < K; k += blockDim.x) out[16 + F.orig[k]] = (float)cs[k];
  for (int s = threadIdx.x; s < S; s += blockDim.x) {
    out[16 + K + s] = K >= 2 ? (float)(cs[K + 2 + s] / (double)(K - 1)) : 0.f;
    out[16 + K + S + s] = (float)cs[K + 2 + S + s];
  }
  if (threadIdx.x == 0) {
    double D = 0.0, A = 0.0, Qw = 0.0;
    for (int w = 0; w < kFinalWarps; ++w) { D += s_red[0][w]; A += s_red[1][w]; }
    bool bad = false;
    for (int k = 0; k < K; ++k) { Qw += F.b[k] * cs[k]; bad = bad || !isfinite((float)cs[k]); }
    const double c = cs[K], pp = cs[K + 1], B = F.B;
    int flags = 0;
    double trS = 0.0;
    if (K >= 2) trS = D * inv; else flags |= 8;
    const double G2 = A - trS / B;
    double gns = 0.0;
    if (G2 > 0.0) gns = trS / G2; else flags |= 2;
    double cosv = 0.0;
    if (A > 0.0 && pp > 0.0) cosv = c / sqrt(A * pp); else flags |= 4;
    const double sig2 = A > 0.0 ? trS / (B * A) : 0.0;
    const double sig = sqrt(sig2 > 0.0 ? sig2 : 0.0);
    if (bad || !isfinite((float)A) || !isfinite((float)pp)) flags |= 1;
    if (*reinterpret_cast<volatile unsigned*>(F.err) != 0u) { flags |= 16; *F.err = 0u; }
    out[0] = (float)B; out[1] = (float)A; out[2] = (float)trS; out[3] = (float)G2; out[4] = (float)gns;
    out[5] = (float)cosv; out[6] = (float)c; out[7] = (float)pp; out[8] = (float)sig2; out[9] = (float)sig;
    out[10] = (float)(Qw / B); out[11] = (float)flags;
    out[12] = out[13] = out[14] = out[15] = 0.f;
    *F.ticket = 0u;
  }
}

}  // namespace dmx

// ------------------------------------------------------------------------------------------
// Pipelined kernel: one producer thread streams whole tiles into a shared-memory ring with
// bulk asynchronous copies (the TMA engine; non-tensor 1-D form, no multicast) completing on
// mbarriers; CW consumer warps read 16 bytes per thread per stream from the ring and do the
// arithmetic. Every wait is bounded; a wait that runs out raises the handle's error word and
// the CTA drains without waiting any more.

namespace dmx {

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

constexpr uint32_t kWaitLimit = 1u << 24;

// Bounded wait. Returns false (at once) when the CTA has given up, and raises the give-up
// flag itself when its own polling budget runs out.
__device__ __forceinline__ bool mbar_wait(uint32_t bar, uint32_t parity, volatile uint32_t* give_up, unsigned* err) {
  if (mbar_try_wait(bar, parity)) return true;
  if (*give_up) return false;
  for (uint32_t i = 0; i < kWaitLimit; ++i) {
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

template <int KT_, bool BF16_, int CW_, int G_, int NSTAGE_, int NSS_>
struct PipeCfg {
  static constexpr int KT = KT_, CW = CW_, G = G_, NSTAGE = NSTAGE_, NSS = NSS_;
  static constexpr bool BF16 = BF16_;
  static constexpr int VEC = Elem<BF16>::VEC;
  static constexpr int CT = CW * 32;                 // consumer threads
  static constexpr int THREADS = CT + 32;            // + the producer warp
  static constexpr int T = CT * VEC;                 // elements per tile
  static constexpr int SLOT = CT * 16;               // one gradient stream's tile, bytes
  static constexpr int STAGE = G * SLOT;
  static constexpr int SSLOT = T * 4;                // one state stream's tile, bytes
  static constexpr int SSTAGE = 3 * SSLOT;
  static constexpr int RING = NSTAGE * STAGE;
  static constexpr int SRING = NSS * SSTAGE;
  static constexpr int RED = CW * (KT + 4) * 4;
  static constexpr int NBAR = 2 * NSTAGE + 2 * NSS;
  static constexpr size_t SMEM = (size_t)RING + SRING + RED + NBAR * 8 + 16;
};

template <class C>
__global__ void __launch_bounds__(C::THREADS, 1) pipe_kernel(const __grid_constant__ StepArgs A) {
  constexpr int KT = C::KT, VEC = C::VEC, CW = C::CW, G = C::G, NSTAGE = C::NSTAGE, NSS = C::NSS, T = C::T;
  constexpr bool BF16 = C::BF16;
  extern __shared__ __align__(128) unsigned char smem[];
  const uint32_t ring = smem_u32(smem);
  const uint32_t sring = ring + C::RING;
  float* red = reinterpret_cast<float*>(smem + C::RING + C::SRING);
  const uint32_t bars = sring + C::SRING + C::RED;
  volatile uint32_t* give_up = reinterpret_cast<volatile uint32_t*>(smem + C::RING + C::SRING + C::RED + C::NBAR * 8);
  // barrier i: full_g[i] = bars + 8 i ; empty_g[i] = bars + 8 (NSTAGE + i)
  //            full_s[i] = bars + 8 (2 NSTAGE + i) ; empty_s[i] = bars + 8 (2 NSTAGE + NSS + i)
  const uint32_t full_g = bars, empty_g = bars + 8 * NSTAGE, full_s = bars + 16 * NSTAGE, empty_s = full_s + 8 * NSS;
  const int wid = threadIdx.x >> 5, lane = threadIdx.x & 31;
  if (threadIdx.x == 0) {
    for (int i = 0; i < NSTAGE; ++i) { mbar_init(full_g + 8 * i, 1); mbar_init(empty_g + 8 * i, CW); }
    for (int i = 0; i < NSS; ++i) { mbar_init(full_s + 8 * i, 1); mbar_init(empty_s + 8 * i, CW); }
    *give_up = 0u;
    asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory");
    asm volatile("fence.proxy.async.shared::cta;" ::: "memory");
  }
  __syncthreads();
  const int c_begin = A.cta_chunk0[blockIdx.x], c_end = A.cta_chunk0[blockIdx.x + 1];
  constexpr int ESZ = BF16 ? 2 : 4;

  if (wid == CW) {
    // ---------------- producer ----------------
    if (lane != 0) return;
    const uint64_t pol = policy_evict_first();
    uint32_t stage = 0, phase = 0, ss = 0, sphase = 0;
    bool ok = true;
    const int t_begin = A.chunk_tile0[c_begin], t_end = A.chunk_tile0[c_end];
    for (int t = t_begin; t < t_end && ok; ++t) {
      const int64_t tile_begin = (int64_t)t * T;
      if (tile_begin + T > A.P) break;  // the ragged last tile is read with plain loads
      for (int k0 = 0; k0 < A.K && ok; k0 += G) {
        ok = mbar_wait(empty_g + 8 * stage, phase ^ 1u, give_up, A.err);
        if (!ok) break;
        const int n = A.K - k0 < G ? A.K - k0 : G;
        mbar_expect_tx(full_g + 8 * stage, (uint32_t)n * C::SLOT);
        for (int u = 0; u < n; ++u)
          bulk_load(ring + stage * C::STAGE + u * C::SLOT,
                    static_cast<const unsigned char*>(A.grad[k0 + u]) + tile_begin * ESZ, C::SLOT, full_g + 8 * stage, pol);
        if (++stage == NSTAGE) { stage = 0; phase ^= 1u; }
      }
      if (!ok) break;
      ok = mbar_wait(empty_s + 8 * ss, sphase ^ 1u, give_up, A.err);
      if (!ok) break;
      mbar_expect_tx(full_s + 8 * ss, C::SSTAGE);
      const uint32_t dst = sring + ss * C::SSTAGE;
      bulk_load(dst, A.prev + tile_begin, C::SSLOT, full_s + 8 * ss, pol);
      bulk_load(dst + C::SSLOT, A.momentum + tile_begin, C::SSLOT, full_s + 8 * ss, pol);
      bulk_load(dst + 2 * C::SSLOT, A.params + tile_begin, C::SSLOT, full_s + 8 * ss, pol);
      if (++ss == NSS) { ss = 0; sphase ^= 1u; }
    }
    if (!ok) {
      // gave up: let the copies already issued land before the CTA's shared memory is released
      for (uint32_t i = 0; i < (uint32_t)NSTAGE; ++i) {
        const uint32_t par = i < stage ? phase : phase ^ 1u;
        for (uint32_t n = 0; n < kWaitLimit && !mbar_try_wait(full_g + 8 * i, par); ++n) {}
      }
      for (uint32_t i = 0; i < (uint32_t)NSS; ++i) {
        const uint32_t par = i < ss ? sphase : sphase ^ 1u;
        for (uint32_t n = 0; n < kWaitLimit && !mbar_try_wait(full_s + 8 * i, par); ++n) {}
      }
    }
    return;
  }

  // ---------------- consumers ----------------
  const int tid = threadIdx.x;  // 0 .. CT-1
  Acc<KT, VEC> a;
  a.reset_chunk();
  uint32_t stage = 0, phase = 0, ss = 0, sphase = 0;
  bool ok = true;
  for (int c = c_begin; c < c_end; ++c) {
    const int t0 = A.chunk_tile0[c], t1 = A.chunk_tile0[c + 1];
    const int seg0 = A.chunk_seg0[c], slot0 = A.chunk_slot0[c];
    int cur_seg = seg0;
    int64_t next_bound = A.seg_off[cur_seg + 1];
    for (int t = t0; t < t1; ++t) {
      const int64_t tile_begin = (int64_t)t * T;
      const int64_t jt = tile_begin + (int64_t)tid * VEC;
      int64_t tile_end = tile_begin + T;
      float dv[VEC], nv[VEC];
      if (tile_end <= A.P) {
#pragma unroll
        for (int s = 0; s < (KT + G - 1) / G; ++s) {
          if (s * G < A.K) {
            ok = mbar_wait(full_g + 8 * stage, phase, give_up, A.err) && ok;
            uint4 r[G];
            const uint32_t src = ring + stage * C::STAGE + tid * 16;
#pragma unroll
            for (int u = 0; u < G; ++u)
              if (s * G + u < KT && s * G + u < A.K) r[u] = lds128(src + u * C::SLOT);
            __syncwarp();
            if (lane == 0) mbar_arrive(empty_g + 8 * stage);
            if (++stage == NSTAGE) { stage = 0; phase ^= 1u; }
#pragma unroll
            for (int u = 0; u < G; ++u) {
              if (s * G + u < KT && s * G + u < A.K) {
                float x[VEC];
                unpack<BF16>(r[u], x);
                a.add(s * G + u, x, A.w[s * G + u], A.bf[s * G + u]);
              }
            }
          }
        }
        ok = mbar_wait(full_s + 8 * ss, sphase, give_up, A.err) && ok;
        float th[VEC], m[VEC], pv[VEC];
        {
          const uint32_t src = sring + ss * C::SSTAGE + tid * (VEC * 4);
#pragma unroll
          for (int h = 0; h < VEC / 4; ++h) {
            uint4 r = lds128(src + 16 * h);               unpack<false>(r, pv + 4 * h);
            r = lds128(src + C::SSLOT + 16 * h);          unpack<false>(r, m + 4 * h);
            r = lds128(src + 2 * C::SSLOT + 16 * h);      unpack<false>(r, th + 4 * h);
          }
        }
        __syncwarp();
        if (lane == 0) mbar_arrive(empty_s + 8 * ss);
        if (++ss == NSS) { ss = 0; sphase ^= 1u; }
        finish_elements<KT, VEC>(a, A, th, m, pv, dv, nv);
        if (ok) {
#pragma unroll
          for (int h = 0; h < VEC / 4; ++h) {
            st_stream(A.params + jt + 4 * h, th[4 * h], th[4 * h + 1], th[4 * h + 2], th[4 * h + 3]);
            st_stream(A.momentum + jt + 4 * h, m[4 * h], m[4 * h + 1], m[4 * h + 2], m[4 * h + 3]);
            st_stream(A.prev + jt + 4 * h, pv[4 * h], pv[4 * h + 1], pv[4 * h + 2], pv[4 * h + 3]);
          }
        }
      } else {
        tile_end = A.P;
        direct_tile<KT, BF16, true, 4>(a, A, jt, dv, nv);
      }
      segment_accumulate<KT, VEC, CW>(a, A, dv, nv, jt, tile_begin, tile_end, cur_seg, next_bound, red, seg0, slot0, 1, wid, lane);
    }
    flush_chunk<KT, VEC, CW>(a, A.K, red, A.rows + (int64_t)c * (A.K + 2),
                             A.slots + 2 * (int64_t)(slot0 + cur_seg - seg0), 1, wid, lane);
  }
}

}  // namespace dmx

// dmx_static.cu — dmx_step_static: the gradient step for callers that must not allocate.
//
// Who needs it: code that runs where device allocation is off the table: inside a region
// whose memory is owned by a pool or a framework allocator that must see every byte, in a
// latency-critical loop where a cudaMalloc would synchronise the device, or in a process that
// has handed all of its memory budget to something else. dmx_create allocates tables and
// reduction scratch; this entry point needs neither a handle nor an allocation. Its reduction
// scratch is a fixed array in the library's device image, so every GPU that loads the library
// carries it (kScratchBytes) until the process exits.
//
// The price: the plain-load kernel with a contiguous range of tiles per CTA (slower than the
// pipelined kernel of dmx_step), at most DMX_STATIC_MAX_SEGMENTS segments, and one call at a
// time per GPU: all calls share the array.
#include "dmx.h"

#include <cstring>
#include <mutex>

#include "dmx_host.h"
#include "dmx_kernels.cuh"

namespace {

using dmxh::cuda_ok;

constexpr size_t kScratchBytes = DMX_STATIC_SCRATCH_BYTES;

// The scratch itself. In host code this name is only a handle for the runtime's symbol
// calls, never an address a kernel can use: the device address comes from
// cudaGetSymbolAddress (see device_scratch below).
static __device__ __align__(256) unsigned char g_scratch[kScratchBytes];

struct StaticArgs {
  int grid;
  int64_t ntiles;
  const int64_t* seg_off;   // S+1, in the scratch
  float* rows;              // (K+2) x grid, one column after the other
  float2* cells;            // grid x S: (V, N) partial of CTA b for segment s
};

struct StaticFinal {
  int K, S, grid;
  int orig[dmx::kMaxK];
  double b[dmx::kMaxK];
  double B;
  const float* rows;
  const float2* cells;
  float* out_state;
};

constexpr int NW = 8;  // warps per CTA

// Sum (vs, ns) over the CTA in warp order and store the pair to *dst (all threads call it).
__device__ __forceinline__ void block_pair(float vs, float ns, float (*red)[2], float2* dst, int wid, int lane) {
  vs = dmx::warp_sum(vs); ns = dmx::warp_sum(ns);
  __syncthreads();
  if (lane == 0) { red[wid][0] = vs; red[wid][1] = ns; }
  __syncthreads();
  if (threadIdx.x == 0) {
    float v = 0.f, n = 0.f;
#pragma unroll
    for (int w = 0; w < NW; ++w) { v += red[w][0]; n += red[w][1]; }
    *dst = make_float2(v, n);
  }
}

// A variant of the plain-load kernel: CTA b takes tiles [ntiles b/grid, ntiles (b+1)/grid),
// keeps its partial sums in registers over the whole range and writes them to its own row of
// the static scratch. Nothing is shared between CTAs, so there are no atomics and no waits.
template <int KT, bool BF16>
__global__ void __launch_bounds__(NW * 32) static_step_kernel(const __grid_constant__ dmx::StepArgs A,
                                                            const __grid_constant__ StaticArgs X) {
  constexpr int VEC = dmx::Elem<BF16>::VEC;
  constexpr int T = NW * 32 * VEC;
  __shared__ float red2[NW][2];
  __shared__ float redq[NW][KT + 2];
  const int wid = threadIdx.x >> 5, lane = threadIdx.x & 31;
  const int b = blockIdx.x, S = A.S;
  float2* my_cells = X.cells + (int64_t)b * S;
  // the array keeps the previous call's contents: every cell of this CTA starts at zero
  for (int s = threadIdx.x; s < S; s += NW * 32) my_cells[s] = make_float2(0.f, 0.f);
  __syncthreads();
  const int64_t t0 = X.ntiles * b / X.grid, t1 = X.ntiles * (b + 1) / X.grid;
  dmx::Acc<KT, VEC> a;
  a.reset_chunk();
  // segment holding the CTA's first element
  int cur = 0;
  {
    const int64_t j0 = t0 * T;
    int lo = 0, hi = S - 1;
    while (lo < hi) {
      const int mid = (lo + hi + 1) >> 1;
      if (X.seg_off[mid] <= j0) lo = mid; else hi = mid - 1;
    }
    cur = lo;
  }
  int64_t next_bound = X.seg_off[cur + 1];
  for (int64_t t = t0; t < t1; ++t) {
    const int64_t tile_begin = t * T;
    const int64_t jt = tile_begin + (int64_t)threadIdx.x * VEC;
    int64_t tile_end = tile_begin + T;
    float dv[VEC], nv[VEC];
    if (tile_end <= A.P) {
      dmx::direct_tile<KT, BF16, false, 4>(a, A, jt, dv, nv);
    } else {
      tile_end = A.P;
      dmx::direct_tile<KT, BF16, true, 4>(a, A, jt, dv, nv);
    }
    if (next_bound >= tile_end || cur >= S - 1) {
#pragma unroll
      for (int e = 0; e < VEC; ++e) { a.vs += dv[e]; a.ns += nv[e]; }
    } else {
      int64_t lo = tile_begin;
      while (cur < S - 1 && next_bound < tile_end) {       // uniform across the CTA
#pragma unroll
        for (int e = 0; e < VEC; ++e) {
          const int64_t j = jt + e;
          if (j >= lo && j < next_bound) { a.vs += dv[e]; a.ns += nv[e]; }
        }
        block_pair(a.vs, a.ns, red2, my_cells + cur, wid, lane);
        a.vs = 0.f; a.ns = 0.f;
        lo = next_bound;
        ++cur;
        next_bound = X.seg_off[cur + 1];
      }
#pragma unroll
      for (int e = 0; e < VEC; ++e)
        if (jt + e >= lo) { a.vs += dv[e]; a.ns += nv[e]; }
    }
  }
  if (t1 > t0) block_pair(a.vs, a.ns, red2, my_cells + cur, wid, lane);
  // q_k, c, pp of this CTA
  constexpr int NV = KT + 2;
  float v[NV];
#pragma unroll
  for (int k = 0; k < KT; ++k) v[k] = dmx::warp_sum(a.q[k]);
  v[KT] = dmx::warp_sum(a.c); v[KT + 1] = dmx::warp_sum(a.pp);
  if (lane == 0) {
#pragma unroll
    for (int i = 0; i < NV; ++i) redq[wid][i] = v[i];
  }
  __syncthreads();
  if (threadIdx.x < NV) {
    const int t = threadIdx.x;
    float s = 0.f;
#pragma unroll
    for (int w = 0; w < NW; ++w) s += redq[w][t];
    if (t < KT) { if (t < A.K) X.rows[(int64_t)t * X.grid + b] = s; }
    else X.rows[(int64_t)(A.K + t - KT) * X.grid + b] = s;
  }
}

// Second level for the static path: one CTA; fp64, fixed order. The derived scalars come from
// the same device function as the handle path's (dmx::emit_header).
__global__ void __launch_bounds__(NW * 32) static_finalize_kernel(const __grid_constant__ StaticFinal F) {
  __shared__ double cs[dmx::kMaxK + 2 + 2 * DMX_STATIC_MAX_SEGMENTS];
  __shared__ double s_red[2][NW];
  const int wid = threadIdx.x >> 5, lane = threadIdx.x & 31;
  const int K = F.K, S = F.S;
  for (int unit = wid; unit < K + 2 + S; unit += NW) {
    if (unit < K + 2) {
      double acc = 0.0;
      for (int b = lane; b < F.grid; b += 32) acc += (double)F.rows[(int64_t)unit * F.grid + b];
      acc = dmx::warp_sum_d(acc);
      if (lane == 0) cs[unit] = acc;
    } else {
      const int s = unit - (K + 2);
      double v = 0.0, n = 0.0;
      for (int b = lane; b < F.grid; b += 32) {
        const float2 t = F.cells[(int64_t)b * S + s];
        v += (double)t.x; n += (double)t.y;
      }
      v = dmx::warp_sum_d(v); n = dmx::warp_sum_d(n);
      if (lane == 0) { cs[K + 2 + s] = v; cs[K + 2 + S + s] = n; }
    }
  }
  __syncthreads();
  double aV = 0.0, aN = 0.0;
  for (int s = threadIdx.x; s < S; s += blockDim.x) { aV += cs[K + 2 + s]; aN += cs[K + 2 + S + s]; }
  aV = dmx::warp_sum_d(aV); aN = dmx::warp_sum_d(aN);
  if (lane == 0) { s_red[0][wid] = aV; s_red[1][wid] = aN; }
  __syncthreads();
  float* out = F.out_state;
  for (int k = threadIdx.x; k < K; k += blockDim.x) out[DMX_ST_HDR + F.orig[k]] = (float)cs[k];
  for (int s = threadIdx.x; s < S; s += blockDim.x) {
    out[DMX_ST_HDR + K + s] = K >= 2 ? (float)(cs[K + 2 + s] / (double)(K - 1)) : 0.f;
    out[DMX_ST_HDR + K + S + s] = (float)cs[K + 2 + S + s];
  }
  if (threadIdx.x == 0) {
    double D = 0.0, A = 0.0, Qw = 0.0;
    for (int w = 0; w < NW; ++w) { D += s_red[0][w]; A += s_red[1][w]; }
    bool bad = false;
    for (int k = 0; k < K; ++k) { Qw += F.b[k] * cs[k]; bad = bad || !isfinite((float)cs[k]); }
    dmx::emit_header(out, K, F.B, D, A, Qw, cs[K], cs[K + 1], bad, false, 0, 0.0, 0.0, 0.0);
  }
}

typedef void (*StaticKernel)(const dmx::StepArgs, const StaticArgs);

template <bool BF16>
StaticKernel pick_kernel(int K) {
  if (K <= 4) return static_step_kernel<4, BF16>;
  if (K <= 8) return static_step_kernel<8, BF16>;
  if (K <= 16) return static_step_kernel<16, BF16>;
  if (K <= 32) return static_step_kernel<32, BF16>;
  return static_step_kernel<64, BF16>;
}

// Per-device set-up, done by the first call on each device with that device current: the
// device address of the scratch array and the number of SMs.
constexpr int kMaxDevices = 64;
struct DeviceInfo { bool ready = false; unsigned char* scratch = nullptr; int sms = 0; };
DeviceInfo g_dev[kMaxDevices];
std::mutex g_mu;

int device_scratch(DeviceInfo** out) {
  int dev = 0;
  if (!cuda_ok(cudaGetDevice(&dev)) || dev < 0 || dev >= kMaxDevices) return DMX_ERR_CUDA;
  std::lock_guard<std::mutex> lock(g_mu);
  DeviceInfo& d = g_dev[dev];
  if (!d.ready) {
    void* p = nullptr;
    if (!cuda_ok(cudaGetSymbolAddress(&p, g_scratch)) || !p) return DMX_ERR_CUDA;
    int sms = 0;
    if (!cuda_ok(cudaDeviceGetAttribute(&sms, cudaDevAttrMultiProcessorCount, dev)) || sms < 1) return DMX_ERR_CUDA;
    d.scratch = static_cast<unsigned char*>(p);
    d.sms = sms;
    d.ready = true;
  }
  *out = &d;
  return DMX_OK;
}

size_t align256(size_t x) { return (x + 255) & ~(size_t)255; }

}  // namespace

extern "C" int dmx_step_static(int K, int64_t P, const int64_t* seg_offsets, int S, int grad_dtype,
                               const void* const* grad_ptrs, const int32_t* batch_sizes, float* params,
                               float* momentum, float lr, float beta, float* prev_agg, float* out_state,
                               void* cuda_stream) {
  if (K < 1 || K > DMX_MAX_WORKERS || P < 1 || P >= DMX_MAX_PARAMS || S < 1 || !seg_offsets ||
      (grad_dtype != DMX_F32 && grad_dtype != DMX_BF16))
    return DMX_ERR_ARG;
  if (S > DMX_STATIC_MAX_SEGMENTS) return DMX_ERR_LIMIT;
  if (!grad_ptrs || !batch_sizes || !params || !momentum || !prev_agg || !out_state) return DMX_ERR_ARG;
  if (seg_offsets[0] != 0 || seg_offsets[S] != P) return DMX_ERR_SEGMENTS;
  for (int s = 0; s < S; ++s)
    if (seg_offsets[s] > seg_offsets[s + 1]) return DMX_ERR_SEGMENTS;
  const dmxh::StepBuffers sb = {grad_ptrs, batch_sizes, params, momentum, prev_agg, nullptr, out_state,
                                (size_t)(DMX_ST_HDR + K + 2 * S) * 4, 3u};
  int64_t B = 0;
  int pivot = 0;
  const int rcb = dmxh::check_step_buffers(K, P, grad_dtype, sb, &B, &pivot);
  if (rcb != DMX_OK) return rcb;

  DeviceInfo* dev = nullptr;
  const int rc = device_scratch(&dev);
  if (rc != DMX_OK) return rc;

  const bool bf16 = grad_dtype == DMX_BF16;
  const int tile = NW * 32 * (bf16 ? 8 : 4);
  const int64_t ntiles = (P + tile - 1) / tile;
  const int grid = (int)(ntiles < dev->sms ? ntiles : dev->sms);
  // carve the scratch: segment offsets | chunk rows | per-CTA segment cells
  const size_t off_seg = 0;
  const size_t off_rows = align256(off_seg + (size_t)(S + 1) * sizeof(int64_t));
  const size_t off_cells = align256(off_rows + (size_t)(K + 2) * grid * sizeof(float));
  const size_t need = off_cells + (size_t)grid * S * sizeof(float2);
  if (need > kScratchBytes) return DMX_ERR_LIMIT;

  dmx::StepArgs A;
  StaticArgs X;
  StaticFinal F;
  std::memset(&A, 0, sizeof(A));
  std::memset(&X, 0, sizeof(X));
  std::memset(&F, 0, sizeof(F));
  dmxh::pack_workers(K, grad_ptrs, batch_sizes, pivot, B, lr, beta, A, F.orig, F.b);   // as in dmx_step
  A.params = params; A.momentum = momentum; A.prev = prev_agg;
  A.K = K; A.S = S; A.P = P;
  X.grid = grid; X.ntiles = ntiles;
  X.seg_off = reinterpret_cast<const int64_t*>(dev->scratch + off_seg);
  X.rows = reinterpret_cast<float*>(dev->scratch + off_rows);
  X.cells = reinterpret_cast<float2*>(dev->scratch + off_cells);
  F.K = K; F.S = S; F.grid = grid; F.B = (double)B;
  F.rows = X.rows; F.cells = X.cells; F.out_state = out_state;

  cudaStream_t stream = static_cast<cudaStream_t>(cuda_stream);
  // the segment table travels host -> scratch on the stream (pageable source: the runtime
  // has taken its copy when the call returns)
  if (!cuda_ok(cudaMemcpyAsync(dev->scratch + off_seg, seg_offsets, (size_t)(S + 1) * sizeof(int64_t),
                               cudaMemcpyHostToDevice, stream)))
    return DMX_ERR_CUDA;
  StaticKernel kern = bf16 ? pick_kernel<true>(K) : pick_kernel<false>(K);
  kern<<<grid, NW * 32, 0, stream>>>(A, X);
  if (!cuda_ok(cudaGetLastError())) return DMX_ERR_CUDA;
  static_finalize_kernel<<<1, NW * 32, 0, stream>>>(F);
  if (!cuda_ok(cudaGetLastError())) return DMX_ERR_CUDA;
  return DMX_OK;
}

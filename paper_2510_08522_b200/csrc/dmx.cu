// dmx.cu — host side of the C ABI declared in dmx.h: validation, launch planning, the two
// launches of a step (fused pass, finalize). All device work of a step is in dmx_kernels.cuh.
#include "dmx.h"

#include <algorithm>
#include <cmath>
#include <cstdlib>
#include <cstring>
#include <mutex>
#include <new>
#include <unordered_map>
#include <vector>

#include <nvtx3/nvToolsExt.h>

#include "dmx_host.h"
#include "dmx_kernels.cuh"

namespace {
thread_local int g_last_cuda = 0;
thread_local int g_alloc_count = 0, g_alloc_fail = 0;
std::mutex g_live_mu;
std::unordered_map<const void*, int> g_live;
}

namespace dmxh {

bool cuda_ok(cudaError_t e) {
  if (e == cudaSuccess) return true;
  g_last_cuda = (int)e;
  (void)cudaGetLastError();
  return false;
}

static bool overlap(const void* a, size_t na, const void* b, size_t nb) {
  const uintptr_t x = (uintptr_t)a, y = (uintptr_t)b;
  return x < y + nb && y < x + na;
}

int check_step_buffers(int K, int64_t P, int grad_dtype, const StepBuffers& sb, int64_t* B, int* pivot) {
  if (!sb.grad_ptrs || !sb.batch_sizes || !sb.params || !sb.momentum || !sb.prev_agg || !sb.out) return DMX_ERR_ARG;
  const size_t gbytes = (size_t)P * (grad_dtype == DMX_BF16 ? 2 : 4), sbytes = (size_t)P * 4;
  *B = 0;
  *pivot = 0;
  for (int k = 0; k < K; ++k) {
    if (!sb.grad_ptrs[k]) return DMX_ERR_ARG;
    if (sb.batch_sizes[k] < 1) return DMX_ERR_BATCH;
    *B += sb.batch_sizes[k];
    if (sb.batch_sizes[k] > sb.batch_sizes[*pivot]) *pivot = k;
  }
  for (int k = 0; k < K; ++k)
    if ((uintptr_t)sb.grad_ptrs[k] & 15) return DMX_ERR_ALIGN;
  if (((uintptr_t)sb.params & 15) || ((uintptr_t)sb.momentum & 15) || ((uintptr_t)sb.prev_agg & 15) ||
      ((uintptr_t)sb.out & sb.out_align_mask) || ((uintptr_t)sb.second & 15))
    return DMX_ERR_ALIGN;
  const void* st[5] = {sb.params, sb.momentum, sb.prev_agg, sb.out, sb.second};
  const size_t sn[5] = {sbytes, sbytes, sbytes, sb.out_bytes, sbytes};
  const int nst = sb.second ? 5 : 4;
  for (int i = 0; i < nst; ++i) {
    for (int j = i + 1; j < nst; ++j)
      if (overlap(st[i], sn[i], st[j], sn[j])) return DMX_ERR_ARG;
    for (int k = 0; k < K; ++k)
      if (overlap(st[i], sn[i], sb.grad_ptrs[k], gbytes)) return DMX_ERR_ARG;
  }
  return DMX_OK;
}

void pack_workers(int K, const void* const* grad_ptrs, const int32_t* batch_sizes, int pivot, int64_t B, float lr,
                  float beta, dmx::StepArgs& A, int* orig, double* b) {
  int slot = 0;
  for (int i = -1; i < K; ++i) {
    const int k = i < 0 ? pivot : i;
    if (i >= 0 && k == pivot) continue;
    A.grad[slot] = grad_ptrs[k];
    A.w[slot] = (float)((double)batch_sizes[k] / (double)B);
    A.bf[slot] = (float)batch_sizes[k];
    A.bd[slot] = (double)batch_sizes[k];
    orig[slot] = k;
    b[slot] = (double)batch_sizes[k];
    ++slot;
  }
  A.lr = lr; A.beta = beta; A.Bf = (float)B;
  A.rB = 1.0 / (double)B; A.lr64 = (double)lr; A.beta64 = (double)beta;
}

void live_add(const void* p, int kind) {
  std::lock_guard<std::mutex> lock(g_live_mu);
  g_live[p] = kind;
}

bool live_has(const void* p, int kind) {
  if (!p) return false;
  std::lock_guard<std::mutex> lock(g_live_mu);
  const auto it = g_live.find(p);
  return it != g_live.end() && it->second == kind;
}

bool live_remove(const void* p, int kind) {
  std::lock_guard<std::mutex> lock(g_live_mu);
  const auto it = g_live.find(p);
  if (it == g_live.end() || it->second != kind) return false;
  g_live.erase(it);
  return true;
}

void alloc_begin() {
  g_alloc_count = 0;
  const char* v = std::getenv("DMX_TEST_FAIL_ALLOC");
  g_alloc_fail = (v && *v) ? std::atoi(v) : 0;
}

bool alloc_host_ok() { return ++g_alloc_count != g_alloc_fail; }

bool dev_alloc(void** p, size_t bytes) {
  *p = nullptr;
  if (++g_alloc_count == g_alloc_fail) {
    g_last_cuda = (int)cudaErrorMemoryAllocation;
    return false;
  }
  return cuda_ok(cudaMalloc(p, bytes));
}

int check_current_device(int device) {
  int cur = -1;
  if (!cuda_ok(cudaGetDevice(&cur))) return DMX_ERR_CUDA;
  return cur == device ? DMX_OK : DMX_ERR_HANDLE;
}

}  // namespace dmxh

namespace {

using dmxh::cuda_ok;

bool live(const dmx_handle* h) { return dmxh::live_has(h, dmxh::kStepHandle); }

typedef void (*StepKernel)(const dmx::StepArgs);

struct Plan {
  StepKernel kernel = nullptr;       // SGD-momentum update
  StepKernel kernel_adam = nullptr;  // Adam update (one more state stream)
  int threads = 0;       // threads per CTA
  int tile = 0;          // elements per tile
  size_t smem = 0, smem_adam = 0;    // dynamic shared memory
  int grid = 0;
};

int env_int(const char* name, int dflt) {
  const char* v = std::getenv(name);
  if (!v || !*v) return dflt;
  return std::atoi(v);
}

template <typename T>
bool upload(const std::vector<T>& v, T** dptr) {
  *dptr = nullptr;
  if (v.empty()) return true;
  if (!dmxh::dev_alloc((void**)dptr, v.size() * sizeof(T))) return false;
  return cuda_ok(cudaMemcpy(*dptr, v.data(), v.size() * sizeof(T), cudaMemcpyHostToDevice));
}

}  // namespace

struct dmx_handle {
  int K = 0, S = 0, dtype = 0, device = 0;
  int64_t P = 0;
  Plan plan;
  int nchunks = 0, nslots = 0, tile_group = 1;
  int64_t ntiles = 0;
  // device tables
  int64_t* seg_off = nullptr;
  int32_t *tile_seg = nullptr, *chunk_stride = nullptr, *chunk_tile0 = nullptr, *chunk_ntiles = nullptr;
  int32_t *chunk_slot0 = nullptr, *slot_dest = nullptr, *seg_ptr = nullptr, *unit_lo = nullptr, *unit_hi = nullptr,
          *seg_unit_ptr = nullptr;
  double2* segpart = nullptr;
  int nunits = 0;
  // device scratch; each array sits between two guard regions (see alloc_guarded)
  float* rows = nullptr;
  float2* slots = nullptr;
  double* colsum = nullptr;
  unsigned* flags = nullptr;  // [0] ticket, [1] err, [2] the fused pass's chunk counter
  struct Guarded { unsigned char* raw; size_t bytes; };
  std::vector<Guarded> guarded;
  // optional per-kernel timing
  bool profiling = false, profiled = false;
  cudaEvent_t ev[3] = {nullptr, nullptr, nullptr};
};

namespace {

// Kernel table: capacity KT in {4, 8, 16, 32, 64} (runtime K <= KT), fp32 / bf16 gradients.
template <int KT, bool BF16>
Plan direct_plan() {
  constexpr int NW = 8;
  constexpr int U = BF16 ? 4 : 8;
  Plan p;
  p.kernel = dmx::direct_kernel<KT, BF16, NW, U, false>;
  p.kernel_adam = dmx::direct_kernel<KT, BF16, NW, U, true>;
  p.threads = NW * 32;
  p.tile = NW * 32 * dmx::Elem<BF16>::VEC;
  p.smem = 0;
  return p;
}

template <bool BF16>
Plan pick_direct(int K) {
  if (K <= 4) return direct_plan<4, BF16>();
  if (K <= 8) return direct_plan<8, BF16>();
  if (K <= 16) return direct_plan<16, BF16>();
  if (K <= 32) return direct_plan<32, BF16>();
  return direct_plan<64, BF16>();
}

// Pipelined (bulk-copy ring) kernels. Ring geometry. A CTA of up to 8 warps may use 255 registers
// per thread, one of 9 to 12 warps 168 (registers are allocated per scheduler: three warps there
// instead of two).
//  - bf16 gradients, and fp32 gradients for more than 32 workers: 7 consumer warps + the
//    producer. A thread holds 8 elements (bf16) or 64 per-worker sums and needs more than 168
//    registers (with 11 consumer warps the K = 32 bf16 kernel spilled and lost 1-7 %).
//  - fp32 gradients, up to 32 workers: 11 consumer warps + the producer; 168 registers suffice
//    when a thread loads a stage's streams four at a time instead of all at once. More warps hide
//    the consumers' latencies better: K = 8 128 -> 118 us per step (the fp64 aggregate had made 7
//    warps the limiter), K = 32 +1.6 % at full clock and +6.7 % when the board's power limit has
//    lowered the SM clock (3331 -> 3122 us back to back, same box).
// A stage holds up to 16 gradient streams (8 in the 11-warp kernels, whose tile pieces are
// larger): 45-56 KB. The consumers pay one wait, one release and one batch of shared-memory loads
// per stage, and with 4 streams per stage (14 KB) that per-stage work made the consumers the limiter as
// soon as the SM clock dropped under the power limit (steps launched back to back: 5.8 -> 6.5 TB/s
// at K = 32 bf16, 6.2 -> 6.8 TB/s at K = 32 fp32; the time at full clock is unchanged).
// Stages smaller than 4 streams lose even at full clock.
// The producer runs at most NSS tiles ahead of the consumers (a tile's state stage is freed when
// the consumers have read it), so the bytes in flight per SM are min(ring, NSS tiles). With many
// workers one tile already fills the ring and one state stage is enough; with few workers a tile
// is small, and one state stage left only ~40 KB per SM in flight (0.76 of the copy rate at
// K = 8): there the ring is split into as many whole tiles (gradient stages + a state stage
// each) as fit.
template <int KT, bool BF16, bool ADAM>
struct Ring {
  static constexpr bool kWide = !BF16 && KT <= 32;                                  // the 11-consumer-warp kernels
  static constexpr int CW = kWide ? 11 : 7;
  static constexpr int G = KT < 16 ? KT : (kWide ? 8 : 16);                         // gradient streams per stage
  static constexpr int LB = (kWide && G > 4) ? 4 : G;                               // streams loaded before they are accumulated
  static constexpr int kStage = CW * 32 * 16 * G;                                   // bytes of a gradient stage
  static constexpr int kState = CW * 32 * (BF16 ? 8 : 4) * 4 * (ADAM ? 4 : 3);      // bytes of a state stage
  static constexpr int kTile = (KT + G - 1) / G * kStage + kState;                  // shared memory of one tile
  static constexpr int kAhead = 240 * 1024 / kTile;
  static constexpr int NSS = kAhead < 1 ? 1 : (kAhead > 8 ? 8 : kAhead);
  static constexpr int kRed = (int)((sizeof(dmx::RedArea<KT, CW>) + 15) / 16 * 16);
  static constexpr int kFit = (227 * 1024 - NSS * (kState + 16) - kRed - 128) / (kStage + 16);
  static constexpr int NSTAGE = kFit > 32 ? 32 : kFit;
  static_assert(NSTAGE >= 2, "the ring needs two gradient stages");
  typedef dmx::PipeCfg<KT, BF16, CW, G, NSTAGE, NSS, ADAM, LB> Cfg;
};

template <int KT, bool BF16>
Plan pipe_plan() {
  typedef typename Ring<KT, BF16, false>::Cfg C;
  typedef typename Ring<KT, BF16, true>::Cfg CA;
  static_assert(C::T == CA::T && C::THREADS == CA::THREADS, "both updates share the tile tables");
  Plan p;
  p.kernel = dmx::pipe_kernel<C>;
  p.kernel_adam = dmx::pipe_kernel<CA>;
  p.threads = C::THREADS;
  p.tile = C::T;
  p.smem = C::SMEM;
  p.smem_adam = CA::SMEM;
  return p;
}

template <bool BF16>
Plan pick_pipe(int K) {
  if (K <= 4) return pipe_plan<4, BF16>();
  if (K <= 8) return pipe_plan<8, BF16>();
  if (K <= 16) return pipe_plan<16, BF16>();
  if (K <= 32) return pipe_plan<32, BF16>();
  return pipe_plan<64, BF16>();
}

// The chunk list of a problem: a function of (P, K, dtype, tile, resident CTAs, knobs) only.
//
// Tiles are taken in groups of R consecutive tiles; a chunk is a few groups, interleaved with
// the other chunks of its wave: chunk l of a wave of n chunks that starts at group g0 holds
// groups g0+l, g0+l+n, ... A full wave has one chunk per CTA. Chunks are about a sixth of a
// CTA's share, at most 32 tiles (so that fp32 per-thread partials stay short) and at least 8:
// SM speeds drift during a kernel, and on the mid-sized workloads 16-tile chunks measured 3-4 %
// faster than 32-tile ones, while below 8 tiles the per-chunk work shows. Once fewer than two
// such waves remain, every wave takes about half of what is left, down to a minimum chunk, so
// that the CTAs finish together under the dynamic schedule. A chunk's sums do not depend on the
// CTA that computes it, so results are reproducible on a given device.
// Groups of 4 tiles measured 0.5-1 % faster than single tiles on the large workloads, groups of
// 2 about 1 % faster on the mid-sized ones.
struct ChunkPlan {
  int R = 1, grid = 1;
  std::vector<int32_t> tile0, ntiles, stride;   // per chunk: first tile, tiles, tiles between group starts
};

void plan_chunks(int64_t P, int K, int grad_dtype, int tile, int64_t sm_ctas, int want_R, int want_chunk, int want_min_kb,
                 ChunkPlan& cp) {
  const int64_t ntiles = (P + tile - 1) / tile;
  const int auto_R = ntiles >= 4 * 64 * sm_ctas ? 4 : (ntiles >= 32 * sm_ctas ? 2 : 1);
  const int R = std::max(1, std::min(want_R > 0 ? want_R : auto_R, 1 << 16));          // tiles per group
  const int64_t share = (ntiles + sm_ctas - 1) / sm_ctas;                              // tiles per CTA
  const int auto_chunk = (int)std::max<int64_t>(8, std::min<int64_t>(32, share / 6));
  const int chunk_groups = std::max(1, (want_chunk > 0 ? want_chunk : auto_chunk) / R);
  const int64_t ngroups = (ntiles + R - 1) / R;
  const int grid = (int)std::min<int64_t>(sm_ctas, ngroups);
  cp.R = R;
  cp.grid = grid;
  cp.tile0.clear(); cp.ntiles.clear(); cp.stride.clear();
  size_t last_tile_chunk = 0;                                   // the chunk that holds the last tile
  // smallest chunk: about 192 KB of streamed bytes (a few microseconds of one SM), so that the
  // per-chunk work (the draw, the reduction flush) stays small beside it
  const int64_t group_bytes = (int64_t)R * tile * ((int64_t)K * (grad_dtype == DMX_BF16 ? 2 : 4) + 24);
  const int64_t min_bytes = (int64_t)(want_min_kb > 0 ? want_min_kb : 192) * 1024;
  const int64_t min_groups = std::min<int64_t>(chunk_groups, std::max<int64_t>(1, (min_bytes + group_bytes - 1) / group_bytes));
  for (int64_t g0 = 0; g0 < ngroups;) {
    const int64_t rem = ngroups - g0;
    // a problem of less than two minimum chunks per CTA is one wave, split evenly (nothing to balance)
    const bool single = g0 == 0 && rem <= 2 * min_groups * (int64_t)grid;
    const int64_t ng = single ? (rem + grid - 1) / grid
                              : std::max<int64_t>(min_groups, std::min<int64_t>(chunk_groups, rem / (2 * (int64_t)grid)));
    const int64_t nl = single ? std::min<int64_t>(grid, rem) : std::min<int64_t>(grid, (rem + ng - 1) / ng);
    const int64_t wave = std::min<int64_t>(rem, nl * ng);      // groups g0 .. g0+wave-1, lane l takes g0+l, g0+l+nl, ...
    for (int64_t l = 0; l < nl; ++l) {
      const int64_t n_l = (wave - l + nl - 1) / nl;
      const int64_t glast = g0 + l + (n_l - 1) * nl;            // only the very last group may be cut short by ntiles
      cp.tile0.push_back((int32_t)((g0 + l) * R));
      cp.ntiles.push_back((int32_t)((n_l - 1) * R + std::min<int64_t>(R, ntiles - glast * R)));
      cp.stride.push_back((int32_t)(nl * R));
      if (glast == ngroups - 1) last_tile_chunk = cp.tile0.size() - 1;
    }
    g0 += wave;
  }
  // If the last tile is ragged it goes through the guarded plain-load path, several times slower
  // than a full tile: drawn near the end it would extend the kernel by that much (8 % at
  // P = 25.6 M), so its chunk is moved to the front of the list, where CTA 0 starts with it.
  if (P % tile != 0 && last_tile_chunk > 0) {
    for (std::vector<int32_t>* v : {&cp.tile0, &cp.ntiles, &cp.stride})
      std::rotate(v->begin(), v->begin() + last_tile_chunk, v->begin() + last_tile_chunk + 1);
  }
}

// Scratch that kernels write is allocated between two guard regions of kGuardBytes filled with a
// fixed word; dmx_check_guards reads them back. A write that strays just outside its array (the
// kind of bug no result check would notice if it landed in a neighbouring allocation) shows
// there. The array itself starts 256-byte aligned.
constexpr size_t kGuardBytes = 256;
constexpr uint32_t kGuardWord = 0x5afe6a4du;

template <typename T>
bool alloc_guarded(dmx_handle* h, T** p, size_t bytes) {
  *p = nullptr;
  const size_t body = (bytes + 255) & ~(size_t)255;
  void* raw = nullptr;
  if (!dmxh::dev_alloc(&raw, body + 2 * kGuardBytes)) return false;
  h->guarded.push_back({static_cast<unsigned char*>(raw), body});
  uint32_t pat[kGuardBytes / 4];
  for (uint32_t& w : pat) w = kGuardWord;
  unsigned char* base = static_cast<unsigned char*>(raw);
  if (!cuda_ok(cudaMemcpy(base, pat, kGuardBytes, cudaMemcpyHostToDevice)) ||
      !cuda_ok(cudaMemcpy(base + kGuardBytes + body, pat, kGuardBytes, cudaMemcpyHostToDevice)))
    return false;
  *p = reinterpret_cast<T*>(base + kGuardBytes);
  return true;
}

void free_handle(dmx_handle* h) {
  if (!h) return;
  cudaFree(h->seg_off); cudaFree(h->tile_seg); cudaFree(h->chunk_stride); cudaFree(h->chunk_tile0);
  cudaFree(h->chunk_ntiles); cudaFree(h->chunk_slot0); cudaFree(h->slot_dest); cudaFree(h->seg_ptr); cudaFree(h->unit_lo);
  cudaFree(h->unit_hi); cudaFree(h->seg_unit_ptr);
  for (const dmx_handle::Guarded& g : h->guarded) cudaFree(g.raw);
  for (int i = 0; i < 3; ++i)
    if (h->ev[i]) cudaEventDestroy(h->ev[i]);
  (void)cudaGetLastError();
  delete h;
}

}  // namespace

extern "C" {

int dmx_create(int K, int64_t P, const int64_t* seg_offsets, int S, int grad_dtype, dmx_handle** out) {
  if (!out) return DMX_ERR_ARG;
  *out = nullptr;
  if (K < 1 || K > DMX_MAX_WORKERS || P < 1 || P >= DMX_MAX_PARAMS || S < 1 || S > DMX_MAX_SEGMENTS ||
      !seg_offsets || (grad_dtype != DMX_F32 && grad_dtype != DMX_BF16))
    return DMX_ERR_ARG;
  if (seg_offsets[0] != 0 || seg_offsets[S] != P) return DMX_ERR_SEGMENTS;
  for (int s = 0; s < S; ++s)
    if (seg_offsets[s] > seg_offsets[s + 1]) return DMX_ERR_SEGMENTS;

  dmxh::alloc_begin();
  dmx_handle* h = dmxh::alloc_host_ok() ? new (std::nothrow) dmx_handle : nullptr;
  if (!h) return DMX_ERR_NOMEM;
  h->K = K; h->P = P; h->S = S; h->dtype = grad_dtype;
  cudaDeviceProp prop;
  if (!cuda_ok(cudaGetDevice(&h->device)) || !cuda_ok(cudaGetDeviceProperties(&prop, h->device))) {
    free_handle(h);
    return DMX_ERR_CUDA;
  }

  // DMX_KERNEL=direct selects the plain-load kernel (a tuning and cross-check knob); the
  // default is the bulk-copy pipeline.
  const char* kv = std::getenv("DMX_KERNEL");
  const bool direct = kv && std::strcmp(kv, "direct") == 0;
  Plan plan = direct ? (grad_dtype == DMX_BF16 ? pick_direct<true>(K) : pick_direct<false>(K))
                     : (grad_dtype == DMX_BF16 ? pick_pipe<true>(K) : pick_pipe<false>(K));
  if ((plan.smem > 48 * 1024 &&
       !cuda_ok(cudaFuncSetAttribute(plan.kernel, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)plan.smem))) ||
      (plan.smem_adam > 48 * 1024 &&
       !cuda_ok(cudaFuncSetAttribute(plan.kernel_adam, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)plan.smem_adam)))) {
    free_handle(h);
    return DMX_ERR_CUDA;
  }
  int occ = 0;
  if (!cuda_ok(cudaOccupancyMaxActiveBlocksPerMultiprocessor(&occ, plan.kernel, plan.threads, plan.smem)) || occ < 1) {
    free_handle(h);
    return DMX_ERR_CUDA;
  }
  const int want = env_int("DMX_CTAS_PER_SM", 0);   // tuning knob: resident CTAs per SM (0 = all that fit)
  if (want > 0 && want < occ) occ = want;
  const int64_t ntiles = (P + plan.tile - 1) / plan.tile;
  const int64_t sm_ctas = (int64_t)prop.multiProcessorCount * occ;
  ChunkPlan cp;
  plan_chunks(P, K, grad_dtype, plan.tile, sm_ctas, env_int("DMX_TILE_GROUP", 0), env_int("DMX_CHUNK_TILES", 0),
              env_int("DMX_MIN_CHUNK_KB", 0), cp);
  const int R = cp.R;
  plan.grid = cp.grid;
  h->plan = plan;
  h->tile_group = R;
  // per-tile segment table
  std::vector<int32_t> tile_seg((size_t)ntiles);
  {
    int s = 0;
    for (int64_t t = 0; t < ntiles; ++t) {
      const int64_t j0 = t * plan.tile, j1 = std::min<int64_t>(j0 + plan.tile, P);
      while (seg_offsets[s + 1] <= j0) ++s;
      tile_seg[(size_t)t] = s | (seg_offsets[s + 1] < j1 && s < S - 1 ? dmx::kTileBoundaryBit : 0);
    }
  }
  std::vector<int32_t>&chunk_tile0 = cp.tile0, &chunk_ntiles = cp.ntiles, &chunk_stride = cp.stride;
  std::vector<int32_t> chunk_slot0;
  const int nchunks = (int)chunk_tile0.size();
  // Enumerate, with the kernel's own rules, the (V, N) entries every chunk emits: a new entry
  // whenever the running segment changes between tiles, at every boundary crossed inside a
  // tile, and at the end of the chunk.
  chunk_slot0.resize(nchunks);
  std::vector<int32_t> slot_seg;                             // segment of every slot, in slot order
  for (int c = 0; c < nchunks; ++c) {
    chunk_slot0[c] = (int32_t)slot_seg.size();
    int cur = -1;
    const int ntc = chunk_ntiles[c];
    const auto tile_at = [&](int i) { return chunk_tile0[c] + (int64_t)(i / R) * chunk_stride[c] + i % R; };
    const bool ragged_last = P % plan.tile != 0 && tile_at(ntc - 1) == ntiles - 1;
    for (int ii = 0; ii < ntc; ++ii) {
      const int64_t t = tile_at(dmx::chunk_order(ii, ntc, ragged_last));
      const int64_t j1 = std::min<int64_t>((t + 1) * plan.tile, P);
      const int s0 = tile_seg[(size_t)t] & (dmx::kTileBoundaryBit - 1);
      if (s0 != cur) {
        if (cur >= 0) slot_seg.push_back(cur);
        cur = s0;
      }
      if (tile_seg[(size_t)t] & dmx::kTileBoundaryBit) {
        while (cur < S - 1 && seg_offsets[cur + 1] < j1) { slot_seg.push_back(cur); ++cur; }
      }
    }
    if (cur >= 0) slot_seg.push_back(cur);
    if (slot_seg.size() > ((size_t)1 << 30)) { free_handle(h); return DMX_ERR_NOMEM; }
  }
  // the slots are stored grouped by segment (each group in entry order): entry i goes to slot_dest[i]
  const int64_t nslots = (int64_t)slot_seg.size();
  std::vector<int32_t> seg_ptr(S + 1, 0), slot_dest((size_t)nslots);
  for (int64_t i = 0; i < nslots; ++i) ++seg_ptr[slot_seg[(size_t)i] + 1];
  for (int s = 0; s < S; ++s) seg_ptr[s + 1] += seg_ptr[s];
  {
    std::vector<int32_t> fill(seg_ptr.begin(), seg_ptr.end() - 1);
    for (int64_t i = 0; i < nslots; ++i) slot_dest[(size_t)i] = fill[slot_seg[(size_t)i]]++;
  }
  // finalize units: runs of at most kFinalPart slots of one segment
  std::vector<int32_t> unit_lo, unit_hi, seg_unit_ptr(S + 1, 0);
  for (int s = 0; s < S; ++s) {
    seg_unit_ptr[s] = (int32_t)unit_lo.size();
    for (int32_t lo = seg_ptr[s]; lo < seg_ptr[s + 1]; lo += dmx::kFinalPart) {
      unit_lo.push_back(lo);
      unit_hi.push_back(std::min<int32_t>(lo + dmx::kFinalPart, seg_ptr[s + 1]));
    }
  }
  seg_unit_ptr[S] = (int32_t)unit_lo.size();
  h->nchunks = nchunks; h->nslots = (int)nslots; h->nunits = (int)unit_lo.size();
  h->ntiles = ntiles;

  std::vector<int64_t> seg(seg_offsets, seg_offsets + S + 1);
  bool ok = upload(seg, &h->seg_off) && upload(tile_seg, &h->tile_seg) && upload(chunk_stride, &h->chunk_stride) &&
            upload(chunk_tile0, &h->chunk_tile0) && upload(chunk_ntiles, &h->chunk_ntiles) &&
            upload(chunk_slot0, &h->chunk_slot0) && upload(slot_dest, &h->slot_dest) && upload(seg_ptr, &h->seg_ptr) &&
            upload(unit_lo, &h->unit_lo) &&
            upload(unit_hi, &h->unit_hi) && upload(seg_unit_ptr, &h->seg_unit_ptr);
  ok = ok && alloc_guarded(h, &h->segpart, (size_t)std::max(h->nunits, 1) * sizeof(double2));
  ok = ok && alloc_guarded(h, &h->rows, (size_t)nchunks * (K + 4) * sizeof(float));
  ok = ok && alloc_guarded(h, &h->slots, (size_t)std::max<int64_t>(nslots, 1) * sizeof(float2));
  ok = ok && alloc_guarded(h, &h->colsum, (size_t)(K + 4) * sizeof(double));
  ok = ok && alloc_guarded(h, &h->flags, 4 * sizeof(unsigned));
  ok = ok && cuda_ok(cudaMemset(h->flags, 0, 4 * sizeof(unsigned)));
  ok = ok && cuda_ok(cudaDeviceSynchronize());
  if (!ok) {
    const bool nomem = g_last_cuda == (int)cudaErrorMemoryAllocation;
    free_handle(h);
    return nomem ? DMX_ERR_NOMEM : DMX_ERR_CUDA;
  }
  dmxh::live_add(h, dmxh::kStepHandle);
  *out = h;
  return DMX_OK;
}

int dmx_state_len(const dmx_handle* h) {
  if (!live(h)) return DMX_ERR_HANDLE;
  return DMX_ST_HDR + h->K + 2 * h->S;
}

}  // extern "C"

namespace {

struct AdamParams { float* second; float beta2, eps; int64_t t; };

// A named range around the enqueueing of a step's launches, for timeline tools (NVTX; a call costs
// a pointer test when no tool is attached).
struct TraceRange {
  explicit TraceRange(const char* name) { nvtxRangePushA(name); }
  ~TraceRange() { nvtxRangePop(); }
  TraceRange(const TraceRange&) = delete;
  TraceRange& operator=(const TraceRange&) = delete;
};

// One step with either update; `ap` is null for SGD with momentum.
int step_impl(dmx_handle* h, const void* const* grad_ptrs, const int32_t* batch_sizes, float* params,
              float* momentum, float lr, float beta, float* prev_agg, float* out_state, void* cuda_stream,
              const AdamParams* ap, double* partials = nullptr) {
  // `partials` (a parameter shard of a larger problem): the raw sums go there and out_state is not written
  if (!live(h)) return DMX_ERR_HANDLE;
  if (!out_state && !partials) return DMX_ERR_ARG;
  if (ap && (!ap->second || ap->t < 1 || !(beta >= 0.f && beta < 1.f) || !(ap->beta2 >= 0.f && ap->beta2 < 1.f) ||
             !(ap->eps >= 0.f)))
    return DMX_ERR_ARG;
  const int K = h->K;
  dmxh::StepBuffers sb = {grad_ptrs, batch_sizes, params, momentum, prev_agg, ap ? ap->second : nullptr,
                          partials ? (const void*)partials : (const void*)out_state,
                          partials ? (size_t)(K + 5 + 2 * h->S) * 8 : (size_t)(DMX_ST_HDR + K + 2 * h->S) * 4,
                          partials ? 7u : 3u};
  int64_t B = 0;
  int pivot = 0;
  int rc = dmxh::check_step_buffers(K, h->P, h->dtype, sb, &B, &pivot);
  if (rc != DMX_OK) return rc;
  // the handle's tables and scratch live on the device that was current in dmx_create
  rc = dmxh::check_current_device(h->device);
  if (rc != DMX_OK) return rc;

  dmx::StepArgs A;
  dmx::FinalArgs F;
  std::memset(&A, 0, sizeof(A));
  std::memset(&F, 0, sizeof(F));
  // processing order: the worker with the largest batch first (the pivot), the others in
  // the caller's order
  dmxh::pack_workers(K, grad_ptrs, batch_sizes, pivot, B, lr, beta, A, F.orig, F.b);
  A.params = params; A.momentum = momentum; A.prev = prev_agg;
  if (ap) {
    // bias corrections in fp64 from the fp32 coefficients, handed over as fp32 factors
    A.second = ap->second; A.beta2 = ap->beta2; A.eps = ap->eps;
    A.omb1 = (float)(1.0 - (double)beta); A.omb2 = (float)(1.0 - (double)ap->beta2);
    A.c1 = (float)(1.0 / (1.0 - std::pow((double)beta, (double)ap->t)));
    A.c2 = (float)(1.0 / (1.0 - std::pow((double)ap->beta2, (double)ap->t)));
  }
  A.K = K; A.S = h->S; A.P = h->P;
  A.tile_group = h->tile_group; A.nchunks = h->nchunks;
  // the chunk counter is zero here: the finalize kernel of the previous step (or dmx_create) left it so,
  // which also makes a step that was captured in a CUDA graph replayable
  A.next_chunk = h->flags + 2;
  A.seg_off = h->seg_off; A.tile_seg = h->tile_seg; A.chunk_stride = h->chunk_stride; A.chunk_tile0 = h->chunk_tile0;
  A.chunk_ntiles = h->chunk_ntiles; A.chunk_slot0 = h->chunk_slot0; A.slot_dest = h->slot_dest;
  A.rows = h->rows; A.slots = h->slots; A.err = h->flags + 1;
  A.ntiles = (int)h->ntiles; A.nslots = h->nslots;

  F.K = K; F.S = h->S; F.nchunks = h->nchunks; F.B = (double)B;
  F.adam = ap ? 1 : 0; F.P = (double)h->P;
  F.rows = h->rows; F.slots = h->slots; F.seg_ptr = h->seg_ptr; F.nslots = h->nslots; F.nunits = h->nunits;
  F.unit_lo = h->unit_lo; F.unit_hi = h->unit_hi; F.seg_unit_ptr = h->seg_unit_ptr; F.segpart = h->segpart;
  F.colsum = h->colsum; F.ticket = h->flags; F.err = h->flags + 1; F.next_chunk = h->flags + 2;
  F.out_state = out_state;
  F.partials = partials;

  cudaStream_t stream = static_cast<cudaStream_t>(cuda_stream);
  const bool prof = h->profiling;
  const TraceRange step_range(ap ? "dmx_step_adam" : "dmx_step");
  if (prof && !cuda_ok(cudaEventRecord(h->ev[0], stream))) return DMX_ERR_CUDA;
  {
    const TraceRange r("dmx fused pass");
    if (ap) h->plan.kernel_adam<<<h->plan.grid, h->plan.threads, h->plan.smem_adam, stream>>>(A);
    else h->plan.kernel<<<h->plan.grid, h->plan.threads, h->plan.smem, stream>>>(A);
  }
  if (!cuda_ok(cudaGetLastError())) return DMX_ERR_CUDA;
  if (prof && !cuda_ok(cudaEventRecord(h->ev[1], stream))) return DMX_ERR_CUDA;
  const TraceRange fin_range("dmx finalize");
  // one block per chunk-row column, one warp per segment unit. Launched as a programmatic
  // dependent of the fused pass: its blocks may become resident while that kernel drains and
  // wait (griddepcontrol.wait) for its completion, which hides the launch latency between the
  // two kernels. With per-kernel timing on, the event between them needs the plain ordering.
  const int fblocks = K + 2 + 2 * F.adam + (h->nunits + dmx::kFinalWarps - 1) / dmx::kFinalWarps;
  cudaLaunchConfig_t cfg = {};
  cfg.gridDim = dim3((unsigned)fblocks);
  cfg.blockDim = dim3(dmx::kFinalWarps * 32);
  cfg.stream = stream;
  cudaLaunchAttribute attr[1] = {};
  attr[0].id = cudaLaunchAttributeProgrammaticStreamSerialization;
  attr[0].val.programmaticStreamSerializationAllowed = 1;
  cfg.attrs = attr;
  cfg.numAttrs = prof ? 0 : 1;
  if (!cuda_ok(cudaLaunchKernelEx(&cfg, dmx::finalize_kernel, F))) {
    (void)cudaMemsetAsync(h->flags, 0, 4 * sizeof(unsigned), stream);   // the fused pass ran: leave the handle usable
    return DMX_ERR_CUDA;
  }
  if (prof) {
    if (!cuda_ok(cudaEventRecord(h->ev[2], stream))) return DMX_ERR_CUDA;
    h->profiled = true;
  }
  return DMX_OK;
}

}  // namespace

extern "C" {

int dmx_step(dmx_handle* h, const void* const* grad_ptrs, const int32_t* batch_sizes, float* params,
             float* momentum, float lr, float beta, float* prev_agg, float* out_state, void* cuda_stream) {
  return step_impl(h, grad_ptrs, batch_sizes, params, momentum, lr, beta, prev_agg, out_state, cuda_stream, nullptr);
}

int dmx_step_adam(dmx_handle* h, const void* const* grad_ptrs, const int32_t* batch_sizes, float* params,
                  float* first_moment, float* second_moment, float lr, float beta1, float beta2, float eps,
                  int64_t t, float* prev_agg, float* out_state, void* cuda_stream) {
  const AdamParams ap = {second_moment, beta2, eps, t};
  return step_impl(h, grad_ptrs, batch_sizes, params, first_moment, lr, beta1, prev_agg, out_state, cuda_stream, &ap);
}

int dmx_partials_len(const dmx_handle* h) {
  if (!live(h)) return DMX_ERR_HANDLE;
  return h->K + 5 + 2 * h->S;
}

int dmx_step_partial(dmx_handle* h, const void* const* grad_ptrs, const int32_t* batch_sizes, float* params,
                     float* momentum, float lr, float beta, float* prev_agg, double* partials, void* cuda_stream) {
  if (!partials) return DMX_ERR_ARG;
  return step_impl(h, grad_ptrs, batch_sizes, params, momentum, lr, beta, prev_agg, nullptr, cuda_stream, nullptr, partials);
}

int dmx_step_adam_partial(dmx_handle* h, const void* const* grad_ptrs, const int32_t* batch_sizes, float* params,
                          float* first_moment, float* second_moment, float lr, float beta1, float beta2, float eps,
                          int64_t t, float* prev_agg, double* partials, void* cuda_stream) {
  if (!partials) return DMX_ERR_ARG;
  const AdamParams ap = {second_moment, beta2, eps, t};
  return step_impl(h, grad_ptrs, batch_sizes, params, first_moment, lr, beta1, prev_agg, nullptr, cuda_stream, &ap, partials);
}

int dmx_finalize_partials(int K, int S, const int32_t* batch_sizes, const double* partials, int adam, int64_t P_total,
                          float* out_state, void* cuda_stream) {
  if (K < 1 || K > DMX_MAX_WORKERS || S < 1 || S > DMX_MAX_SEGMENTS || !batch_sizes || !partials || !out_state ||
      P_total < 1 || P_total >= DMX_MAX_PARAMS)
    return DMX_ERR_ARG;
  if (((uintptr_t)partials & 7) || ((uintptr_t)out_state & 3)) return DMX_ERR_ALIGN;
  dmx::DeriveArgs G;
  std::memset(&G, 0, sizeof(G));
  int64_t B = 0;
  for (int k = 0; k < K; ++k) {
    if (batch_sizes[k] < 1) return DMX_ERR_BATCH;
    G.b[k] = (double)batch_sizes[k];
    B += batch_sizes[k];
  }
  G.K = K; G.S = S; G.adam = adam ? 1 : 0; G.P = (double)P_total; G.B = (double)B;
  G.partials = partials; G.out_state = out_state;
  dmx::derive_kernel<<<1, dmx::kFinalWarps * 32, 0, static_cast<cudaStream_t>(cuda_stream)>>>(G);
  if (!cuda_ok(cudaGetLastError())) return DMX_ERR_CUDA;
  return DMX_OK;
}

int dmx_shard_range(int64_t P, int nshards, int shard, int64_t* lo, int64_t* hi) {
  if (P < 1 || nshards < 1 || shard < 0 || shard >= nshards || !lo || !hi) return DMX_ERR_ARG;
  // boundaries on multiples of 1024 elements: shard pointers keep their 16-byte alignment for either
  // gradient type; a shard may be empty when P is small
  const int64_t align = 1024;
  const int64_t units = (P + align - 1) / align;
  const int64_t a = units * shard / nshards * align, b = units * (shard + 1) / nshards * align;
  *lo = std::min<int64_t>(a, P);
  *hi = shard == nshards - 1 ? P : std::min<int64_t>(b, P);
  return DMX_OK;
}

int dmx_shard_segments(const int64_t* seg_offsets, int S, int64_t lo, int64_t hi, int64_t* shard_offsets) {
  if (!seg_offsets || !shard_offsets || S < 1 || S > DMX_MAX_SEGMENTS || lo < 0 || hi < lo) return DMX_ERR_ARG;
  if (seg_offsets[0] != 0 || hi > seg_offsets[S]) return DMX_ERR_SEGMENTS;
  for (int s = 0; s <= S; ++s) {
    if (s < S && seg_offsets[s] > seg_offsets[s + 1]) return DMX_ERR_SEGMENTS;
    shard_offsets[s] = std::min<int64_t>(std::max<int64_t>(seg_offsets[s], lo), hi) - lo;
  }
  return DMX_OK;
}

int dmx_step_host(dmx_handle* h, const void* const* host_grad_ptrs, void* const* staging_ptrs,
                  const int32_t* batch_sizes, float* params, float* momentum, float lr, float beta,
                  float* prev_agg, float* out_state_dev, float* out_state_host, void* cuda_stream) {
  if (!live(h)) return DMX_ERR_HANDLE;
  if (!host_grad_ptrs || !staging_ptrs || !out_state_host || !out_state_dev) return DMX_ERR_ARG;
  if (const int rcd = dmxh::check_current_device(h->device); rcd != DMX_OK) return rcd;
  const size_t gbytes = (size_t)h->P * (h->dtype == DMX_BF16 ? 2 : 4);
  for (int k = 0; k < h->K; ++k) {
    if (!host_grad_ptrs[k] || !staging_ptrs[k]) return DMX_ERR_ARG;
    if ((uintptr_t)staging_ptrs[k] & 15) return DMX_ERR_ALIGN;
  }
  cudaStream_t stream = static_cast<cudaStream_t>(cuda_stream);
  for (int k = 0; k < h->K; ++k)
    if (!cuda_ok(cudaMemcpyAsync(staging_ptrs[k], host_grad_ptrs[k], gbytes, cudaMemcpyHostToDevice, stream)))
      return DMX_ERR_CUDA;
  const int rc = dmx_step(h, (const void* const*)staging_ptrs, batch_sizes, params, momentum, lr, beta, prev_agg,
                          out_state_dev, cuda_stream);
  if (rc != DMX_OK) return rc;
  const size_t obytes = (size_t)(DMX_ST_HDR + h->K + 2 * h->S) * sizeof(float);
  if (!cuda_ok(cudaMemcpyAsync(out_state_host, out_state_dev, obytes, cudaMemcpyDeviceToHost, stream))) return DMX_ERR_CUDA;
  if (!cuda_ok(cudaStreamSynchronize(stream))) return DMX_ERR_CUDA;
  return DMX_OK;
}

int dmx_set_profiling(dmx_handle* h, int on) {
  if (!live(h)) return DMX_ERR_HANDLE;
  if (on) {
    for (int i = 0; i < 3; ++i)
      if (!h->ev[i] && !cuda_ok(cudaEventCreate(&h->ev[i]))) return DMX_ERR_CUDA;
  }
  h->profiling = on != 0;
  h->profiled = false;
  return DMX_OK;
}

int dmx_get_profile(dmx_handle* h, float* fused_ms, float* finalize_ms) {
  if (!live(h)) return DMX_ERR_HANDLE;
  if (!fused_ms || !finalize_ms || !h->profiling || !h->profiled) return DMX_ERR_ARG;
  if (!cuda_ok(cudaEventSynchronize(h->ev[2]))) return DMX_ERR_CUDA;
  if (!cuda_ok(cudaEventElapsedTime(fused_ms, h->ev[0], h->ev[1]))) return DMX_ERR_CUDA;
  if (!cuda_ok(cudaEventElapsedTime(finalize_ms, h->ev[1], h->ev[2]))) return DMX_ERR_CUDA;
  return DMX_OK;
}

int dmx_plan_chunks(int64_t P, int K, int grad_dtype, int tile_elems, int resident_ctas, int32_t* first_tile,
                    int32_t* num_tiles, int32_t* group_stride, int capacity, int* group_tiles, int* grid) {
  if (P < 1 || P >= DMX_MAX_PARAMS || K < 1 || K > DMX_MAX_WORKERS || tile_elems < 1 || resident_ctas < 1 ||
      (grad_dtype != DMX_F32 && grad_dtype != DMX_BF16) || capacity < 0)
    return DMX_ERR_ARG;
  ChunkPlan cp;
  plan_chunks(P, K, grad_dtype, tile_elems, resident_ctas, env_int("DMX_TILE_GROUP", 0), env_int("DMX_CHUNK_TILES", 0),
              env_int("DMX_MIN_CHUNK_KB", 0), cp);
  if (group_tiles) *group_tiles = cp.R;
  if (grid) *grid = cp.grid;
  const int n = (int)cp.tile0.size();
  if (capacity >= n && first_tile && num_tiles && group_stride) {
    std::copy(cp.tile0.begin(), cp.tile0.end(), first_tile);
    std::copy(cp.ntiles.begin(), cp.ntiles.end(), num_tiles);
    std::copy(cp.stride.begin(), cp.stride.end(), group_stride);
  }
  return n;
}

int dmx_launches_per_step(const dmx_handle* h) {
  if (!live(h)) return DMX_ERR_HANDLE;
  return 2;
}

int dmx_scratch_info(const dmx_handle* h, int* grid, int* nchunks, int* nslots) {
  if (!live(h)) return DMX_ERR_HANDLE;
  if (grid) *grid = h->plan.grid;
  if (nchunks) *nchunks = h->nchunks;
  if (nslots) *nslots = h->nslots;
  return DMX_OK;
}

int dmx_check_guards(dmx_handle* h) {
  if (!live(h)) return DMX_ERR_HANDLE;
  if (const int rc = dmxh::check_current_device(h->device); rc != DMX_OK) return rc;
  uint32_t got[2 * kGuardBytes / 4];
  for (const dmx_handle::Guarded& g : h->guarded) {
    if (!cuda_ok(cudaMemcpy(got, g.raw, kGuardBytes, cudaMemcpyDeviceToHost)) ||
        !cuda_ok(cudaMemcpy(got + kGuardBytes / 4, g.raw + kGuardBytes + g.bytes, kGuardBytes, cudaMemcpyDeviceToHost)))
      return DMX_ERR_CUDA;
    for (uint32_t w : got)
      if (w != kGuardWord) return DMX_ERR_GUARD;
  }
  return DMX_OK;
}

int dmx_selftest_wait(dmx_handle* h, uint32_t polls, int* timed_out, double* waited_ms, void* cuda_stream) {
  if (!live(h)) return DMX_ERR_HANDLE;
  if (!timed_out || !waited_ms || polls < 1 || polls > (1u << 24)) return DMX_ERR_ARG;
  if (const int rc = dmxh::check_current_device(h->device); rc != DMX_OK) return rc;
  unsigned long long* d_out = nullptr;
  if (!cuda_ok(cudaMalloc((void**)&d_out, 4 * sizeof(unsigned long long)))) return DMX_ERR_NOMEM;
  cudaStream_t stream = static_cast<cudaStream_t>(cuda_stream);
  unsigned long long out[4] = {0, 0, 0, 0};
  dmx::wait_selftest_kernel<<<1, 32, 0, stream>>>(h->flags + 1, polls, d_out);
  const bool ok = cuda_ok(cudaGetLastError()) &&
                  cuda_ok(cudaMemcpyAsync(out, d_out, sizeof(out), cudaMemcpyDeviceToHost, stream)) &&
                  cuda_ok(cudaStreamSynchronize(stream));
  cudaFree(d_out);
  if (!ok) return DMX_ERR_CUDA;
  *timed_out = (int)out[0];
  *waited_ms = (double)out[2] * 1e-6;
  return DMX_OK;
}

int dmx_destroy(dmx_handle* h) {
  if (!h) return DMX_OK;
  if (!dmxh::live_remove(h, dmxh::kStepHandle)) return DMX_ERR_HANDLE;
  free_handle(h);
  return DMX_OK;
}

const char* dmx_strerror(int code) {
  switch (code) {
    case DMX_OK: return "ok";
    case DMX_ERR_ARG: return "invalid argument (null pointer, size out of range, or aliasing buffers)";
    case DMX_ERR_SEGMENTS: return "segment table must satisfy o[0]=0 <= o[1] <= ... <= o[S]=P";
    case DMX_ERR_BATCH: return "every batch size must be >= 1";
    case DMX_ERR_ALIGN: return "device pointers must be 16-byte aligned";
    case DMX_ERR_NOMEM: return "out of host or device memory";
    case DMX_ERR_CUDA: return "a CUDA runtime call failed";
    case DMX_ERR_HANDLE: return "invalid or destroyed handle";
    case DMX_ERR_LIMIT: return "problem exceeds the fixed scratch of dmx_step_static (too many segments)";
    case DMX_ERR_GUARD: return "a guard word beside the handle's scratch was overwritten";
    default: return "unknown dmx error code";
  }
}

int dmx_last_cuda_error(void) { return g_last_cuda; }

}  // extern "C"

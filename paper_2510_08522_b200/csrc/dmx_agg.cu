// dmx_agg.cu — window statistics of the state vector over k consecutive steps, on the device.
//
// The controller acts on metrics aggregated over k iterations (Section "System architecture";
// Section "State representation": each state vector is built from metrics collected every k
// iterations, as means and standard deviations). Keeping the running mean and spread of
// out_state on the GPU means the host reads one small vector every k steps instead of k.
// Per entry, Welford's update in fp64: n-th value x: d = x - mean; mean += d/n; M2 += d (x - mean).
#include "dmx.h"

#include <cuda_runtime.h>
#include <new>

#include "dmx_host.h"

namespace {

__global__ void agg_push_kernel(const float* __restrict__ x, double* __restrict__ mean, double* __restrict__ m2,
                                unsigned* __restrict__ flags_or, float* __restrict__ out, int len, int n, int k, int emit) {
  const int i = blockIdx.x * blockDim.x + threadIdx.x;
  if (i >= len) return;
  const double v = (double)x[i];
  double mu = n == 1 ? 0.0 : mean[i];
  double s = n == 1 ? 0.0 : m2[i];
  const double d = v - mu;
  mu += d / (double)n;
  s += d * (v - mu);
  unsigned f = 0u;
  if (i == DMX_ST_FLAGS) {
    f = (n == 1 ? 0u : *flags_or) | (unsigned)(int)x[i];
    *flags_or = f;
  }
  if (emit) {
    if (i == DMX_ST_FLAGS) {       // a bit mask: the window's OR, no spread
      out[i] = (float)f;
      out[len + i] = 0.f;
    } else {
      const double var = s / (double)k;
      out[i] = (float)mu;
      out[len + i] = (float)sqrt(var > 0.0 ? var : 0.0);
    }
  }
  mean[i] = mu;
  m2[i] = s;
}

}  // namespace

struct dmx_agg {
  int len = 0, k = 0, n = 0;       // n: pushes into the current window so far
  double* mean = nullptr;
  double* m2 = nullptr;
  unsigned* flags_or = nullptr;
};

extern "C" {

int dmx_agg_create(int state_len, int k, dmx_agg** out) {
  if (!out) return DMX_ERR_ARG;
  *out = nullptr;
  if (state_len <= DMX_ST_FLAGS || k < 1) return DMX_ERR_ARG;
  dmxh::alloc_begin();
  dmx_agg* a = dmxh::alloc_host_ok() ? new (std::nothrow) dmx_agg : nullptr;
  if (!a) return DMX_ERR_NOMEM;
  a->len = state_len; a->k = k;
  const bool ok = dmxh::dev_alloc((void**)&a->mean, sizeof(double) * state_len) &&
                  dmxh::dev_alloc((void**)&a->m2, sizeof(double) * state_len) &&
                  dmxh::dev_alloc((void**)&a->flags_or, sizeof(unsigned));
  if (!ok) {
    cudaFree(a->mean); cudaFree(a->m2); cudaFree(a->flags_or);
    (void)cudaGetLastError();
    delete a;
    return DMX_ERR_NOMEM;
  }
  dmxh::live_add(a, dmxh::kAggHandle);
  *out = a;
  return DMX_OK;
}

int dmx_agg_push(dmx_agg* a, const float* out_state, float* window_out, int* emitted, void* cuda_stream) {
  if (!dmxh::live_has(a, dmxh::kAggHandle)) return DMX_ERR_HANDLE;
  if (!out_state || !window_out) return DMX_ERR_ARG;
  const int n = a->n + 1;
  const int emit = n == a->k ? 1 : 0;
  const int threads = 128, blocks = (a->len + threads - 1) / threads;
  agg_push_kernel<<<blocks, threads, 0, static_cast<cudaStream_t>(cuda_stream)>>>(out_state, a->mean, a->m2, a->flags_or,
                                                                                window_out, a->len, n, a->k, emit);
  if (!dmxh::cuda_ok(cudaGetLastError())) return DMX_ERR_CUDA;
  a->n = emit ? 0 : n;
  if (emitted) *emitted = emit;
  return DMX_OK;
}

int dmx_agg_destroy(dmx_agg* a) {
  if (!a) return DMX_OK;
  if (!dmxh::live_remove(a, dmxh::kAggHandle)) return DMX_ERR_HANDLE;
  cudaFree(a->mean); cudaFree(a->m2); cudaFree(a->flags_or);
  (void)cudaGetLastError();
  delete a;
  return DMX_OK;
}

}  // extern "C"

// dmx_host.h — host-side pieces shared by the entry points of the library (dmx.cu defines them):
// the CUDA error bookkeeping behind dmx_last_cuda_error, the argument checks every form of the
// step applies before it enqueues anything, and the packing of the workers into kernel arguments.
#pragma once
#include <cuda_runtime.h>
#include <stddef.h>
#include <stdint.h>

#include "dmx_kernels.cuh"

namespace dmxh {

// true on success; otherwise remembers the code for dmx_last_cuda_error and clears the
// runtime's sticky last-error slot
bool cuda_ok(cudaError_t e);

// The buffers of one step. `out` is the state vector (4-byte aligned) or the partial sums
// (8-byte aligned); `second` is Adam's second-moment buffer or null.
struct StepBuffers {
  const void* const* grad_ptrs;
  const int32_t* batch_sizes;
  const float *params, *momentum, *prev_agg, *second;
  const void* out;
  size_t out_bytes;
  unsigned out_align_mask;
};

// Null pointers, batch sizes, alignment and aliasing, in that order (DMX_ERR_ARG, DMX_ERR_BATCH,
// DMX_ERR_ALIGN, DMX_ERR_ARG). On success *B is the total batch and *pivot the worker with the
// largest batch (lowest index on ties).
int check_step_buffers(int K, int64_t P, int grad_dtype, const StepBuffers& sb, int64_t* B, int* pivot);

// Workers in processing order (the pivot first, the others in the caller's order): gradient
// pointers, weights and batch sizes into A; orig[slot] = caller's index, b[slot] = batch size.
// Also sets lr, beta, the total batch and their fp64 forms.
void pack_workers(int K, const void* const* grad_ptrs, const int32_t* batch_sizes, int pivot, int64_t B, float lr,
                  float beta, dmx::StepArgs& A, int* orig, double* b);

// Live handles. A handle is valid while its address is registered under its kind; the entry
// points look it up instead of reading through the pointer, so a call on a destroyed handle
// returns DMX_ERR_HANDLE without touching freed memory. (An address that a later create
// happens to reuse names the new handle: the usual limit of pointer handles.)
enum HandleKind { kStepHandle = 1, kAggHandle = 2 };
void live_add(const void* p, int kind);
bool live_has(const void* p, int kind);
bool live_remove(const void* p, int kind);   // false if it was not registered

// Allocations of the create calls go through these, so that a test can make the n-th one fail
// on the host (environment variable DMX_TEST_FAIL_ALLOC=n, counted from 1 within each create
// call, the handle structure itself being allocation 1): no device is harmed. alloc_begin()
// starts the count; alloc_host_ok() stands for the handle structure's allocation; a refused
// dev_alloc records cudaErrorMemoryAllocation like a real failure.
void alloc_begin();
bool alloc_host_ok();
bool dev_alloc(void** p, size_t bytes);

// DMX_OK if `device` is the calling thread's current CUDA device, else DMX_ERR_HANDLE (a kernel
// launched on another device would be handed pointers it cannot reach).
int check_current_device(int device);

}  // namespace dmxh

// dmx_gen.cu — device-side fill kernels of the synthetic workloads (inputs only).
//
// A counter-based generator, Philox4x32-10 written from its published definition (Salmon,
// Moraes, Dror, Shaw, SC'11): the four normals of elements 4i..4i+3 of stream (tag, c2, c3)
// come from counter (i lo, i hi, c2, c3) under key (seed, tag), through Box-Muller on
// u = (r + 0.5) / 2^32. The Python module workload.py holds the host twin of the integer
// core and the recipes; this file holds none of the gradient step's arithmetic and is a
// separate shared object from the step library.
#include <cuda_bf16.h>
#include <cuda_runtime.h>
#include <stdint.h>

namespace {

struct U4 { uint32_t v[4]; };

__device__ __forceinline__ U4 philox4x32_10(uint32_t c0, uint32_t c1, uint32_t c2, uint32_t c3,
                                            uint32_t k0, uint32_t k1) {
#pragma unroll
  for (int r = 0; r < 10; ++r) {
    const uint32_t hi0 = __umulhi(0xD2511F53u, c0), lo0 = 0xD2511F53u * c0;
    const uint32_t hi1 = __umulhi(0xCD9E8D57u, c2), lo1 = 0xCD9E8D57u * c2;
    const uint32_t n0 = hi1 ^ c1 ^ k0, n2 = hi0 ^ c3 ^ k1;
    c0 = n0; c1 = lo1; c2 = n2; c3 = lo0;
    k0 += 0x9E3779B9u; k1 += 0xBB67AE85u;
  }
  U4 out; out.v[0] = c0; out.v[1] = c1; out.v[2] = c2; out.v[3] = c3;
  return out;
}

__device__ __forceinline__ void normals4(int64_t i, uint32_t c2, uint32_t c3, uint32_t seed,
                                         uint32_t tag, float z[4]) {
  const U4 r = philox4x32_10((uint32_t)(i & 0xffffffff), (uint32_t)(i >> 32), c2, c3, seed, tag);
  const float s = 2.3283064365386963e-10f;  // 2^-32
  const float u0 = ((float)r.v[0] + 0.5f) * s, u1 = ((float)r.v[1] + 0.5f) * s;
  const float u2 = ((float)r.v[2] + 0.5f) * s, u3 = ((float)r.v[3] + 0.5f) * s;
  const float rad0 = sqrtf(-2.0f * logf(u0)), rad1 = sqrtf(-2.0f * logf(u2));
  float sn, cs;
  sincospif(2.0f * u1, &sn, &cs);
  z[0] = rad0 * cs; z[1] = rad0 * sn;
  sincospif(2.0f * u3, &sn, &cs);
  z[2] = rad1 * cs; z[3] = rad1 * sn;
}

// mode 0: dst = base + scale*z (base may be null -> mean)   mode 1: dst += scale*z
template <bool BF16>
__global__ void fill_kernel(void* __restrict__ dst, const float* __restrict__ base, float mean,
                            float scale, int64_t n, uint32_t seed, uint32_t tag, uint32_t c2,
                            uint32_t c3, int accumulate) {
  const int64_t ngroups = (n + 3) / 4;
  for (int64_t i = blockIdx.x * (int64_t)blockDim.x + threadIdx.x; i < ngroups;
       i += (int64_t)gridDim.x * blockDim.x) {
    float z[4];
    normals4(i, c2, c3, seed, tag, z);
    const int64_t j = 4 * i;
    const int m = (n - j) < 4 ? (int)(n - j) : 4;
    float v[4];
#pragma unroll
    for (int e = 0; e < 4; ++e) {
      float b = mean;
      if (e < m) {
        if (accumulate) b = static_cast<const float*>(dst)[j + e];
        else if (base) b = base[j + e];
      }
      v[e] = fmaf(scale, z[e], b);
    }
    if (BF16) {
      __nv_bfloat16* o = static_cast<__nv_bfloat16*>(dst);
      for (int e = 0; e < m; ++e) o[j + e] = __float2bfloat16_rn(v[e]);
    } else {
      float* o = static_cast<float*>(dst);
      if (m == 4) *reinterpret_cast<float4*>(o + j) = make_float4(v[0], v[1], v[2], v[3]);
      else for (int e = 0; e < m; ++e) o[j + e] = v[e];
    }
  }
}

// Number of SMs of the current device (asked once per device).
int sm_count() {
  static int cached[64] = {0};
  int dev = 0;
  if (cudaGetDevice(&dev) != cudaSuccess || dev < 0 || dev >= 64) return 1;
  if (cached[dev] == 0) {
    int n = 0;
    if (cudaDeviceGetAttribute(&n, cudaDevAttrMultiProcessorCount, dev) != cudaSuccess || n < 1) n = 1;
    cached[dev] = n;
  }
  return cached[dev];
}

int launch(void* dst, const float* base, float mean, float scale, int64_t n, int bf16,
           uint32_t seed, uint32_t tag, uint32_t c2, uint32_t c3, int accumulate, void* stream) {
  if (!dst || n < 1) return -1;
  if (accumulate && bf16) return -1;
  if (!bf16 && (reinterpret_cast<uintptr_t>(dst) & 15)) return -4;
  const int threads = 256;
  int64_t blocks = ((n + 3) / 4 + threads - 1) / threads;
  const int64_t cap = (int64_t)sm_count() * 64;
  if (blocks > cap) blocks = cap;
  cudaStream_t st = static_cast<cudaStream_t>(stream);
  if (bf16) fill_kernel<true><<<(unsigned)blocks, threads, 0, st>>>(dst, base, mean, scale, n, seed, tag, c2, c3, accumulate);
  else fill_kernel<false><<<(unsigned)blocks, threads, 0, st>>>(dst, base, mean, scale, n, seed, tag, c2, c3, accumulate);
  return cudaGetLastError() == cudaSuccess ? 0 : -6;
}

// Read-only streaming probe: every thread reads 16-byte pieces of up to 64 buffers with eight
// loads in flight and folds them into a checksum (one word per CTA). It measures what the
// memory system delivers for plain reads of the benchmark's own buffers.
struct ProbeArgs { const uint4* src[64]; int nsrc; long long n16; uint32_t* sink; };

__global__ void __launch_bounds__(256) read_probe_kernel(const __grid_constant__ ProbeArgs A) {
  uint32_t acc = 0;
  const long long stride = (long long)gridDim.x * blockDim.x;
  for (long long i = (long long)blockIdx.x * blockDim.x + threadIdx.x; i < A.n16; i += stride) {
#pragma unroll 8
    for (int k = 0; k < A.nsrc; ++k) {
      uint4 v;
      asm volatile("ld.global.cs.v4.u32 {%0,%1,%2,%3}, [%4];" : "=r"(v.x), "=r"(v.y), "=r"(v.z), "=r"(v.w) : "l"(A.src[k] + i));
      acc ^= v.x + v.y + v.z + v.w;
    }
  }
#pragma unroll
  for (int o = 16; o > 0; o >>= 1) acc ^= __shfl_xor_sync(0xffffffffu, acc, o);
  if ((threadIdx.x & 31) == 0) atomicXor(A.sink + blockIdx.x, acc);
}

}  // namespace

extern "C" {

// Reads `bytes` bytes (a multiple of 16) of each of nsrc DEVICE buffers (16-byte aligned) once;
// sink: DEVICE, at least dmxgen_probe_sink_words() words (8 per SM of the current device), receives
// checksums. Returns 0 or a negative code.
int dmxgen_read_probe(const void* const* src, int nsrc, int64_t bytes, uint32_t* sink, void* stream) {
  if (!src || nsrc < 1 || nsrc > 64 || bytes < 16 || (bytes & 15) || !sink) return -1;
  ProbeArgs A;
  for (int k = 0; k < nsrc; ++k) {
    if (!src[k] || (reinterpret_cast<uintptr_t>(src[k]) & 15)) return -4;
    A.src[k] = static_cast<const uint4*>(src[k]);
  }
  A.nsrc = nsrc; A.n16 = bytes / 16; A.sink = sink;
  read_probe_kernel<<<sm_count() * 8, 256, 0, static_cast<cudaStream_t>(stream)>>>(A);
  return cudaGetLastError() == cudaSuccess ? 0 : -6;
}

int dmxgen_probe_sink_words(void) { return sm_count() * 8; }

// dst[j] = mean + std * z_j                                  (fp32, DEVICE, 16-byte aligned)
int dmxgen_normal_fill(float* dst, int64_t n, uint32_t seed, uint32_t tag, uint32_t c2, uint32_t c3,
                       float mean, float std, void* stream) {
  return launch(dst, nullptr, mean, std, n, 0, seed, tag, c2, c3, 0, stream);
}

// dst[j] += std * z_j                                        (fp32, DEVICE, 16-byte aligned)
int dmxgen_normal_add(float* dst, int64_t n, uint32_t seed, uint32_t tag, uint32_t c2, uint32_t c3,
                      float std, void* stream) {
  return launch(dst, nullptr, 0.f, std, n, 0, seed, tag, c2, c3, 1, stream);
}

// dst[j] = round_dtype(mu[j] + scale * z_j): one worker's gradient (dtype 0 fp32, 1 bf16)
int dmxgen_grad_fill(void* dst, int dtype, const float* mu, int64_t n, uint32_t seed, uint32_t tag,
                     uint32_t k, uint32_t step, float scale, void* stream) {
  if (!mu || (dtype != 0 && dtype != 1)) return -1;
  return launch(dst, mu, 0.f, scale, n, dtype, seed, tag, k, step, 0, stream);
}

}  // extern "C"

// dmx_ctl.cu — the controller's decision at the end of an adjustment cycle, on the device.
//
// Algorithm 1, after the k training iterations of a cycle: every worker's metrics become a state
// vector, the policy maps it to an action a_i from {-100, -25, 0, +25, +100}, the batch size
// becomes max(min(x_i + a_i, x_max), x_min), and the reward
//   r_i = Abar_i + alpha max(0, dA_i) - beta T_iter,i - delta (log2 x_i - 5) - eta (sigma^2_norm + sigma_norm)
// is computed (Sections "Action space and batch size adjustment", "Reward function design"; eta = 0
// is the SGD form). One CTA per worker; all arithmetic in fp64 (a few hundred thousand
// operations per decision: latency, not throughput, is what matters here), results stored as fp32.
// The state layout and the policy network (two tanh hidden layers) are this library's
// definitions: the paper names the metric categories and "a PPO-based agent", nothing more.
#include "dmx.h"

#include <cuda_runtime.h>

namespace {

constexpr int kThreads = 256;
constexpr int kMaxF = DMX_CTL_MAX_AUX + DMX_CTL_LOCAL_EXTRA + DMX_CTL_GLOBAL_FEATURES;
constexpr int kMaxIn = DMX_CTL_MAX_HIDDEN;     // longest input vector of a layer
static_assert(kMaxF <= kMaxIn && kMaxIn % 32 == 0, "a layer's input fits the per-lane weight registers");

struct CtlArgs {
  int K, M, H, state_len;
  const float* window;   // 2 * state_len: means, then deviations
  const float* aux;      // K x M
  const int32_t* batch;  // K
  const float* weights;  // W1 (H x F), c1 (H), W2 (H x H), c2 (H), W3 (5 x H), c3 (5)
  const float* uniforms; // K, or null for the greedy choice
  int col_acc, col_gain, col_titer;
  double alpha, beta_t, delta, eta;
  int b_min, b_max;
  int32_t* next_batch;
  int32_t* action;
  float* reward;
  float* logits;    // K x 5
  float* features;  // K x F, or null
};

// One layer, a warp per group of four output rows (four independent chains of loads in flight:
// the layer is latency-bound): out[r] = sum_j W[r][j] x[j] + c[r] for r < rows, fp64, lanes
// striding through the row (coalesced weight loads), then a shuffle tree in a fixed order. The
// activation is applied afterwards by one thread per row (fp64 tanh is a long dependent chain:
// 32 of them in a row on one lane cost more than the dot products).
__device__ __forceinline__ void layer(const float* __restrict__ W, const float* __restrict__ c, const double* x,
                                      double* out, int rows, int n, int wid, int lane) {
  for (int r0 = wid * 4; r0 < rows; r0 += (kThreads / 32) * 4) {
    double s[4] = {0.0, 0.0, 0.0, 0.0};
    // all of the group's weights are requested before the first one is used (n <= 256: at most
    // eight per lane and row)
    float w[4][kMaxIn / 32];
#pragma unroll
    for (int it = 0; it < kMaxIn / 32; ++it) {
      const int j = lane + 32 * it;
#pragma unroll
      for (int q = 0; q < 4; ++q) w[q][it] = (j < n && r0 + q < rows) ? W[(size_t)(r0 + q) * n + j] : 0.f;
    }
#pragma unroll
    for (int it = 0; it < kMaxIn / 32; ++it) {
      const int j = lane + 32 * it;
      const double xj = j < n ? x[j] : 0.0;
#pragma unroll
      for (int q = 0; q < 4; ++q) s[q] = fma((double)w[q][it], xj, s[q]);
    }
#pragma unroll
    for (int q = 0; q < 4; ++q) {
#pragma unroll
      for (int o = 16; o > 0; o >>= 1) s[q] += __shfl_xor_sync(0xffffffffu, s[q], o);
      if (lane == 0 && r0 + q < rows) {
        out[r0 + q] = s[q] + (double)c[r0 + q];
      }
    }
  }
}

__global__ void __launch_bounds__(kThreads) ctl_kernel(const CtlArgs A) {
  __shared__ double f[kMaxF];
  __shared__ double h1[DMX_CTL_MAX_HIDDEN], h2[DMX_CTL_MAX_HIDDEN];
  __shared__ float z[DMX_CTL_ACTIONS];
  __shared__ double zd[8];
  const int i = blockIdx.x, t = threadIdx.x;
  const int M = A.M, H = A.H, F = M + DMX_CTL_LOCAL_EXTRA + DMX_CTL_GLOBAL_FEATURES;
  const float* mean = A.window;
  const float* dev = A.window + A.state_len;
  const double b = (double)A.batch[i];
  const double Bbar = (double)mean[DMX_ST_B_TOTAL];

  // --- state vector of worker i
  if (t < M) {
    f[t] = (double)A.aux[(size_t)i * M + t];
  } else if (t < F) {
    const double Wq = (double)mean[DMX_ST_WMEAN_SQNORM];
    double v = 0.0;
    switch (t - M) {
      case 0: v = log2(b) - 5.0; break;                                            // the regulariser's argument
      case 1: v = Bbar > 0.0 ? b * (double)A.K / Bbar : 0.0; break;                // share of the global batch
      case 2: v = Wq > 0.0 ? (double)mean[DMX_ST_HDR + i] / Wq : 0.0; break;       // own |x_i|^2 against the weighted mean
      case 3: v = (double)mean[DMX_ST_SIGMA_NORM]; break;
      case 4: v = (double)mean[DMX_ST_SIGMA2_NORM]; break;
      case 5: v = (double)dev[DMX_ST_SIGMA_NORM]; break;
      case 6: v = (double)mean[DMX_ST_COS_PREV]; break;
      case 7: v = (double)dev[DMX_ST_COS_PREV]; break;
      default: {                                                                   // noise scale per unit of global batch
        const double gns = (double)mean[DMX_ST_GNS];
        v = Bbar > 0.0 ? log2(1.0 + (gns > 0.0 ? gns : 0.0) / Bbar) : 0.0;
      }
    }
    f[t] = v;
  }
  __syncthreads();
  if (A.features && t < F) A.features[(size_t)i * F + t] = (float)f[t];

  // --- policy network: tanh(W1 f + c1), tanh(W2 h1 + c2), W3 h2 + c3
  const float* W1 = A.weights;
  const float* c1 = W1 + (size_t)H * F;
  const float* W2 = c1 + H;
  const float* c2 = W2 + (size_t)H * H;
  const float* W3 = c2 + H;
  const float* c3 = W3 + (size_t)DMX_CTL_ACTIONS * H;
  const int wid = t >> 5, lane = t & 31;
  layer(W1, c1, f, h1, H, F, wid, lane);
  __syncthreads();
  if (t < H) h1[t] = tanh(h1[t]);
  __syncthreads();
  layer(W2, c2, h1, h2, H, H, wid, lane);
  __syncthreads();
  if (t < H) h2[t] = tanh(h2[t]);
  __syncthreads();
  layer(W3, c3, h2, zd, DMX_CTL_ACTIONS, H, wid, lane);
  __syncthreads();
  if (t < DMX_CTL_ACTIONS) {
    z[t] = (float)zd[t];
    A.logits[(size_t)i * DMX_CTL_ACTIONS + t] = (float)zd[t];
  }
  __syncthreads();
  if (t != 0) return;

  // --- action: taken on the logits as emitted (fp32), so that the choice can be checked from them
  int a = 0;
  if (!A.uniforms) {
    for (int j = 1; j < DMX_CTL_ACTIONS; ++j)
      if (z[j] > z[a]) a = j;                       // ties keep the lowest index
  } else {
    double zmax = (double)z[0];
    for (int j = 1; j < DMX_CTL_ACTIONS; ++j) zmax = fmax(zmax, (double)z[j]);
    double p[DMX_CTL_ACTIONS], sum = 0.0;
    for (int j = 0; j < DMX_CTL_ACTIONS; ++j) { p[j] = exp((double)z[j] - zmax); sum += p[j]; }
    const double u = (double)A.uniforms[i];
    double c = 0.0;
    a = DMX_CTL_ACTIONS - 1;
    for (int j = 0; j < DMX_CTL_ACTIONS; ++j) {
      c += p[j] / sum;
      if (c > u) { a = j; break; }
    }
  }
  const int step[DMX_CTL_ACTIONS] = {-100, -25, 0, 25, 100};
  int nb = A.batch[i] + step[a];
  nb = nb > A.b_max ? A.b_max : nb;
  nb = nb < A.b_min ? A.b_min : nb;
  A.action[i] = a;
  A.next_batch[i] = nb;

  // --- reward of the cycle that just ended (batch size as used during it)
  const double acc = A.col_acc >= 0 ? f[A.col_acc] : 0.0;
  const double gain = A.col_gain >= 0 ? f[A.col_gain] : 0.0;
  const double titer = A.col_titer >= 0 ? f[A.col_titer] : 0.0;
  const double sig2 = (double)mean[DMX_ST_SIGMA2_NORM], sig = (double)mean[DMX_ST_SIGMA_NORM];
  const double r = acc + A.alpha * (gain > 0.0 ? gain : 0.0) - A.beta_t * titer - A.delta * (log2(b) - 5.0) -
                   A.eta * (sig2 + sig);
  A.reward[i] = (float)r;
}

}  // namespace

extern "C" {

int dmx_ctl_num_features(int M) {
  if (M < 0 || M > DMX_CTL_MAX_AUX) return DMX_ERR_ARG;
  return M + DMX_CTL_LOCAL_EXTRA + DMX_CTL_GLOBAL_FEATURES;
}

int64_t dmx_ctl_num_weights(int M, int H) {
  if (M < 0 || M > DMX_CTL_MAX_AUX || H < 1 || H > DMX_CTL_MAX_HIDDEN) return DMX_ERR_ARG;
  const int64_t F = M + DMX_CTL_LOCAL_EXTRA + DMX_CTL_GLOBAL_FEATURES;
  return (int64_t)H * F + H + (int64_t)H * H + H + (int64_t)DMX_CTL_ACTIONS * H + DMX_CTL_ACTIONS;
}

int dmx_ctl_decide(int K, int M, int H, int state_len, const float* window, const float* aux, const int32_t* batch,
                   const float* weights, int col_acc, int col_gain, int col_titer, float alpha, float beta_t,
                   float delta, float eta, int b_min, int b_max, const float* uniforms, int32_t* next_batch,
                   int32_t* action, float* reward, float* logits, float* features, void* cuda_stream) {
  if (K < 1 || K > DMX_MAX_WORKERS || M < 0 || M > DMX_CTL_MAX_AUX || H < 1 || H > DMX_CTL_MAX_HIDDEN) return DMX_ERR_ARG;
  if (state_len < DMX_ST_HDR + K) return DMX_ERR_ARG;
  if (!window || (M > 0 && !aux) || !batch || !weights || !next_batch || !action || !reward || !logits) return DMX_ERR_ARG;
  if (col_acc < -1 || col_acc >= M || col_gain < -1 || col_gain >= M || col_titer < -1 || col_titer >= M) return DMX_ERR_ARG;
  if (b_min < 1 || b_max < b_min) return DMX_ERR_ARG;
  CtlArgs A;
  A.K = K; A.M = M; A.H = H; A.state_len = state_len;
  A.window = window; A.aux = aux; A.batch = batch; A.weights = weights; A.uniforms = uniforms;
  A.col_acc = col_acc; A.col_gain = col_gain; A.col_titer = col_titer;
  A.alpha = (double)alpha; A.beta_t = (double)beta_t; A.delta = (double)delta; A.eta = (double)eta;
  A.b_min = b_min; A.b_max = b_max;
  A.next_batch = next_batch; A.action = action; A.reward = reward; A.logits = logits; A.features = features;
  ctl_kernel<<<K, kThreads, 0, static_cast<cudaStream_t>(cuda_stream)>>>(A);
  if (cudaGetLastError() != cudaSuccess) return DMX_ERR_CUDA;
  return DMX_OK;
}

}  // extern "C"

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

__global__ void __launch_bounds__(kThreads) ctl_kernel(const CtlArgs A) {
  __shared__ double f[kMaxF];
  __shared__ double h1[DMX_CTL_MAX_HIDDEN], h2[DMX_CTL_MAX_HIDDEN];
  __shared__ float z[DMX_CTL_ACTIONS];
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
  if (t < H) {
    double s = (double)c1[t];
    for (int j = 0; j < F; ++j) s = fma((double)W1[(size_t)t * F + j], f[j], s);
    h1[t] = tanh(s);
  }
  __syncthreads();
  if (t < H) {
    double s = (double)c2[t];
    for (int j = 0; j < H; ++j) s = fma((double)W2[(size_t)t * H + j], h1[j], s);
    h2[t] = tanh(s);
  }
  __syncthreads();
  if (t < DMX_CTL_ACTIONS) {
    double s = (double)c3[t];
    for (int j = 0; j < H; ++j) s = fma((double)W3[(size_t)t * H + j], h2[j], s);
    z[t] = (float)s;
    A.logits[(size_t)i * DMX_CTL_ACTIONS + t] = (float)s;
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

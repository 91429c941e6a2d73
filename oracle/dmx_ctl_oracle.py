"""CPU oracle of the controller's decision at the end of an adjustment cycle.

TEST INFRASTRUCTURE, not product code: only the tests and the smoke check import this file. It
imports nothing from the CUDA package, and the index constants of the window vector are typed
in again here on purpose.

What it computes, in fp64 numpy, in the order of Algorithm 1 (the three loops that follow the
k training iterations of a cycle):
  1. each worker's state vector s_i from the window statistics of the step's state vector
     (Section "State representation": metrics aggregated over k iterations) and the metrics the
     caller collected itself (accuracy, accuracy gain, iteration time, network and system
     figures: the `aux` columns);
  2. the policy a_i = pi_theta(s_i, s_global) over the discrete action space
     {-100, -25, 0, +25, +100} (Section "Action space and batch size adjustment") and the
     batch-size update x_i <- max(min(x_i + a_i, x_max), x_min);
  3. the reward (Section "Reward function design"):
       r_i = Abar_i + alpha max(0, dA_i) - beta T_iter,i - delta (log2 x_i - 5)
             - eta (sigma^2_norm + sigma_norm)            (eta = 0 gives the SGD form)
     with x_i the batch size used during the cycle.

The paper fixes the action set, the clamp and the reward formula; it gives neither the layout
of the state vector nor the policy network. Those are this library's definitions ("parity
unpinned" with respect to the paper): the state layout below, and a two-hidden-layer tanh MLP
whose weights the caller supplies. Pinned by tests/test_ctl.py: hand-computed rewards and
clamps, the action table, the MLP against torch.nn layers in fp64, softmax sampling
frequencies, special cases (zero weights, one-hot features).
"""
from __future__ import annotations

import numpy as np

ACTIONS = np.array([-100, -25, 0, 25, 100], dtype=np.int64)
N_GLOBAL = 6
N_LOCAL_EXTRA = 3

# positions in the step's state vector (header of 16, then per-worker squared norms)
_B, _GNS, _COS, _SIG2, _SIG, _WQ, _HDR = 0, 4, 5, 8, 9, 10, 16


def n_features(M: int) -> int:
    return M + N_LOCAL_EXTRA + N_GLOBAL


def features(window, state_len, aux, batch):
    """K x (M + 9) state vectors.  window: 2*state_len values (means, then deviations)."""
    w = np.asarray(window, dtype=np.float64)
    mean, std = w[:state_len], w[state_len:2 * state_len]
    aux = np.asarray(aux, dtype=np.float64)
    b = np.asarray(batch, dtype=np.float64)
    K, M = aux.shape
    f = np.zeros((K, n_features(M)))
    Bbar, Wq = mean[_B], mean[_WQ]
    for i in range(K):
        f[i, :M] = aux[i]
        f[i, M] = np.log2(b[i]) - 5.0                       # the reward's regulariser argument
        f[i, M + 1] = b[i] * K / Bbar if Bbar > 0 else 0.0  # share of the global batch (1 = average)
        f[i, M + 2] = mean[_HDR + i] / Wq if Wq > 0 else 0.0   # own squared gradient norm / weighted mean
        g = M + N_LOCAL_EXTRA
        f[i, g + 0] = mean[_SIG]
        f[i, g + 1] = mean[_SIG2]
        f[i, g + 2] = std[_SIG]
        f[i, g + 3] = mean[_COS]
        f[i, g + 4] = std[_COS]
        # noise scale in units of the global batch: > 0 means the critical batch exceeds the one in use
        f[i, g + 5] = np.log2(1.0 + max(mean[_GNS], 0.0) / Bbar) if Bbar > 0 else 0.0
    return f


def unpack_weights(weights, F, H):
    """W1 (H x F), c1 (H), W2 (H x H), c2 (H), W3 (5 x H), c3 (5), packed in this order, row-major."""
    w = np.asarray(weights, dtype=np.float64)
    sizes = [H * F, H, H * H, H, 5 * H, 5]
    assert w.size == sum(sizes), (w.size, sum(sizes))
    parts, o = [], 0
    for n in sizes:
        parts.append(w[o:o + n])
        o += n
    return (parts[0].reshape(H, F), parts[1], parts[2].reshape(H, H), parts[3], parts[4].reshape(5, H), parts[5])


def logits(f, weights, H):
    W1, c1, W2, c2, W3, c3 = unpack_weights(weights, f.shape[1], H)
    z = np.zeros((f.shape[0], 5))
    for i in range(f.shape[0]):
        h1 = np.tanh(W1 @ f[i] + c1)
        h2 = np.tanh(W2 @ h1 + c2)
        z[i] = W3 @ h2 + c3
    return z


def choose(z, uniforms=None):
    """Action index per row. Greedy: the largest logit as rounded to fp32, lowest index on ties.
    Sampling: the smallest a whose cumulative softmax probability exceeds u_i."""
    z32 = np.asarray(z, dtype=np.float32).astype(np.float64)
    K = z32.shape[0]
    a = np.zeros(K, dtype=np.int64)
    for i in range(K):
        if uniforms is None:
            a[i] = int(np.argmax(z32[i]))        # numpy returns the first maximum
        else:
            p = np.exp(z32[i] - z32[i].max())
            p /= p.sum()
            c, pick = 0.0, 4
            for j in range(5):
                c += p[j]
                if c > float(uniforms[i]):
                    pick = j
                    break
            a[i] = pick
    return a


def reward(window, state_len, aux, batch, cols, alpha, beta_t, delta, eta):
    """cols = (column of Abar, of dA, of T_iter) in aux; -1 leaves the term out."""
    w = np.asarray(window, dtype=np.float64)
    aux = np.asarray(aux, dtype=np.float64)
    b = np.asarray(batch, dtype=np.float64)
    sig2, sig = w[_SIG2], w[_SIG]
    r = np.zeros(aux.shape[0])
    for i in range(aux.shape[0]):
        acc = aux[i, cols[0]] if cols[0] >= 0 else 0.0
        gain = aux[i, cols[1]] if cols[1] >= 0 else 0.0
        titer = aux[i, cols[2]] if cols[2] >= 0 else 0.0
        r[i] = acc + alpha * max(0.0, gain) - beta_t * titer - delta * (np.log2(b[i]) - 5.0) - eta * (sig2 + sig)
    return r


def decide(window, state_len, aux, batch, weights, H, cols=(0, 1, 2), alpha=1.0, beta_t=0.0, delta=0.0, eta=0.0,
           b_min=32, b_max=1024, uniforms=None):
    """One decision for all K workers. Returns dict(next_batch, action, reward, logits, features)."""
    f = features(window, state_len, aux, batch)
    z = logits(f, weights, H)
    a = choose(z, uniforms)
    b = np.asarray(batch, dtype=np.int64)
    nxt = np.maximum(np.minimum(b + ACTIONS[a], b_max), b_min)
    r = reward(window, state_len, aux, batch, cols, alpha, beta_t, delta, eta)
    return dict(next_batch=nxt, action=a, reward=r, logits=z, features=f)

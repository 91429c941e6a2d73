"""Writes tests/golden/seeded_small_k3.json: inputs and the oracle's outputs for a small problem
whose arithmetic is exact (integer-valued gradients, batch sizes summing to a power of two), so
the stored values do not depend on the platform. Calls only oracle/.

    python tests/golden/make_seeded_golden.py
"""
import json
import os
import sys

import numpy as np

HERE = os.path.dirname(os.path.abspath(__file__))
sys.path.insert(0, os.path.dirname(os.path.dirname(HERE)))
from oracle.dmx_oracle import Oracle  # noqa: E402


def main():
    rng = np.random.default_rng(20251008)
    K, P = 3, 37
    seg = [0, 5, 5, 20, 37]                       # one empty segment
    b = [1, 2, 5]                                 # B = 8: the weighted mean is exact in fp32 and fp64
    grads = [rng.integers(-8, 9, P).astype(np.float32) for _ in range(K)]
    params = (rng.integers(-16, 17, P) / 4.0).astype(np.float32)
    momentum = (rng.integers(-8, 9, P) / 2.0).astype(np.float32)
    prev = rng.integers(-4, 5, P).astype(np.float32)
    lr, beta = 0.25, 0.5
    rec = dict(source="written by tests/golden/make_seeded_golden.py from the CPU oracle (exact arithmetic: integers, B = 8, "
                      "lr and beta powers of two); the paper prints no worked example",
               K=K, P=P, seg_offsets=seg, batch_sizes=b, lr=lr, beta=beta,
               grads=[g.tolist() for g in grads], params=params.tolist(), momentum=momentum.tolist(), prev_agg=prev.tolist())
    st = Oracle(K, P, seg, 0).step(grads, b, params, momentum, lr, beta, prev)
    rec["expect"] = dict(state=[float(v) for v in st], agg=prev.tolist(), momentum=momentum.tolist(), params=params.tolist())
    with open(os.path.join(HERE, "seeded_small_k3.json"), "w") as f:
        json.dump(rec, f, indent=1)
    print("wrote", os.path.join(HERE, "seeded_small_k3.json"))


if __name__ == "__main__":
    main()

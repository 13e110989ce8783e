"""The GPU harness spreads oracle calls over threads; the split must not
change a single bit of what the single-threaded oracle returns."""
import numpy as np

import oracle
import gpu_harness as H


def test_chunked_oracle_step_is_the_oracle_step(monkeypatch):
    monkeypatch.setattr(H, "_STEP_CHUNK", 1 << 12)
    rng = np.random.default_rng(5)
    n = 5 * (1 << 12) + 37
    hp = oracle.HParams(lr=1e-3, beta1=0.9, beta2=0.999, eps=1e-8, weight_decay=0.01,
                        max_grad_norm=1.0)
    p = rng.standard_normal(n).astype(np.float32)
    m = (rng.standard_normal(n) * 1e-2).astype(np.float32)
    v = (rng.random(n) * 1e-4).astype(np.float32)
    g = rng.standard_normal(n).astype(np.float32)
    a = [p.copy(), m.copy(), v.copy()]
    b = [p.copy(), m.copy(), v.copy()]
    oracle.adamw_step_range(*a, g, 0, n, 0.37, 3, hp)
    H._oracle_step_chunked(*b, g, 0.37, 3, hp)
    for x, y in zip(a, b):
        assert x.tobytes() == y.tobytes()

"""The five workload configurations (zero-based C0..C4) and scaled-down variants.

Notation follows the paper: W is J x D; P simulated workers each contribute B
sufficient-factor pairs per step, K = P*B.
"""
from __future__ import annotations

import copy
import math

# `path`: arithmetic path the workload is quoted on ("f32" CUDA-core, "tf32" or "bf16" tensor-core).
# `pool`: number of resident minibatches; step t uses minibatch t mod pool.
CONFIGS = {
    # MLR tiny: one SF compute + apply step.
    "C0": dict(index=0, model="mlr", J=10, D=64, P=4, B=8, eta=0.1, steps=1, pool=1,
               path="f32", w_std=0.01, labels="uniform", normalise=False),
    # MLR large: dense L2-normalised features, uniform labels, 100 steps.
    "C1": dict(index=1, model="mlr", J=1000, D=20000, P=8, B=128, eta=1e-2, steps=100, pool=8,
               path="f32", w_std=0.01, labels="uniform", normalise=True),
    # DML: L is 600 x 10000; pairs ~N(0,1); even pairs similar, odd pairs dissimilar; margin 1.
    # w_std = 1/sqrt(2*J*D) puts E||L d||^2 at the margin so about half the dissimilar pairs are active.
    "C2": dict(index=2, model="dml", J=600, D=10000, P=8, B=256, eta=1e-5, steps=20, pool=1,
               path="f32", w_std=1.0 / math.sqrt(2.0 * 600 * 10000), margin=1.0),
    # Sparse-coding dictionary update: W is (feature dim 4096) x (10000 atoms), codes 5% dense.
    "C3": dict(index=3, model="sc", J=4096, D=10000, P=16, B=64, eta=1e-4, steps=20, pool=1,
               path="f32", density=0.05, noise_std=0.01, init_mix=0.5),
    # MLR at scale, bf16 in / fp32 accumulate, Zipf(1.1) labels, 50 steps.
    "C4": dict(index=4, model="mlr", J=32768, D=8192, P=16, B=256, eta=1e-5, steps=50, pool=4,
               path="bf16", w_std=0.01, labels="zipf", zipf_s=1.1, normalise=False),
}


def get_config(name: str) -> dict:
    cfg = copy.deepcopy(CONFIGS[name])
    cfg["name"] = name
    cfg["K"] = cfg["P"] * cfg["B"]
    return cfg


def scaled(name: str, **overrides) -> dict:
    """A copy of config `name` with some sizes replaced (parity tests at oracle-friendly sizes)."""
    cfg = get_config(name)
    cfg.update(overrides)
    cfg["K"] = cfg["P"] * cfg["B"]
    if cfg["model"] == "dml" and "w_std" not in overrides:
        cfg["w_std"] = 1.0 / math.sqrt(2.0 * cfg["J"] * cfg["D"])
    cfg["name"] = name + "'" if overrides else name
    return cfg

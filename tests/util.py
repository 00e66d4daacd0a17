"""Shared helpers of the GPU parity tests: run the oracle on a batch, fetch device results."""
from __future__ import annotations

import numpy as np

from oracle import sfb_oracle as orc

MODEL_ID = {"mlr": orc.MODEL_MLR, "dml": orc.MODEL_DML, "sc": orc.MODEL_SC}

# Tolerances on the relative Frobenius error against the fp64 oracle, per arithmetic path.
TOL = {"f32": 1e-5, "tf32": 2e-3, "bf16": 1e-2}
# DML pairs whose oracle slack | |z|^2 - margin | is within this band may take either gate value.
GATE_BAND = {"f32": 1e-5, "tf32": 5e-3, "bf16": 1e-2}


def batch_of(inputs: dict, cfg: dict, b: int = 0) -> dict:
    m = cfg["model"]
    if m == "mlr":
        return dict(X=inputs["X"][b], labels=inputs["labels"][b])
    if m == "dml":
        return dict(Xa=inputs["Xa"][b], Xb=inputs["Xb"][b], similar=inputs["similar"])
    return dict(rowptr=inputs["rowptr"][b], idx=inputs["idx"][b], val=inputs["val"][b], Xdata=inputs["Xdata"][b])


def oracle_factors(cfg: dict, W, batch: dict):
    """Returns (U, V or None, extra) from the oracle for one minibatch."""
    m = cfg["model"]
    if m == "mlr":
        U, V = orc.mlr_factors(W, batch["X"], batch["labels"])
        return U, V, {}
    if m == "dml":
        U, V, n, active = orc.dml_factors(W, batch["Xa"], batch["Xb"], batch["similar"], cfg.get("margin", 1.0))
        return U, V, dict(n=n, active=active, Z=V @ np.asarray(W, dtype=np.float64).T)
    U = orc.sc_factors(W, batch["rowptr"], batch["idx"], batch["val"], batch["Xdata"])
    return U, None, {}


def oracle_apply(cfg: dict, W, U, V, batch: dict, eta: float):
    if cfg["model"] == "sc":
        return orc.apply_sparse(W, U, batch["rowptr"], batch["idx"], batch["val"], eta)
    return orc.apply_dense(W, U, V, eta)


def to_f64(t) -> np.ndarray:
    """torch tensor (fp32 or bf16) -> numpy fp64."""
    import torch
    return t.detach().to(torch.float32).cpu().numpy().astype(np.float64)


def dml_accept_gate(cfg: dict, U_gpu: np.ndarray, U_or: np.ndarray, extra: dict, path: str) -> np.ndarray:
    """DML: the gate of a pair must match the oracle's unless the pair sits inside the tie band.

    Returns the oracle U with the GPU's gate substituted on the in-band pairs (so a legitimate
    flip of a near-tie does not count as an error).
    """
    n, active = extra["n"], extra["active"]
    gpu_active = np.abs(U_gpu).sum(axis=1) > 0
    band = np.abs(n - cfg.get("margin", 1.0)) <= GATE_BAND[path]
    mism = gpu_active != active
    # an all-zero z (L d = 0) is "active" with u = 0; do not count that as a mismatch
    mism &= ~((np.abs(U_or).sum(axis=1) == 0) & ~gpu_active)
    assert not (mism & ~band).any(), f"gate mismatch outside the tie band on pairs {np.nonzero(mism & ~band)[0][:8]}"
    U_fix = U_or.copy()
    for i in np.nonzero(mism & band)[0]:
        # near-tie: take the oracle's u under the GPU's gate decision (-z if active, 0 if not)
        U_fix[i] = -extra["Z"][i] if gpu_active[i] else 0.0
    return U_fix

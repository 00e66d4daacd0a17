"""Shared helpers of the GPU parity tests: run the oracle on a batch, fetch device results."""
from __future__ import annotations

import numpy as np

from oracle import sfb_oracle as orc
from sfbgen import batch_of  # noqa: F401  (re-exported: the tests take it from here)

MODEL_ID = {"mlr": orc.MODEL_MLR, "dml": orc.MODEL_DML, "sc": orc.MODEL_SC}

# Tolerances on the relative Frobenius error against the fp64 oracle, per arithmetic path.
TOL = {"f32": 1e-5, "tf32": 2e-3, "bf16": 1e-2, "tf32x3": 1e-5}   # tf32x3: error-compensated tf32, fp32-grade
# Localised faults (one wrong row of the update, a mis-addressed strip of a tile, a dropped reduction block of
# one tile) barely move a Frobenius norm taken over a large matrix: at J = 32768 a completely wrong row costs
# sqrt(1/J) = 5.5e-3.  So every matrix comparison also bounds each row and each column on its own:
#     || got[r] - ref[r] || / max(|| ref[r] ||, || ref ||_F / sqrt(#rows))  <=  C_ROW * tol.
# The floor (the root-mean-square row norm) keeps rows that are legitimately almost zero from dividing by
# nothing.  C_ROW = 4: the worst row may be four times worse than the tolerance stated for the whole matrix
# (the largest measured ratio of worst row to whole matrix is about 2.5); a wrong row or strip scores about 1.
C_ROW = 4.0
# The fp32 storage rounding of W that is added to a multi-step tolerance may not exceed this multiple of the
# tolerance itself, or the check would say nothing about the kernels.
MAX_STORAGE_OVER_TOL = 1.0
# DML pairs whose oracle slack | |z|^2 - margin | is within this band may take either gate value.
GATE_BAND = {"f32": 1e-5, "tf32": 5e-3, "bf16": 1e-2, "tf32x3": 3e-5}


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
        if int(batch["rowptr"][-1]) < 100000:
            return orc.apply_sparse(W, U, batch["rowptr"], batch["idx"], batch["val"], eta)
        # full-size workloads: the K outer products of the sparse definition take its Python loop minutes; the dense
        # product of the same codes is the same sum (the two routes are pinned equal on the CPU)
        A = orc.csr_to_dense(batch["rowptr"], batch["idx"], batch["val"], cfg["D"])
        return orc.apply_dense(W, U, A, eta)
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


def worst_line(got: np.ndarray, ref: np.ndarray, axis: int = 1, extra: np.ndarray | None = None):
    """Largest per-row (axis=1) or per-column (axis=0) relative error and where it is.

    The error of line r is || got[r] - ref[r] || / max(|| ref[r] ||, rms line norm of ref); `extra` (one value
    per line, already in absolute terms) is subtracted from the numerator first: an allowance that is not the
    kernel's error, e.g. the fp32 storage rounding of that line of W.
    """
    got, ref = np.asarray(got, dtype=np.float64), np.asarray(ref, dtype=np.float64)
    diff = np.sqrt(((got - ref) ** 2).sum(axis=axis))
    if extra is not None:
        diff = np.maximum(diff - extra, 0.0)
    norms = np.sqrt((ref ** 2).sum(axis=axis))
    floor = np.linalg.norm(ref) / np.sqrt(max(norms.size, 1))
    den = np.maximum(norms, floor)
    den[den == 0.0] = 1.0
    e = diff / den
    r = int(np.argmax(e)) if e.size else 0
    return (float(e[r]) if e.size else 0.0), r


def assert_lines(got, ref, tol: float, what: str, extra_rows=None, extra_cols=None):
    """Every row and every column of `got` within C_ROW * tol of `ref` (see C_ROW)."""
    e, r = worst_line(got, ref, 1, extra_rows)
    assert e <= C_ROW * tol, f"{what}: row {r} is off by {e:.3e} > {C_ROW} x {tol}"
    e, c = worst_line(got, ref, 0, extra_cols)
    assert e <= C_ROW * tol, f"{what}: column {c} is off by {e:.3e} > {C_ROW} x {tol}"

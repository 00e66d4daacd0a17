"""Draws the synthetic tensors of one workload configuration.

Distributions and structure (stand-ins for the paper's ImageNet-LLC and
Wikipedia-LSHTC workloads, which are not available offline):

* MLR: W ~ N(0, std w_std); features ~ N(0,1), optionally L2-normalised per
  sample (in fp64, before the single rounding to the storage type); labels
  uniform or Zipf(s) over class ranks (inverse CDF in fp64).
* DML: L ~ N(0, std w_std); pairs x_a, x_b ~ N(0,1); pair i is "similar" iff i
  is even, so every worker holds both kinds.
* SC: W_true has N(0,1) columns normalised to unit L2 norm; the starting
  dictionary is unitcols(W_true + init_mix * unitcols(G)), G ~ N(0,1); every
  code entry is nonzero with probability `density`, values Laplace(0,1); data
  x = W_true a + N(0, std noise_std).  Codes are stored CSR with strictly
  ascending column indices per row.

"N(0, 0.01)" in the workload descriptions is read as standard deviation 0.01.
"""
from __future__ import annotations

import numpy as np

_MASTER_SEED = 0x5FB00000

# tensor ids (one Philox stream each)
_T_W, _T_X, _T_LABEL, _T_CODE_MASK, _T_CODE_VAL, _T_NOISE, _T_XB, _T_G = range(1, 9)


def philox(config_index: int, tensor_id: int, batch: int = 0) -> np.random.Generator:
    """Counter-based generator for (config, tensor, minibatch)."""
    key = (_MASTER_SEED + int(config_index)) & 0xFFFFFFFFFFFFFFFF
    counter = [int(batch), int(tensor_id), 0, 0]
    return np.random.Generator(np.random.Philox(key=key, counter=counter))


def bf16_round_bits(x: np.ndarray) -> np.ndarray:
    """fp32 -> bf16 bit pattern (uint16), round to nearest even.  Pure format conversion."""
    u = np.ascontiguousarray(x, dtype=np.float32).view(np.uint32)
    lsb = (u >> np.uint32(16)) & np.uint32(1)
    r = u + np.uint32(0x7FFF) + lsb
    return (r >> np.uint32(16)).astype(np.uint16)


def bf16_bits_to_f32(b: np.ndarray) -> np.ndarray:
    """bf16 bit pattern (uint16) -> the fp32 value it denotes (exact)."""
    return (b.astype(np.uint32) << np.uint32(16)).view(np.float32)


def _normal_f64(rng: np.random.Generator, shape) -> np.ndarray:
    return rng.standard_normal(shape, dtype=np.float64)


def _normal_f32_big(rng: np.random.Generator, rows: int, cols: int, std: float) -> np.ndarray:
    """Row-chunked N(0, std) fp32 matrix (drawn in fp64, rounded once) without a full fp64 copy."""
    out = np.empty((rows, cols), dtype=np.float32)
    step = max(1, (1 << 24) // max(cols, 1))
    for r0 in range(0, rows, step):
        r1 = min(rows, r0 + step)
        out[r0:r1] = (_normal_f64(rng, (r1 - r0, cols)) * std).astype(np.float32)
    return out


def _unitcols(m: np.ndarray) -> np.ndarray:
    return m / np.sqrt((m * m).sum(axis=0, keepdims=True))


def _zipf_labels(rng: np.random.Generator, n: int, classes: int, s: float) -> np.ndarray:
    ranks = np.arange(1, classes + 1, dtype=np.float64)
    cdf = np.cumsum(ranks ** (-s))
    cdf /= cdf[-1]
    u = rng.random(n)
    return np.minimum(np.searchsorted(cdf, u, side="left"), classes - 1).astype(np.int32)


def _make_mlr(cfg: dict) -> dict:
    ci, J, D, K, pool = cfg["index"], cfg["J"], cfg["D"], cfg["K"], cfg["pool"]
    bf16 = cfg["path"] == "bf16"
    out = {"W": _normal_f32_big(philox(ci, _T_W), J, D, cfg["w_std"])}
    X = np.empty((pool, K, D), dtype=np.float32)
    labels = np.empty((pool, K), dtype=np.int32)
    for b in range(pool):
        x = _normal_f64(philox(ci, _T_X, b), (K, D))
        if cfg.get("normalise"):
            x /= np.sqrt((x * x).sum(axis=1, keepdims=True))
        X[b] = x.astype(np.float32)
        rng = philox(ci, _T_LABEL, b)
        if cfg.get("labels") == "zipf":
            labels[b] = _zipf_labels(rng, K, J, cfg["zipf_s"])
        else:
            labels[b] = np.minimum((rng.random(K) * J).astype(np.int64), J - 1).astype(np.int32)
    if bf16:
        bits = bf16_round_bits(X)
        out["X_bits"] = bits                      # what the GPU receives (bf16 storage)
        X = bf16_bits_to_f32(bits)                # the same values, exactly, as fp32
    out["X"] = X
    out["labels"] = labels
    return out


def _make_dml(cfg: dict) -> dict:
    ci, J, D, K, pool = cfg["index"], cfg["J"], cfg["D"], cfg["K"], cfg["pool"]
    out = {"W": _normal_f32_big(philox(ci, _T_W), J, D, cfg["w_std"])}
    Xa = np.empty((pool, K, D), dtype=np.float32)
    Xb = np.empty((pool, K, D), dtype=np.float32)
    for b in range(pool):
        Xa[b] = _normal_f64(philox(ci, _T_X, b), (K, D)).astype(np.float32)
        Xb[b] = _normal_f64(philox(ci, _T_XB, b), (K, D)).astype(np.float32)
    out["Xa"], out["Xb"] = Xa, Xb
    out["similar"] = (np.arange(K) % 2 == 0).astype(np.uint8)
    return out


def _make_sc(cfg: dict) -> dict:
    ci, J, D, K, pool, P, B = (cfg[k] for k in ("index", "J", "D", "K", "pool", "P", "B"))
    w_true = _unitcols(_normal_f64(philox(ci, _T_W), (J, D)))
    g = _unitcols(_normal_f64(philox(ci, _T_G), (J, D)))
    w0 = _unitcols(w_true + cfg["init_mix"] * g)
    out = {"W": w0.astype(np.float32)}
    rowptrs, idxs, vals, xs = [], [], [], []
    cap = 0
    for b in range(pool):
        mask = philox(ci, _T_CODE_MASK, b).random((K, D)) < cfg["density"]
        u = philox(ci, _T_CODE_VAL, b).random((K, D))
        lap = -np.sign(u - 0.5) * np.log1p(-2.0 * np.abs(u - 0.5))     # Laplace(0,1) by inverse CDF
        a = np.where(mask, lap, 0.0).astype(np.float32)                 # stored fp32 codes
        a64 = a.astype(np.float64)
        x = a64 @ w_true.T + cfg["noise_std"] * _normal_f64(philox(ci, _T_NOISE, b), (K, J))
        rows, cols = np.nonzero(a)                                      # row-major => ascending cols per row
        rowptr = np.zeros(K + 1, dtype=np.uint32)
        np.cumsum(np.bincount(rows, minlength=K), out=rowptr[1:], dtype=np.uint32)
        rowptrs.append(rowptr)
        idxs.append(cols.astype(np.uint32))
        vals.append(a[rows, cols].astype(np.float32))
        xs.append(x.astype(np.float32))
        per_worker = rowptr[B::B].astype(np.int64) - rowptr[0:K:B].astype(np.int64)
        cap = max(cap, int(per_worker.max()))
    cap_p = max(32, -(-cap // 32) * 32)            # uniform per-worker CSR capacity, multiple of 32 entries
    out.update(rowptr=rowptrs, idx=idxs, val=vals, Xdata=np.stack(xs), nnz_capacity=cap_p * P)
    return out


def make_inputs(cfg: dict) -> dict:
    """All tensors of configuration `cfg` (see `configs.get_config` / `configs.scaled`)."""
    model = cfg["model"]
    if model == "mlr":
        return _make_mlr(cfg)
    if model == "dml":
        return _make_dml(cfg)
    if model == "sc":
        return _make_sc(cfg)
    raise ValueError(f"unknown model {model!r}")


def batch_of(inputs: dict, cfg: dict, b: int = 0) -> dict:
    """Minibatch b of `inputs` as the keyword arrays one step consumes (views of the generated tensors, no arithmetic)."""
    m = cfg["model"]
    if m == "mlr":
        return dict(X=inputs["X"][b], labels=inputs["labels"][b])
    if m == "dml":
        return dict(Xa=inputs["Xa"][b], Xb=inputs["Xb"][b], similar=inputs["similar"])
    return dict(rowptr=inputs["rowptr"][b], idx=inputs["idx"][b], val=inputs["val"][b], Xdata=inputs["Xdata"][b])

"""fp64 CPU oracle for the sufficient-factor (SF) hot path.  TEST INFRASTRUCTURE ONLY.

This file is the slow, plain statement of what the path computes, written from
the paper's definitions.  Only the tests, the smoke check and the benchmark's
CPU-baseline leg may import it; the product (the CUDA library and its Python
binding) never does, and shares no code with it.

What each function follows:

* Problem (P), Section 2: min_W (1/N) sum_i f_i(W a_i) + h(W), W in R^{J x D}.
* SF property, Section 2.1 ("Proximal SGD"): the stochastic gradient of one
  sample is the outer product u v^T with u = d f_i / d (W a_i) and v = a_i.
* Mini-batch, Section 3: K pairs give an update of rank <= K; all pairs of all
  P workers are applied, W <- W - sum_q u_q v_q^T, here with the learning rate
  of proximal SGD: W <- W - eta * sum_i u_i v_i^T (no 1/K inside; the caller
  folds it into eta).
* MLR (Section 1, Figure 2): f_i = logsumexp(W x_i) - (W x_i)[y_i]; the chain
  rule gives u_i = softmax(W x_i) - onehot(y_i), v_i = x_i.
* DML (Section 2): a_i = x_a - x_b; similar pair f = 1/2 ||L a||^2 (u = +L a),
  dissimilar pair f = 1/2 max(0, m - ||L a||^2) (u = -L a while ||L a||^2 < m,
  else 0); v_i = a_i.
* SC (Section 2, Figure 3): f_i = 1/2 ||W a_i - x_i||^2, u_i = W a_i - x_i,
  v_i = a_i (sparse code, an input here).
* SDCA for L2-regularised MLR (Section 2.1): the update of the auxiliary matrix is
  also rank one, (du_i, a_i); the paper gives no closed form for du_i, so
  sdca_mlr_factors follows a stated reading: PARITY UNPINNED by the paper, pinned
  by the fixed point, the primal-dual link and convergence to the primal optimum.

All arithmetic is fp64 on inputs promoted exactly from their stored fp32 (or
bf16-valued fp32) bytes.  One exception fixed by the wire format: the DML pair
difference is formed with one IEEE fp32 subtraction per element, because that
rounded d is the factor v that would be broadcast; it is then promoted to fp64.

Parity pins (tests/test_oracle_pins.py): brute-force full-matrix gradients by a
route that never forms u, central finite differences of the losses, sum_j u_ij
= 0 for MLR, rank(Delta W) <= K by SVD, closed forms (W = 0, J = 2 logistic
regression, one-hot codes, fixed points), additivity / eta-linearity /
worker-split invariance of the apply, byte-level checks of the packer (plain and
compacted), and hand values for the parity metric rel_fro and for wire_bytes.
Multi-step trajectories have no closed form: parity unpinned beyond "the step is
the composition of the pinned pieces" (guarded by loss decrease).
"""
from __future__ import annotations

import struct

import numpy as np

MODEL_MLR, MODEL_DML, MODEL_SC = 0, 1, 2
DTYPE_F32, DTYPE_BF16 = 0, 1
MAGIC = 0x31424653          # "SFB1" little-endian
VERSION = 1
HEADER_BYTES = 128
DIR_ENTRY_BYTES = 32


def _f64(a):
    return np.asarray(a, dtype=np.float64)


# --------------------------------------------------------------------------------------
# Sufficient factors
# --------------------------------------------------------------------------------------
def mlr_logits(W, X):
    """z_i = W x_i for every sample (rows of the result)."""
    return _f64(X) @ _f64(W).T


def mlr_factors(W, X, labels):
    """u_i = softmax(W x_i) - onehot(y_i), v_i = x_i.  Returns U [K][J], V [K][D]."""
    Z = mlr_logits(W, X)
    m = Z.max(axis=1, keepdims=True)
    E = np.exp(Z - m)
    U = E / E.sum(axis=1, keepdims=True)
    U[np.arange(U.shape[0]), np.asarray(labels, dtype=np.int64)] -= 1.0
    return U, _f64(X).copy()


def mlr_loss(W, X, labels):
    """sum_i logsumexp(z_i) - z_i[y_i]."""
    Z = mlr_logits(W, X)
    m = Z.max(axis=1)
    lse = m + np.log(np.exp(Z - m[:, None]).sum(axis=1))
    return float((lse - Z[np.arange(Z.shape[0]), np.asarray(labels, dtype=np.int64)]).sum())


def sdca_mlr_factors(W, X, labels, dual, step):
    """Mini-batch SDCA step for L2-regularised MLR (Section 2.1, "Stochastic DCA"; the L2-MLR workload of Section 6).

    Primal: min_W (1/N) sum_i f_i(W x_i) + (lam/2) ||W||^2, f_i the multiclass logistic loss; dual variables u_i in
    R^J, auxiliary matrix Z = (1/N) sum_i u_i x_i^T, W = grad h*(Z) = Z / lam.  At the optimum u_i = -grad f_i(W x_i).
    The paper updates u_i <- u_i - du_i, Z <- Z - du_i x_i^T (with the 1/N of Z's definition) and leaves du_i to
    "minimising (D) over u_i", which has no closed form for this loss.  READING (parity unpinned by the paper): the
    damped step toward the coordinate's optimality condition,
        du_i = step * (u_i + g_i),   g_i = softmax(W x_i) - onehot(y_i)   (the SGD factor of the same sample),
    0 < step <= 1, all K samples of the mini-batch from the same W.  The update of W is then the same rank-K apply as
    for SGD, W <- W - eta * sum_i du_i x_i^T with eta = 1 / (lam * N): the sufficient factors are (du_i, x_i).

    dual: [K][J] current dual variables of the mini-batch's samples.  Returns (dU [K][J], V [K][D], new dual [K][J]).
    """
    G, V = mlr_factors(W, X, labels)
    dU = float(step) * (_f64(dual) + G)
    return dU, V, _f64(dual) - dU


def dml_difference(Xa, Xb):
    """d = x_a - x_b: one correctly rounded fp32 subtraction per element, promoted to fp64."""
    d32 = np.asarray(Xa, dtype=np.float32) - np.asarray(Xb, dtype=np.float32)
    return d32.astype(np.float64)


def dml_factors(L, Xa, Xb, similar, margin=1.0):
    """u_i = +L d_i (similar) or -L d_i * [||L d_i||^2 < margin] (dissimilar); v_i = d_i.

    Returns U [K][J], V [K][D], n (squared distances ||L d_i||^2), active (bool gate per pair).
    The hinge is strict: at ||L d||^2 == margin the pair is inactive (subgradient 0).
    """
    Dm = dml_difference(Xa, Xb)
    Z = Dm @ _f64(L).T
    n = (Z * Z).sum(axis=1)
    sim = np.asarray(similar).astype(bool)
    active = sim | (n < margin)
    sign = np.where(sim, 1.0, -1.0)
    U = Z * (sign * active)[:, None]
    return U, Dm, n, active


def dml_loss(L, Xa, Xb, similar, margin=1.0):
    Dm = dml_difference(Xa, Xb)
    Z = Dm @ _f64(L).T
    n = (Z * Z).sum(axis=1)
    sim = np.asarray(similar).astype(bool)
    return float(np.where(sim, 0.5 * n, 0.5 * np.maximum(0.0, margin - n)).sum())


def sc_factors(W, rowptr, idx, val, Xdata):
    """u_i = W a_i - x_i with a_i given as CSR row i; v_i = a_i unchanged.  Returns U [K][J]."""
    W64 = _f64(W)
    X64 = _f64(Xdata)
    K = len(rowptr) - 1
    U = np.empty((K, W64.shape[0]), dtype=np.float64)
    for i in range(K):
        s, e = int(rowptr[i]), int(rowptr[i + 1])
        cols = np.asarray(idx[s:e], dtype=np.int64)
        U[i] = W64[:, cols] @ _f64(val[s:e]) - X64[i]
    return U


def sc_loss(W, rowptr, idx, val, Xdata):
    U = sc_factors(W, rowptr, idx, val, Xdata)
    return float(0.5 * (U * U).sum())


def csr_to_dense(rowptr, idx, val, D):
    K = len(rowptr) - 1
    A = np.zeros((K, D), dtype=np.float64)
    for i in range(K):
        s, e = int(rowptr[i]), int(rowptr[i + 1])
        A[i, np.asarray(idx[s:e], dtype=np.int64)] = _f64(val[s:e])
    return A


# --------------------------------------------------------------------------------------
# Rank-K apply
# --------------------------------------------------------------------------------------
def delta_w(U, V):
    """sum_i u_i v_i^T = U^T V  (U [K][J], V [K][D])."""
    return _f64(U).T @ _f64(V)


def apply_dense(W, U, V, eta):
    """W - eta * sum_i u_i v_i^T."""
    return _f64(W) - float(eta) * delta_w(U, V)


def apply_sparse(W, U, rowptr, idx, val, eta):
    """Same update with v_i given as CSR rows: only the columns a code touches change."""
    Wn = _f64(W).copy()
    U64 = _f64(U)
    for i in range(len(rowptr) - 1):
        s, e = int(rowptr[i]), int(rowptr[i + 1])
        cols = np.asarray(idx[s:e], dtype=np.int64)
        Wn[:, cols] -= float(eta) * np.outer(U64[i], _f64(val[s:e]))
    return Wn


def prox_unit_columns(W):
    """Proximal operator of the sparse-coding constraint ||W_k||_2 <= 1 (Section 2, SC; Figure 3 `prox`):
    every column whose norm exceeds 1 is divided by its norm, the others are left alone."""
    Wn = _f64(W).copy()
    n = np.sqrt((Wn * Wn).sum(axis=0))
    big = n > 1.0
    Wn[:, big] /= n[big]
    return Wn


# --------------------------------------------------------------------------------------
# One step = factors from W_t and minibatch t, then apply (BSP: one W serves all workers)
# --------------------------------------------------------------------------------------
def step(model, W, batch, eta, margin=1.0):
    if model == MODEL_MLR:
        U, V = mlr_factors(W, batch["X"], batch["labels"])
        return apply_dense(W, U, V, eta), U, V
    if model == MODEL_DML:
        U, V, _, _ = dml_factors(W, batch["Xa"], batch["Xb"], batch["similar"], margin)
        return apply_dense(W, U, V, eta), U, V
    if model == MODEL_SC:
        U = sc_factors(W, batch["rowptr"], batch["idx"], batch["val"], batch["Xdata"])
        return apply_sparse(W, U, batch["rowptr"], batch["idx"], batch["val"], eta), U, None
    raise ValueError(model)


# --------------------------------------------------------------------------------------
# SF buffer (the message a worker would broadcast): byte-exact CPU packer
# --------------------------------------------------------------------------------------
def _pad(n, a=128):
    return -(-n // a) * a


def _bf16_bits(x32):
    u = np.ascontiguousarray(x32, dtype=np.float32).view(np.uint32)
    r = u + np.uint32(0x7FFF) + ((u >> np.uint32(16)) & np.uint32(1))
    return (r >> np.uint32(16)).astype(np.uint16)


def sf_layout(model, dtype, J, D, P, B, v_sparse=False, nnz_capacity=0):
    """Offsets of every field of the SF buffer.  All offsets are multiples of 128 bytes.

    header (128 B) | directory (P x 32 B, padded) | P worker streams at a uniform stride.
    Worker stream: U block (B rows x ldu elements), then V block: dense B rows x ldv
    elements, or CSR: rowptr u32[B+1] | idx u32[cap_p] | val[cap_p], each padded to 128 B.
    ldu / ldv round J / D up so that a row is a whole number of 16-byte units.
    """
    es = 4 if dtype == DTYPE_F32 else 2
    unit = 16 // es
    ldu, ldv = _pad(J, unit), _pad(D, unit)
    cap_p = (nnz_capacity // P) if v_sparse else 0
    u_bytes = _pad(B * ldu * es)
    if v_sparse:
        rp_bytes, idx_bytes, val_bytes = _pad((B + 1) * 4), _pad(cap_p * 4), _pad(cap_p * es)
        v_bytes = rp_bytes + idx_bytes + val_bytes
    else:
        rp_bytes = idx_bytes = val_bytes = 0
        v_bytes = _pad(B * ldv * es)
    stream_stride = u_bytes + v_bytes
    streams_off = HEADER_BYTES + _pad(P * DIR_ENTRY_BYTES)
    return dict(es=es, ldu=ldu, ldv=ldv, cap_p=cap_p, u_bytes=u_bytes, v_bytes=v_bytes,
                rp_bytes=rp_bytes, idx_bytes=idx_bytes, val_bytes=val_bytes,
                stream_stride=stream_stride, streams_off=streams_off,
                total_bytes=streams_off + P * stream_stride)


FLAG_V_SPARSE, FLAG_COMPACT = 1, 2


def _wire_round(mat, dtype):
    """Values as they sit on the wire (fp32, or bf16 round-to-nearest-even), returned as fp32."""
    m32 = np.asarray(mat, dtype=np.float64).astype(np.float32)
    if dtype == DTYPE_F32:
        return m32
    return (_bf16_bits(m32).astype(np.uint32) << np.uint32(16)).view(np.float32)


def compact_pairs(U, V, P, B):
    """Inactive-pair compaction (Section 6.1: the sufficient factors are sparse and that is used).

    A pair whose u is all zeros (a dissimilar DML pair beyond the margin) contributes u v^T = 0, so a worker need
    not send it.  Per worker, the pairs with a nonzero u move to the front of the worker's B slots in their original
    order; the slots behind them are zero.  Returns (U_c, V_c, n_sf) with n_sf[p] the number of pairs kept.
    """
    U, V = np.asarray(U), np.asarray(V)
    Uc, Vc = np.zeros_like(U), np.zeros_like(V)
    n_sf = []
    for p in range(P):
        rows = [i for i in range(p * B, (p + 1) * B) if np.any(U[i] != 0)]
        for k, i in enumerate(rows):
            Uc[p * B + k] = U[i]
            Vc[p * B + k] = V[i]
        n_sf.append(len(rows))
    return Uc, Vc, n_sf


def pack(model, dtype, J, D, P, B, U, V=None, csr=None, clock=0, nnz_capacity=0, compact=False):
    """Serialise K = P*B (u, v) pairs as P worker streams.  Returns a uint8 array.

    U: [K][J] values (rounded here to the wire dtype, round to nearest even).
    V: [K][D] values for dense v; csr = (rowptr[K+1], idx, val) for sparse v.
    compact (dense v only): pairs whose wire u is all zeros are left out as `compact_pairs` describes; the
    directory then carries each worker's own pair count and header flag bit 1 is set.  The slot layout (offsets,
    strides) is unchanged, so a receiver reads the first n_sf rows of a worker's U and V blocks.
    """
    v_sparse = csr is not None
    lay = sf_layout(model, dtype, J, D, P, B, v_sparse, nnz_capacity)
    buf = np.zeros(lay["total_bytes"], dtype=np.uint8)
    flags = FLAG_V_SPARSE if v_sparse else 0
    n_sf = [B] * P
    if compact:
        if v_sparse:
            raise ValueError("compaction is defined for dense v")
        U, V, n_sf = compact_pairs(_wire_round(U, dtype), _wire_round(V, dtype), P, B)
        flags |= FLAG_COMPACT
    hdr = struct.pack("<IHBBIIIIIIIIQQQI", MAGIC, VERSION, model, dtype, flags, P, B, J, D, clock,
                      lay["ldu"], lay["ldv"], lay["stream_stride"], lay["total_bytes"],
                      lay["streams_off"], lay["cap_p"])
    buf[:len(hdr)] = np.frombuffer(hdr, dtype=np.uint8)

    def put_vals(off, rows, ld, mat):
        m32 = np.zeros((rows, ld), dtype=np.float32)
        m32[:, :mat.shape[1]] = np.asarray(mat, dtype=np.float64).astype(np.float32)
        raw = m32 if dtype == DTYPE_F32 else _bf16_bits(m32)
        b = raw.reshape(-1).view(np.uint8)
        buf[off:off + b.size] = b

    for p in range(P):
        s_off = lay["streams_off"] + p * lay["stream_stride"]
        u_off, v_off = s_off, s_off + lay["u_bytes"]
        nnz_p = 0
        put_vals(u_off, B, lay["ldu"], np.asarray(U)[p * B:(p + 1) * B])
        if v_sparse:
            rowptr, idx, val = csr
            base = int(rowptr[p * B])
            rp = (np.asarray(rowptr[p * B:(p + 1) * B + 1], dtype=np.int64) - base).astype(np.uint32)
            nnz_p = int(rp[-1])
            if nnz_p > lay["cap_p"]:
                raise ValueError("worker stream exceeds CSR capacity")
            buf[v_off:v_off + rp.size * 4] = rp.view(np.uint8)
            io = v_off + lay["rp_bytes"]
            ib = np.asarray(idx[base:base + nnz_p], dtype=np.uint32)
            buf[io:io + nnz_p * 4] = ib.view(np.uint8)
            vo = io + lay["idx_bytes"]
            v32 = np.asarray(val[base:base + nnz_p], dtype=np.float32)
            vb = v32 if dtype == DTYPE_F32 else _bf16_bits(v32)
            buf[vo:vo + vb.size * lay["es"]] = vb.view(np.uint8)
        else:
            put_vals(v_off, B, lay["ldv"], np.asarray(V)[p * B:(p + 1) * B])
        ent = struct.pack("<IIIIQQ", p, n_sf[p], clock, nnz_p, u_off, v_off)
        d_off = HEADER_BYTES + p * DIR_ENTRY_BYTES
        buf[d_off:d_off + DIR_ENTRY_BYTES] = np.frombuffer(ent, dtype=np.uint8)
    return buf


def parse_header(buf):
    f = struct.unpack_from("<IHBBIIIIIIIIQQQI", bytes(buf[:HEADER_BYTES]))
    names = ("magic", "version", "model", "dtype", "flags", "P", "B", "J", "D", "clock", "ldu", "ldv",
             "stream_stride", "total_bytes", "streams_off", "cap_p")
    return dict(zip(names, f))


def wire_bytes(buf):
    """Bytes a broadcast of this buffer carries (Section 5.1 counts these per worker pair): header, directory, and
    per worker its first n_sf rows of U and of dense V, or all B rows of U plus row pointers and nnz (index, value)
    pairs for sparse v.  Padding is not sent."""
    h = parse_header(buf)
    P, B, J, D = h["P"], h["B"], h["J"], h["D"]
    es = 4 if h["dtype"] == DTYPE_F32 else 2
    total = HEADER_BYTES + P * DIR_ENTRY_BYTES
    for p in range(P):
        _, n_sf, _, nnz_p, _, _ = struct.unpack_from(
            "<IIIIQQ", bytes(buf[HEADER_BYTES + p * DIR_ENTRY_BYTES:HEADER_BYTES + (p + 1) * DIR_ENTRY_BYTES]))
        if h["flags"] & FLAG_V_SPARSE:
            total += n_sf * J * es + (B + 1) * 4 + nnz_p * (4 + es)
        else:
            total += n_sf * (J + D) * es
    return total


def unpack(buf):
    """Inverse of `pack`: returns header dict, U [K][J] fp32, and V [K][D] fp32 or CSR (rowptr, idx, val).

    The header dict also carries "n_sf", the per-worker pair counts of the directory (all B unless the buffer is
    compacted; the rows behind a worker's n_sf are returned as stored, i.e. zeros)."""
    h = parse_header(buf)
    h["n_sf"] = []
    P, B, J, D = h["P"], h["B"], h["J"], h["D"]
    lay = sf_layout(h["model"], h["dtype"], J, D, P, B, bool(h["flags"] & 1), h["cap_p"] * P)
    es = lay["es"]

    def get_vals(off, rows, ld, cols):
        raw = buf[off:off + rows * ld * es]
        if es == 4:
            m = raw.view(np.float32).reshape(rows, ld)
        else:
            m = (raw.view(np.uint16).astype(np.uint32) << np.uint32(16)).view(np.float32).reshape(rows, ld)
        return m[:, :cols].copy()

    U = np.empty((P * B, J), dtype=np.float32)
    V = None if h["flags"] & 1 else np.empty((P * B, D), dtype=np.float32)
    rowptr, idx, val = [0], [], []
    for p in range(P):
        wid, n_sf, clk, nnz_p, u_off, v_off = struct.unpack_from(
            "<IIIIQQ", bytes(buf[HEADER_BYTES + p * DIR_ENTRY_BYTES:HEADER_BYTES + (p + 1) * DIR_ENTRY_BYTES]))
        h["n_sf"].append(n_sf)
        U[p * B:(p + 1) * B] = get_vals(u_off, B, lay["ldu"], J)
        if V is not None:
            V[p * B:(p + 1) * B] = get_vals(v_off, B, lay["ldv"], D)
        else:
            rp = buf[v_off:v_off + (B + 1) * 4].view(np.uint32)
            io = v_off + lay["rp_bytes"]
            vo = io + lay["idx_bytes"]
            idx.append(buf[io:io + nnz_p * 4].view(np.uint32).copy())
            vraw = buf[vo:vo + nnz_p * es]
            val.append(vraw.view(np.float32).copy() if es == 4 else
                       (vraw.view(np.uint16).astype(np.uint32) << np.uint32(16)).view(np.float32))
            rowptr.extend((rp[1:].astype(np.int64) + rowptr[p * B]).tolist())
    if V is not None:
        return h, U, V
    return h, U, (np.asarray(rowptr, dtype=np.uint32), np.concatenate(idx) if idx else np.zeros(0, np.uint32),
                  np.concatenate(val) if val else np.zeros(0, np.float32))


# --------------------------------------------------------------------------------------
# Parity metric
# --------------------------------------------------------------------------------------
def rel_fro(a, b):
    """||a - b||_F / ||b||_F with b the oracle's value."""
    a, b = _f64(a), _f64(b)
    nb = np.linalg.norm(b)
    return float(np.linalg.norm(a - b) / nb) if nb > 0 else float(np.linalg.norm(a - b))

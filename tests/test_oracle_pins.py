"""Pins the fp64 oracle to things other than itself.

Each test re-derives a result by a different route (explicit Python loops over the
definition, a brute-force full-matrix gradient that never forms u, central finite
differences of an independently written loss, a closed form, an SVD) so that a dropped
term, a wrong sign or index, or a transposed operand in the oracle fails at least one.
"""
import math

import numpy as np
import pytest

from oracle import sfb_oracle as orc
from sfbgen import make_inputs, scaled

RNG = np.random.default_rng(12345)


# ----------------------------------------------------------------------------- helpers
def loop_softmax(z):
    m = max(z)
    e = [math.exp(v - m) for v in z]
    s = sum(e)
    return [v / s for v in e]


def loop_matvec(W, a):
    return [sum(W[j][d] * a[d] for d in range(len(a))) for j in range(len(W))]


def loop_mlr_loss(W, X, y):
    tot = 0.0
    for i in range(len(X)):
        z = loop_matvec(W, X[i])
        m = max(z)
        tot += m + math.log(sum(math.exp(v - m) for v in z)) - z[y[i]]
    return tot


def loop_dml_loss(L, Xa, Xb, sim, margin):
    tot = 0.0
    for i in range(len(Xa)):
        d = [float(np.float32(Xa[i][k]) - np.float32(Xb[i][k])) for k in range(len(Xa[i]))]
        z = loop_matvec(L, d)
        n = sum(v * v for v in z)
        tot += 0.5 * n if sim[i] else 0.5 * max(0.0, margin - n)
    return tot


def loop_sc_loss(W, A, X):
    tot = 0.0
    for i in range(len(A)):
        z = loop_matvec(W, A[i])
        tot += 0.5 * sum((z[j] - X[i][j]) ** 2 for j in range(len(z)))
    return tot


def central_fd(loss, W, h=1e-5):
    W = np.array(W, dtype=np.float64)
    G = np.zeros_like(W)
    for j in range(W.shape[0]):
        for d in range(W.shape[1]):
            w0 = W[j, d]
            W[j, d] = w0 + h
            lp = loss(W.tolist())
            W[j, d] = w0 - h
            lm = loss(W.tolist())
            W[j, d] = w0
            G[j, d] = (lp - lm) / (2 * h)
    return G


def dense_to_csr(A):
    rowptr, idx, val = [0], [], []
    for row in A:
        nz = np.nonzero(row)[0]
        idx.extend(nz.tolist())
        val.extend(row[nz].tolist())
        rowptr.append(len(idx))
    return np.array(rowptr, np.uint32), np.array(idx, np.uint32), np.array(val, np.float32)


def tiny_mlr(J=5, D=7, K=6):
    W = RNG.normal(0, 0.5, (J, D)).astype(np.float32)
    X = RNG.normal(0, 1, (K, D)).astype(np.float32)
    y = RNG.integers(0, J, K).astype(np.int32)
    return W, X, y


# ----------------------------------------------------------------------------- MLR
def test_mlr_u_matches_definition_by_loops():
    W, X, y = tiny_mlr()
    U, V = orc.mlr_factors(W, X, y)
    for i in range(len(X)):
        p = loop_softmax(loop_matvec(W.astype(np.float64).tolist(), X[i].astype(np.float64).tolist()))
        p[y[i]] -= 1.0
        assert np.allclose(U[i], p, rtol=0, atol=1e-14)
    assert np.array_equal(V, X.astype(np.float64))


def test_mlr_sf_update_equals_bruteforce_gradient():
    # G[j][d] = sum_i softmax(z_i)[j] x_i[d]  -  sum_{i: y_i = j} x_i[d]   (never forms u)
    W, X, y = tiny_mlr(J=6, D=9, K=11)
    U, V = orc.mlr_factors(W, X, y)
    W64, X64 = W.astype(np.float64), X.astype(np.float64)
    G = np.zeros_like(W64)
    for i in range(len(X)):
        p = loop_softmax(loop_matvec(W64.tolist(), X64[i].tolist()))
        for j in range(W.shape[0]):
            G[j] += p[j] * X64[i]
    for i in range(len(X)):
        G[y[i]] -= X64[i]
    assert orc.rel_fro(orc.delta_w(U, V), G) <= 1e-12


def test_mlr_gradient_by_finite_differences_c0():
    # The whole tiny workload C0 (10 x 64, K = 32): 640 parameters.
    cfg = scaled("C0")
    inp = make_inputs(cfg)
    W, X, y = inp["W"], inp["X"][0], inp["labels"][0]
    U, V = orc.mlr_factors(W, X, y)
    X64, yl = X.astype(np.float64).tolist(), y.tolist()
    G = central_fd(lambda Wl: loop_mlr_loss(Wl, X64, yl), W)
    assert orc.rel_fro(orc.delta_w(U, V), G) <= 1e-7
    # the oracle's own loss agrees with the loop loss
    assert abs(orc.mlr_loss(W, X, y) - loop_mlr_loss(W.astype(np.float64).tolist(), X64, yl)) <= 1e-10


def test_mlr_u_rows_sum_to_zero_and_rank_bounds():
    cfg = scaled("C0")
    inp = make_inputs(cfg)
    U, V = orc.mlr_factors(inp["W"], inp["X"][0], inp["labels"][0])
    assert np.abs(U.sum(axis=1)).max() <= 1e-14
    # C0 has J = 10 < K = 32: 1^T dW = 0 gives rank <= J - 1 = 9
    s = np.linalg.svd(orc.delta_w(U, V), compute_uv=False)
    assert s[9] <= 1e-12 * s[0]
    # K = 4 < min(J, D): rank <= K
    s4 = np.linalg.svd(orc.delta_w(U[:4], V[:4]), compute_uv=False)
    assert s4[3] > 1e-8 * s4[0]
    assert s4[4] <= 1e-12 * s4[0]


def test_mlr_closed_form_at_w_zero():
    J, D, K = 7, 5, 9
    X = RNG.normal(0, 1, (K, D)).astype(np.float32)
    y = RNG.integers(0, J, K).astype(np.int32)
    U, V = orc.mlr_factors(np.zeros((J, D), np.float32), X, y)
    expect = np.tile(X.astype(np.float64).sum(axis=0) / J, (J, 1))
    for i in range(K):
        expect[y[i]] -= X[i].astype(np.float64)
    assert np.allclose(orc.delta_w(U, V), expect, rtol=0, atol=1e-13)


def test_mlr_two_classes_is_binary_logistic_regression():
    W, X, y = tiny_mlr(J=2, D=4, K=8)
    U, _ = orc.mlr_factors(W, X, y)
    Z = X.astype(np.float64) @ W.astype(np.float64).T
    sig = 1.0 / (1.0 + np.exp(-(Z[:, 0] - Z[:, 1])))
    assert np.allclose(U[:, 0], sig - (y == 0), atol=1e-14)
    assert np.allclose(U[:, 1], -U[:, 0], atol=1e-14)


# ----------------------------------------------------------------------------- DML
def tiny_dml(J=6, D=16, K=12, scale=0.25):
    L = RNG.normal(0, scale / math.sqrt(D), (J, D)).astype(np.float32)
    Xa = RNG.normal(0, 1, (K, D)).astype(np.float32)
    Xb = RNG.normal(0, 1, (K, D)).astype(np.float32)
    sim = (np.arange(K) % 2 == 0).astype(np.uint8)
    return L, Xa, Xb, sim


def test_dml_gradient_by_finite_differences_and_scatter_matrix():
    L, Xa, Xb, sim = tiny_dml()
    U, V, n, active = orc.dml_factors(L, Xa, Xb, sim, 1.0)
    dis = ~sim.astype(bool)
    assert active[dis].any() and (~active[dis]).any()           # both hinge branches exercised
    assert np.abs(n[dis] - 1.0).min() > 1e-3                      # away from the kink
    G_fd = central_fd(lambda Ll: loop_dml_loss(Ll, Xa.tolist(), Xb.tolist(), sim.tolist(), 1.0), L)
    assert orc.rel_fro(orc.delta_w(U, V), G_fd) <= 1e-7
    # brute force through the D x D scatter matrices: G = L (sum_sim d d^T - sum_{dis, active} d d^T)
    Dm = (Xa - Xb).astype(np.float64)
    S = np.zeros((Dm.shape[1], Dm.shape[1]))
    for i in range(len(Dm)):
        if sim[i]:
            S += np.outer(Dm[i], Dm[i])
        elif sum(v * v for v in loop_matvec(L.astype(np.float64).tolist(), Dm[i].tolist())) < 1.0:
            S -= np.outer(Dm[i], Dm[i])
    assert orc.rel_fro(orc.delta_w(U, V), L.astype(np.float64) @ S) <= 1e-12
    assert np.array_equal(V, Dm)


def test_dml_special_cases():
    L, Xa, Xb, sim = tiny_dml()
    # L = 0 -> U = 0 -> L unchanged
    U0, V0, _, _ = orc.dml_factors(np.zeros_like(L), Xa, Xb, sim)
    assert not U0.any()
    assert np.array_equal(orc.apply_dense(np.zeros_like(L), U0, V0, 0.3), np.zeros(L.shape))
    # all similar -> dL = L (D^T D)
    allsim = np.ones(len(Xa), np.uint8)
    U, V, _, _ = orc.dml_factors(L, Xa, Xb, allsim)
    Dm = (Xa - Xb).astype(np.float64)
    assert orc.rel_fro(orc.delta_w(U, V), L.astype(np.float64) @ (Dm.T @ Dm)) <= 1e-13
    # a dissimilar pair beyond the margin contributes nothing; strictness at equality
    big = np.float32(50.0)
    Ud, _, nd, act = orc.dml_factors(L, Xa * big, Xb * big, np.zeros(len(Xa), np.uint8))
    assert (nd >= 1.0).all() and not act.any() and not Ud.any()
    L1 = np.array([[1.0, 0.0]], np.float32)
    _, _, n1, a1 = orc.dml_factors(L1, np.array([[1.0, 0.0]], np.float32), np.zeros((1, 2), np.float32), [0])
    assert n1[0] == 1.0 and not a1[0]
    # scaling a similar pair's difference by c scales its contribution by c^2 (c a power of two: exact)
    U1, V1, _, _ = orc.dml_factors(L, Xa[:1], Xb[:1], [1])
    U2, V2, _, _ = orc.dml_factors(L, Xa[:1] * np.float32(2), Xb[:1] * np.float32(2), [1])
    assert np.allclose(orc.delta_w(U2, V2), 4.0 * orc.delta_w(U1, V1), rtol=1e-15)
    # sign of an active dissimilar pair is the opposite of a similar one
    small = np.float32(1e-3)
    Us, _, _, _ = orc.dml_factors(L, Xa[:1] * small, Xb[:1] * small, [1])
    Un, _, _, an = orc.dml_factors(L, Xa[:1] * small, Xb[:1] * small, [0])
    assert an[0] and np.array_equal(Un, -Us)


# ----------------------------------------------------------------------------- SC
def tiny_sc(J=8, D=20, K=6, density=0.3):
    W = RNG.normal(0, 1, (J, D)).astype(np.float32)
    A = (RNG.normal(0, 1, (K, D)) * (RNG.random((K, D)) < density)).astype(np.float32)
    X = RNG.normal(0, 1, (K, J)).astype(np.float32)
    return W, A, X


def test_sc_gradient_fd_gram_route_and_sparse_equals_dense():
    W, A, X = tiny_sc()
    rowptr, idx, val = dense_to_csr(A)
    U = orc.sc_factors(W, rowptr, idx, val, X)
    W64, A64, X64 = (m.astype(np.float64) for m in (W, A, X))
    for i in range(len(A)):
        z = loop_matvec(W64.tolist(), A64[i].tolist())
        assert np.allclose(U[i], np.array(z) - X64[i], atol=1e-13)
    dW = orc.delta_w(U, orc.csr_to_dense(rowptr, idx, val, W.shape[1]))
    assert orc.rel_fro(dW, W64 @ (A64.T @ A64) - X64.T @ A64) <= 1e-12        # Gram-matrix route
    G_fd = central_fd(lambda Wl: loop_sc_loss(Wl, A64.tolist(), X64.tolist()), W)
    assert orc.rel_fro(dW, G_fd) <= 1e-7
    Wn_sparse = orc.apply_sparse(W, U, rowptr, idx, val, 0.01)
    assert np.allclose(Wn_sparse, W64 - 0.01 * dW, rtol=0, atol=1e-14)
    assert abs(orc.sc_loss(W, rowptr, idx, val, X) - loop_sc_loss(W64.tolist(), A64.tolist(), X64.tolist())) < 1e-10


def test_sc_special_cases():
    W, A, X = tiny_sc()
    rowptr, idx, val = dense_to_csr(A)
    # fixed point: x_i = W a_i exactly -> u = 0 -> W unchanged
    Xfix = (A.astype(np.float64) @ W.astype(np.float64).T)
    U = orc.sc_factors(W, rowptr, idx, val, Xfix)
    assert np.abs(U).max() <= 1e-14
    # one-hot code a = c e_j: only column j changes, W[:,j] <- W[:,j] - eta c (c W[:,j] - x)
    j, c, eta = 3, 1.5, 0.2
    rp1, ix1, vl1 = np.array([0, 1], np.uint32), np.array([j], np.uint32), np.array([c], np.float32)
    x = X[:1]
    U1 = orc.sc_factors(W, rp1, ix1, vl1, x)
    Wn = orc.apply_sparse(W, U1, rp1, ix1, vl1, eta)
    expect = W.astype(np.float64)
    expect[:, j] -= eta * c * (c * W[:, j].astype(np.float64) - x[0])
    assert np.allclose(Wn, expect, atol=1e-15)
    # with c = 1 and eta = 1 the column becomes x exactly
    vl1[0] = 1.0
    Wn1 = orc.apply_sparse(W, orc.sc_factors(W, rp1, ix1, vl1, x), rp1, ix1, vl1, 1.0)
    assert np.allclose(Wn1[:, j], x[0].astype(np.float64), atol=1e-15)
    # columns of atoms no code uses are bit-identical before and after
    used = np.zeros(W.shape[1], bool)
    used[idx] = True
    Wn2 = orc.apply_sparse(W, orc.sc_factors(W, rowptr, idx, val, X), rowptr, idx, val, 0.1)
    assert (~used).any()
    assert np.array_equal(Wn2[:, ~used], W.astype(np.float64)[:, ~used])


def test_sc_prox_projects_columns_onto_the_unit_ball():
    W = np.array([[3.0, 0.3, 0.0, 1.0], [4.0, 0.4, 0.0, 0.0]])
    Wp = orc.prox_unit_columns(W)
    assert np.allclose(Wp[:, 0], [0.6, 0.8], atol=1e-15)           # norm 5 -> divided by 5
    assert np.array_equal(Wp[:, 1:], W[:, 1:])                       # norms 0.5, 0, exactly 1: untouched
    R = RNG.normal(0, 1, (9, 13))
    Rp = orc.prox_unit_columns(R)
    n0, n1 = np.linalg.norm(R, axis=0), np.linalg.norm(Rp, axis=0)
    assert (n1 <= 1 + 1e-15).all() and np.allclose(n1[n0 > 1], 1.0, atol=1e-15)
    assert np.array_equal(Rp[:, n0 <= 1], R[:, n0 <= 1])
    assert np.allclose(orc.prox_unit_columns(Rp), Rp, atol=1e-15)   # idempotent
    cos = (R * Rp).sum(axis=0) / (n0 * n1)
    assert np.allclose(cos, 1.0, atol=1e-14)                          # direction preserved


# ----------------------------------------------------------------------------- apply
def test_apply_is_the_sum_of_outer_products_and_is_additive_linear_permutation_invariant():
    J, D, K = 5, 7, 9
    W = RNG.normal(0, 1, (J, D))
    U = RNG.normal(0, 1, (K, J))
    V = RNG.normal(0, 1, (K, D))
    # apply-to-zero with eta = -1 is U^T V; checked by the triple loop of the definition
    T = orc.apply_dense(np.zeros((J, D)), U, V, -1.0)
    ref = np.zeros((J, D))
    for i in range(K):
        for j in range(J):
            for d in range(D):
                ref[j, d] += U[i, j] * V[i, d]
    assert np.allclose(T, ref, atol=1e-14)
    full = orc.apply_dense(W, U, V, 0.3)
    assert np.allclose(full, W - 0.3 * ref, atol=1e-14)
    # additivity over a split of the SFs (how workers' streams are applied)
    half = orc.apply_dense(orc.apply_dense(W, U[:4], V[:4], 0.3), U[4:], V[4:], 0.3)
    assert np.allclose(half, full, atol=1e-14)
    # eta-linearity and permutation invariance
    two = orc.apply_dense(orc.apply_dense(W, U, V, 0.1), U, V, 0.2)
    assert np.allclose(two, full, atol=1e-14)
    perm = RNG.permutation(K)
    assert np.allclose(orc.apply_dense(W, U[perm], V[perm], 0.3), full, atol=1e-14)


def test_step_is_independent_of_the_worker_split_and_lowers_the_loss():
    cfg = scaled("C0")
    inp = make_inputs(cfg)
    batch = dict(X=inp["X"][0], labels=inp["labels"][0])
    W1, U, V = orc.step(orc.MODEL_MLR, inp["W"], batch, cfg["eta"] / cfg["K"])
    # the same K pairs split as (P,B) = (1,32), (4,8), (32,1) unpack to identical factors
    for P, B in ((1, 32), (4, 8), (32, 1)):
        buf = orc.pack(orc.MODEL_MLR, orc.DTYPE_F32, cfg["J"], cfg["D"], P, B, U, V)
        _, U2, V2 = orc.unpack(buf)
        assert np.array_equal(U2, U.astype(np.float32)) and np.array_equal(V2, V.astype(np.float32))
    assert orc.mlr_loss(W1, batch["X"], batch["labels"]) < orc.mlr_loss(inp["W"], batch["X"], batch["labels"])


# ----------------------------------------------------------------------------- pack
def test_pack_header_directory_and_alignment():
    J, D, P, B = 10, 64, 4, 8
    U = RNG.normal(0, 1, (P * B, J))
    V = RNG.normal(0, 1, (P * B, D))
    buf = orc.pack(orc.MODEL_MLR, orc.DTYPE_F32, J, D, P, B, U, V, clock=7)
    h = orc.parse_header(buf)
    assert h["magic"] == 0x31424653 and bytes(buf[:4]) == b"SFB1"
    assert (h["version"], h["model"], h["dtype"], h["flags"]) == (1, 0, 0, 0)
    assert (h["P"], h["B"], h["J"], h["D"], h["clock"]) == (P, B, J, D, 7)
    assert h["ldu"] == 12 and h["ldv"] == 64            # 10 floats -> 48 bytes = 3 x 16
    assert h["total_bytes"] == buf.size
    assert h["streams_off"] == 128 + 128 and h["stream_stride"] % 128 == 0
    assert h["stream_stride"] == 384 + 2048             # B*ldu*4 = 384 ; B*ldv*4 = 2048
    for p in range(P):
        e = np.frombuffer(bytes(buf[128 + 32 * p:160 + 32 * p]), dtype=np.uint32)
        assert (e[0], e[1], e[2], e[3]) == (p, B, 7, 0)
        u_off, v_off = np.frombuffer(bytes(buf[128 + 32 * p + 16:160 + 32 * p]), dtype=np.uint64)
        assert u_off == h["streams_off"] + p * h["stream_stride"] and v_off == u_off + 384
        row = buf[int(u_off):int(u_off) + 48].view(np.float32)
        assert np.array_equal(row[:10], U[p * B].astype(np.float32)) and not row[10:].any()
        vrow = buf[int(v_off) + 256:int(v_off) + 512].view(np.float32)          # second v row of the worker
        assert np.array_equal(vrow, V[p * B + 1].astype(np.float32))
    _, U2, V2 = orc.unpack(buf)
    assert np.array_equal(U2, U.astype(np.float32)) and np.array_equal(V2, V.astype(np.float32))


def test_pack_bf16_rounds_to_nearest_even():
    # 1 + 2^-8 is a tie between 1.0 and 1 + 2^-7 -> even mantissa (1.0); 1 + 3*2^-8 ties up to 1 + 2^-6
    vals = np.array([[1.0, 1.0 + 2.0 ** -8, 1.0 + 3 * 2.0 ** -8, 1.0 + 2.0 ** -8 + 2.0 ** -20, -2.5, 0.0, 3.0e-5, 7.0]])
    buf = orc.pack(orc.MODEL_MLR, orc.DTYPE_BF16, 8, 8, 1, 1, vals, vals)
    h, U, V = orc.unpack(buf)
    assert h["ldu"] == 8 and h["dtype"] == 1
    assert U[0, 0] == 1.0 and U[0, 1] == 1.0 and U[0, 2] == 1.0 + 2.0 ** -6 and U[0, 3] == 1.0 + 2.0 ** -7
    assert U[0, 4] == -2.5 and U[0, 5] == 0.0 and U[0, 7] == 7.0
    assert abs(U[0, 6] - 3.0e-5) <= 3.0e-5 * 2.0 ** -8
    raw = buf[h["streams_off"]:h["streams_off"] + 16].view(np.uint16)
    assert raw[0] == 0x3F80 and raw[4] == 0xC020


def test_pack_sparse_v_roundtrip():
    cfg = scaled("C3", J=16, D=40, P=2, B=3, density=0.2)
    inp = make_inputs(cfg)
    rowptr, idx, val = inp["rowptr"][0], inp["idx"][0], inp["val"][0]
    K = cfg["K"]
    for i in range(K):
        seg = idx[rowptr[i]:rowptr[i + 1]]
        assert (np.diff(seg.astype(np.int64)) > 0).all()               # strictly ascending
    U = RNG.normal(0, 1, (K, cfg["J"]))
    buf = orc.pack(orc.MODEL_SC, orc.DTYPE_F32, cfg["J"], cfg["D"], cfg["P"], cfg["B"], U,
                   csr=(rowptr, idx, val), clock=3, nnz_capacity=inp["nnz_capacity"])
    h, U2, (rp2, ix2, vl2) = orc.unpack(buf)
    assert h["flags"] == 1 and h["cap_p"] == inp["nnz_capacity"] // cfg["P"]
    assert np.array_equal(rp2, rowptr) and np.array_equal(ix2, idx) and np.array_equal(vl2, val)
    assert np.array_equal(U2, U.astype(np.float32))
    for p in range(cfg["P"]):
        nnz_p = np.frombuffer(bytes(buf[128 + 32 * p + 12:128 + 32 * p + 16]), dtype=np.uint32)[0]
        assert nnz_p == rowptr[(p + 1) * cfg["B"]] - rowptr[p * cfg["B"]]
    with pytest.raises(ValueError):
        orc.pack(orc.MODEL_SC, orc.DTYPE_F32, cfg["J"], cfg["D"], cfg["P"], cfg["B"], U,
                 csr=(rowptr, idx, val), nnz_capacity=cfg["P"])


def test_losses_closed_forms():
    """Values the definitions fix: W = 0 gives K log J (uniform softmax); L = 0 gives margin / 2 per
    dissimilar pair and 0 per similar pair; a dictionary that reproduces the data exactly gives 0, and
    W = 0 gives half the squared norm of the data.  dml_loss also against the loop version."""
    rng = np.random.default_rng(11)
    K, J, D = 7, 5, 9
    X = rng.standard_normal((K, D)).astype(np.float32)
    y = rng.integers(0, J, K).astype(np.int32)
    assert abs(orc.mlr_loss(np.zeros((J, D), np.float32), X, y) - K * np.log(J)) <= 1e-12
    Xa, Xb = X, rng.standard_normal((K, D)).astype(np.float32)
    sim = np.array([1, 0, 1, 0, 0, 1, 0], np.uint8)
    assert abs(orc.dml_loss(np.zeros((J, D), np.float32), Xa, Xb, sim, 1.5) - 0.5 * 1.5 * 4) <= 1e-12
    L = (0.2 * rng.standard_normal((J, D))).astype(np.float32)
    want = loop_dml_loss(L.astype(np.float64).tolist(), Xa.astype(np.float64).tolist(), Xb.astype(np.float64).tolist(),
                         sim.tolist(), 1.0)
    assert abs(orc.dml_loss(L, Xa, Xb, sim, 1.0) - want) <= 1e-10
    # sparse coding: codes with two nonzeros per sample, data = W a exactly (small integers: exact in fp32)
    W = rng.integers(-3, 4, (J, D)).astype(np.float32)
    rowptr = np.arange(0, 2 * K + 1, 2).astype(np.uint32)
    idx = np.concatenate([np.sort(rng.choice(D, 2, replace=False)) for _ in range(K)]).astype(np.uint32)
    val = rng.integers(1, 4, 2 * K).astype(np.float32)
    A = orc.csr_to_dense(rowptr, idx, val, D)
    Xd = (A @ W.T.astype(np.float64)).astype(np.float32)
    assert orc.sc_loss(W, rowptr, idx, val, Xd) == 0.0
    assert abs(orc.sc_loss(np.zeros_like(W), rowptr, idx, val, Xd) - 0.5 * float((Xd.astype(np.float64) ** 2).sum())) <= 1e-9


# ----------------------------------------------------------------------------- parity metric
def test_rel_fro_hand_values():
    """The metric every GPU tolerance rests on: ||a - b||_F / ||b||_F with b the reference, by hand."""
    # a - b = (3, -1): norm sqrt(10); ||b|| = 5
    assert orc.rel_fro([3.0, 4.0], [0.0, 5.0]) == pytest.approx(math.sqrt(10.0) / 5.0, rel=1e-15)
    # not symmetric: the denominator is the SECOND argument's norm
    assert orc.rel_fro([1.0, 0.0], [0.0, 2.0]) == pytest.approx(math.sqrt(5.0) / 2.0, rel=1e-15)
    assert orc.rel_fro([0.0, 2.0], [1.0, 0.0]) == pytest.approx(math.sqrt(5.0), rel=1e-15)
    # a square root is taken (not the ratio of squared norms), and the norm runs over all entries of a matrix
    a = [[1.0, 2.0], [3.0, 4.0]]
    b = [[1.0, 2.0], [3.0, 0.0]]
    assert orc.rel_fro(a, b) == pytest.approx(4.0 / math.sqrt(14.0), rel=1e-15)
    # scale invariance and the 1e-k reading used by the tolerances
    assert orc.rel_fro([1.0 + 1e-5, 1.0], [1.0, 1.0]) == pytest.approx(1e-5 / math.sqrt(2.0), rel=1e-9)
    # zero reference: the absolute norm of the difference
    assert orc.rel_fro([3.0, 4.0], [0.0, 0.0]) == 5.0
    assert orc.rel_fro([0.0, 0.0], [0.0, 0.0]) == 0.0
    # float32 inputs are promoted, not compared in fp32
    assert orc.rel_fro(np.float32([1.0]), np.float64([1.0 + 1e-12])) == pytest.approx(1e-12, rel=1e-3)


# ----------------------------------------------------------------------------- inactive-pair compaction
def test_compact_pack_hand_example_bytes():
    """Two workers x three slots, J = 2, D = 3, fp32.  Pairs 1, 3 and 4 have u = 0 and are left out: worker 0 keeps
    pairs (0, 2), worker 1 keeps pair 5.  Every offset below is computed by hand from the wire format: header 128 B,
    directory 2 x 32 B padded to 128, so streams start at 256; ldu = 4, ldv = 4 (rows padded to 16 bytes); U block
    3 x 4 x 4 = 48 -> 128 B, V block likewise, stream stride 256."""
    U = np.array([[1, 2], [0, 0], [3, 4], [0, 0], [0, 0], [5, 6]], dtype=np.float64)
    V = np.arange(18, dtype=np.float64).reshape(6, 3) + 1.0
    buf = orc.pack(orc.MODEL_DML, orc.DTYPE_F32, 2, 3, 2, 3, U, V, clock=9, compact=True)
    assert buf.size == 256 + 2 * 256
    assert int(buf[8:12].view(np.uint32)[0]) == 2                       # flags: bit 1 = compacted, bit 0 (sparse v) clear
    assert int(buf[128 + 4:128 + 8].view(np.uint32)[0]) == 2            # worker 0: two pairs kept
    assert int(buf[160 + 4:160 + 8].view(np.uint32)[0]) == 1            # worker 1: one pair kept
    f = lambda off, n: buf[off:off + 4 * n].view(np.float32).tolist()
    assert f(256, 12) == [1, 2, 0, 0, 3, 4, 0, 0, 0, 0, 0, 0]           # worker 0, U block: u_0, u_2, empty slot
    assert f(256 + 128, 12) == [1, 2, 3, 0, 7, 8, 9, 0, 0, 0, 0, 0]     # worker 0, V block: v_0, v_2, empty slot
    assert f(512, 12) == [5, 6, 0, 0, 0, 0, 0, 0, 0, 0, 0, 0]           # worker 1, U block: u_5 only
    assert f(512 + 128, 12) == [16, 17, 18, 0, 0, 0, 0, 0, 0, 0, 0, 0]  # worker 1, V block: v_5 only
    # what a broadcast carries: header + directory entries + three pairs of (2 + 3) fp32 values
    assert orc.wire_bytes(buf) == 128 + 2 * 32 + 3 * 5 * 4
    full = orc.pack(orc.MODEL_DML, orc.DTYPE_F32, 2, 3, 2, 3, U, V, clock=9)
    assert orc.wire_bytes(full) == 128 + 2 * 32 + 6 * 5 * 4


def test_compaction_leaves_the_update_unchanged_and_round_trips():
    """Dropping pairs with u = 0 changes nothing in W' = W - eta sum u v^T; pairs keep their order inside a worker;
    with every pair active the buffer differs from the plain one in the flag bit only."""
    rng = np.random.default_rng(21)
    J, D, P, B = 5, 7, 3, 4
    K = P * B
    L = (0.3 * rng.standard_normal((J, D))).astype(np.float32)
    Xa, Xb = rng.standard_normal((K, D)).astype(np.float32), rng.standard_normal((K, D)).astype(np.float32)
    sim = (np.arange(K) % 2 == 0).astype(np.uint8)
    U, V, n, active = orc.dml_factors(L, Xa, Xb, sim, 1.0)
    assert 0 < (~active).sum() < K                                       # the case has pairs beyond the margin
    buf = orc.pack(orc.MODEL_DML, orc.DTYPE_F32, J, D, P, B, U, V, compact=True)
    h, Uc, Vc = orc.unpack(buf)
    assert h["flags"] == orc.FLAG_COMPACT
    U32 = U.astype(np.float32)
    for p in range(P):
        kept = [i for i in range(p * B, (p + 1) * B) if U32[i].any()]
        assert h["n_sf"][p] == len(kept)
        assert np.array_equal(Uc[p * B:p * B + len(kept)], U32[kept])    # original order inside the worker
        assert np.array_equal(Vc[p * B:p * B + len(kept)], V.astype(np.float32)[kept])
        assert not Uc[p * B + len(kept):(p + 1) * B].any() and not Vc[p * B + len(kept):(p + 1) * B].any()
    W_full = orc.apply_dense(L, U32, V.astype(np.float32), 0.1)
    W_comp = orc.apply_dense(L, Uc, Vc, 0.1)
    assert np.abs(W_full - W_comp).max() <= 1e-15 * np.abs(W_full).max()
    assert sum(h["n_sf"]) == int(active.sum())
    # all pairs active: same bytes except the flag word
    Ua = U.copy()
    Ua[~active] = 1.0
    a, b = (orc.pack(orc.MODEL_DML, orc.DTYPE_F32, J, D, P, B, Ua, V, compact=c) for c in (False, True))
    diff = np.nonzero(a != b)[0]
    assert diff.tolist() == [8]
    with pytest.raises(ValueError):
        orc.pack(orc.MODEL_SC, orc.DTYPE_F32, J, D, P, B, U, csr=(np.zeros(K + 1, np.uint32), np.zeros(0, np.uint32),
                                                                   np.zeros(0, np.float32)), nnz_capacity=32 * P, compact=True)


# ----------------------------------------------------------------------------- SDCA for L2-regularised MLR
def test_sdca_fixed_point_link_and_convergence():
    """The SDCA factor rule is a reading (the paper gives no closed form), so it is pinned by what any correct dual
    coordinate method must satisfy: (1) at u_i = -grad f_i the step is zero; (2) W = (1 / (lam N)) sum_i u_i x_i^T
    holds after every step when W is updated by the rank-K apply with eta = 1 / (lam N); (3) the iterates converge to
    the primal optimum, checked through the primal optimality condition written with independent loops:
    (1/N) sum_i (softmax(W x_i) - e_{y_i}) x_i^T + lam W = 0."""
    rng = np.random.default_rng(5)
    N, J, D, K, lam, step = 12, 4, 6, 3, 0.1, 0.5
    X = rng.standard_normal((N, D)).astype(np.float32)
    y = rng.integers(0, J, N).astype(np.int32)
    W = np.zeros((J, D))
    dual = np.zeros((N, J))
    # (1) fixed point
    G, _ = orc.mlr_factors(W, X[:K], y[:K])
    dU, V, new = orc.sdca_mlr_factors(W, X[:K], y[:K], -G, step)
    assert np.abs(dU).max() == 0.0 and np.array_equal(new, -G) and np.array_equal(V, X[:K].astype(np.float64))
    # first step from zero duals is a damped gradient step: du = step * g
    dU, _, new = orc.sdca_mlr_factors(W, X[:K], y[:K], np.zeros((K, J)), step)
    assert np.allclose(dU, step * G, rtol=0, atol=1e-16) and np.allclose(new, -step * G, rtol=0, atol=1e-16)
    eta = 1.0 / (lam * N)
    for epoch in range(400):
        for b in range(0, N, K):
            sl = slice(b, b + K)
            dU, V, dual[sl] = orc.sdca_mlr_factors(W, X[sl], y[sl], dual[sl], step)
            W = orc.apply_dense(W, dU, V, eta)
        if epoch % 100 == 0:   # (2) primal-dual link
            link = (dual.T @ X.astype(np.float64)) / (lam * N)
            assert np.abs(W - link).max() <= 1e-13
    # (3) primal optimality by loops
    grad = [[lam * W[j][d] for d in range(D)] for j in range(J)]
    for i in range(N):
        p = loop_softmax(loop_matvec(W.tolist(), X[i].astype(np.float64).tolist()))
        for j in range(J):
            g = p[j] - (1.0 if j == y[i] else 0.0)
            for d in range(D):
                grad[j][d] += g * float(X[i][d]) / N
    assert max(abs(v) for row in grad for v in row) <= 1e-9
    assert np.abs(W).max() > 0.05          # a non-trivial optimum
    # at the optimum the duals are minus the gradients of the losses
    G, _ = orc.mlr_factors(W, X, y)
    assert np.abs(dual + G).max() <= 1e-7
